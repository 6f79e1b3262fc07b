"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every function the
header declares, and rejects bad parameters before touching a device."""
import ctypes as C
import os
import re

import pytest

from paper_2608_12780_b200 import binding as sb
from paper_2608_12780_b200 import build as cuda_build
from paper_2608_12780_b200 import inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    cuda_build.build()  # nvcc cross-compiles without a GPU
    return sb.lib()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "scope.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(scope_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared_functions()
    assert len(names) >= 15
    assert set(names) == set(sb.EXPORTS), "binding and header disagree"
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in scope.h but not exported"


def _params(**kw):
    cfg = inputs.CONFIGS["tiny"]
    p = sb.make_params(cfg)
    for k, v in kw.items():
        setattr(p, k, v)
    return p


def test_workspace_bytes_grow_with_the_problem(lib):
    small = lib.scope_plan_workspace_bytes(C.byref(_params()))
    big = lib.scope_plan_workspace_bytes(C.byref(sb.make_params(inputs.CONFIGS["small"])))
    assert 0 < small < big
    hy = sb.make_params(inputs.CONFIGS["HY720"])
    need = lib.scope_plan_workspace_bytes(C.byref(hy))
    # dominated by the key-index buffer and the per-token arrays
    assert need > hy.index_capacity * 4 and need < hy.index_capacity * 4 + (1 << 30)


@pytest.mark.parametrize("field,value", [
    ("N", 0), ("H", 0), ("d_t", 0), ("d_w", 57), ("Cq", 0), ("Cq", 257), ("Ct", 300), ("kmeans_iters", 0),
    ("top_p", 0.0), ("top_p", -0.5), ("top_p", float("nan")), ("k_fix", 0), ("k_fix", 257), ("scale", -1.0),
    ("index_capacity", 0), ("stride_n", 64),
])
def test_invalid_parameters_are_rejected(lib, field, value):
    assert lib.scope_plan_workspace_bytes(C.byref(_params(**{field: value}))) == 0


def test_partitions_with_fewer_ranges(lib):
    """Trailing key ranges may be empty (two-way and full-dimension partitions); an empty range has exactly one
    centroid, empty ranges come last, and every range holds whole channel pairs."""
    ok = lambda **kw: lib.scope_plan_workspace_bytes(C.byref(_params(**kw))) > 0
    assert ok(d_t=72, d_h=56, d_w=0, Cw=1)
    assert ok(d_t=128, d_h=0, d_w=0, Ch=1, Cw=1)
    assert not ok(d_t=72, d_h=56, d_w=0)             # Cw must be 1
    assert not ok(d_t=72, d_h=0, d_w=56, Ch=1)       # an empty range before a non-empty one
    assert not ok(d_t=0, d_h=64, d_w=64, Ct=1)
    h = C.c_void_p()
    p = _params(d_t=17, d_h=55, d_w=56)
    assert lib.scope_plan_create(C.byref(p), C.c_void_p(1 << 20), 1 << 30, None, C.byref(h)) == sb.SCOPE_ERR_UNSUPPORTED


def test_partitions_with_more_ranges(lib):
    def params(**kw):
        p = _params(**{k: v for k, v in kw.items() if k not in ("d_x", "C_x")})
        for k in ("d_x", "C_x"):
            for i, v in enumerate(kw.get(k, ())):
                getattr(p, k)[i] = v
        return p
    ok = lambda **kw: lib.scope_plan_workspace_bytes(C.byref(params(**kw))) > 0
    assert ok(d_t=32, d_h=32, d_w=32, n_extra=1, d_x=(32,), C_x=(5,))
    assert ok(d_t=16, d_h=16, d_w=16, n_extra=5, d_x=(16,) * 5, C_x=(3, 4, 5, 6, 7))
    assert not ok(d_t=32, d_h=32, d_w=32, n_extra=1, d_x=(30,), C_x=(5,))       # channels do not add up
    assert not ok(d_t=32, d_h=32, d_w=32, n_extra=1, d_x=(32,), C_x=(0,))
    assert not ok(d_t=96, d_h=0, d_w=0, Ch=1, Cw=1, n_extra=1, d_x=(32,), C_x=(5,))  # extras after empty ranges
    assert not ok(d_t=16, d_h=16, d_w=16, n_extra=6, d_x=(16,) * 5, C_x=(3,) * 5)


def test_permute_channels_rejects_bad_arguments(lib):
    p = _params()
    perm = (C.c_int32 * 128)(*range(128))
    x, y = C.c_void_p(1 << 20), C.c_void_p(1 << 24)  # never dereferenced: validation fails first
    assert lib.scope_permute_channels(None, C.byref(p), perm, y, None) == sb.SCOPE_ERR_INVALID_ARG
    assert lib.scope_permute_channels(x, C.byref(p), perm, x, None) == sb.SCOPE_ERR_INVALID_ARG
    perm[5] = 4  # not a permutation
    assert lib.scope_permute_channels(x, C.byref(p), perm, y, None) == sb.SCOPE_ERR_INVALID_ARG
    perm[5] = 128
    assert lib.scope_permute_channels(x, C.byref(p), perm, y, None) == sb.SCOPE_ERR_INVALID_ARG


def test_unsupported_and_alignment_codes(lib):
    h = C.c_void_p()
    ws = C.c_void_p(1 << 20)  # never dereferenced: every call below fails validation first
    p = _params(d=64, d_t=16, d_h=24, d_w=24)
    assert lib.scope_plan_create(C.byref(p), ws, 1 << 30, None, C.byref(h)) == sb.SCOPE_ERR_UNSUPPORTED
    p = _params(Cq=2000, N=4096, k_fix=32)
    assert lib.scope_plan_create(C.byref(p), ws, 1 << 30, None, C.byref(h)) == sb.SCOPE_ERR_UNSUPPORTED
    p = _params(stride_b=2 * 256 * 132, stride_h=256 * 132, stride_n=132)  # 132 elements: not 16-byte rows
    assert lib.scope_plan_create(C.byref(p), ws, 1 << 30, None, C.byref(h)) == sb.SCOPE_ERR_ALIGNMENT
    p = _params()
    assert lib.scope_plan_create(C.byref(p), None, 1 << 30, None, C.byref(h)) == sb.SCOPE_ERR_INVALID_ARG
    assert lib.scope_plan_create(C.byref(p), C.c_void_p((1 << 20) + 16), 1 << 30, None, C.byref(h)) == sb.SCOPE_ERR_ALIGNMENT
    assert lib.scope_plan_create(C.byref(p), ws, 1024, None, C.byref(h)) == sb.SCOPE_ERR_WORKSPACE
    assert lib.scope_plan_create(None, ws, 1 << 30, None, C.byref(h)) == sb.SCOPE_ERR_INVALID_ARG
    assert h.value is None


def test_null_plan_and_pointer_checks(lib):
    assert lib.scope_plan(None, None, None, None) == sb.SCOPE_ERR_INVALID_ARG
    assert lib.scope_forward(None, None, None, None, None, None) == sb.SCOPE_ERR_INVALID_ARG
    assert lib.scope_sparse_attn(None, None, None, None, None, None) == sb.SCOPE_ERR_INVALID_ARG
    assert lib.scope_plan_status(None, None, None) == sb.SCOPE_ERR_INVALID_ARG
    assert lib.scope_plan_rope(None, None, None, None, None) == sb.SCOPE_ERR_INVALID_ARG
    assert lib.scope_recall(None, None, None, None, 4, 0.1, None, 0, None, None, None) == sb.SCOPE_ERR_INVALID_ARG
    assert lib.scope_plan_field_bytes(None, 0) == 0
    lib.scope_plan_destroy(None)


def test_status_strings_and_kfix(lib):
    seen = {sb.status_string(s) for s in range(9)}
    assert len(seen) == 9 and "ok" in seen
    assert sb.status_string(99) == "unknown status"
    assert sb.scope_kfix_from_alpha(118800, 1, 10) == 11880
    assert sb.scope_kfix_from_alpha(75600, 1, 10) == 7560
    assert sb.scope_kfix_from_alpha(7, 1, 10) == 1
    assert sb.scope_kfix_from_alpha(10, 3, 2) == -1 and sb.scope_kfix_from_alpha(0, 1, 10) == -1


def test_missing_library_is_a_hard_error(monkeypatch, tmp_path):
    monkeypatch.setattr(sb, "_lib", None)
    monkeypatch.setattr(sb, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        sb.lib()


def test_product_path_never_touches_the_oracle():
    pkg = os.path.join(ROOT, "paper_2608_12780_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower() or f == "inputs.py", f"{f} mentions the oracle"
