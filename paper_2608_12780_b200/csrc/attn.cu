// Sparse attention of Eq. 11 (Algorithm 1 lines 10-12): every query of cluster c attends to the
// original keys/values listed in S_c.  Flash-style: one block owns a tile of 64 queries of one
// cluster (gathered through the query permutation), streams the cluster's key list in tiles of
// 64 gathered K and V rows (cp.async, double buffered, XOR-swizzled shared memory), keeps the
// running row maximum / row sum in registers and never materialises the logits.  bf16 operands,
// fp32 accumulation on the tensor cores, bf16 output.  With `dense` set the key list is 0..N-1
// and the grouping is the identity, which is Eq. 1.
#include "scope_internal.cuh"

namespace scope {

namespace {

constexpr int BM = kAttnTileRows;  // query rows per block
constexpr int BN = 64;             // keys per tile
constexpr int NT = 128;            // 4 warps x 16 query rows
constexpr int ROW_BYTES = kHeadDim * 2;
constexpr int TILE_BYTES = BN * ROW_BYTES;  // 16 KB

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
// byte offset of 16-byte chunk `chunk` of row `row` inside a swizzled [rows][128] bf16 tile
__device__ __forceinline__ uint32_t swz(int row, int chunk)
{
    return (uint32_t)(row * ROW_BYTES + ((chunk ^ (row & 7)) << 4));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src));
}
__device__ __forceinline__ void cp_async_commit()
{
    asm volatile("cp.async.commit_group;\n" ::);
}
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

__global__ void __launch_bounds__(NT) sparse_attn_kernel(AttnArgs a)
{
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char *sQ = smem;                       // [BM][128] bf16, later the output tile
    unsigned char *sK = smem + BM * ROW_BYTES;      // 2 stages
    unsigned char *sV = sK + 2 * TILE_BYTES;        // 2 stages

    if (!a.dense && a.status[ST_CODE] != 0)
        return;
    const int bh = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = bh / a.H, h = bh % a.H;
    const int64_t base = (int64_t)b * a.sb + (int64_t)h * a.sh;
    const bf16 *Qh = a.Q + base, *Kh = a.K + base, *Vh = a.V + base;
    bf16 *Oh = a.O + base;

    // which cluster / which rows
    int nrows, nkeys;
    const int32_t *rowlist = nullptr;  // tokens of this tile (null: identity)
    const int32_t *keylist = nullptr;  // key indices (null: identity)
    int row0 = 0;
    if (a.dense) {
        row0 = blockIdx.x * BM;
        if (row0 >= a.N)
            return;
        nrows = min(BM, a.N - row0);
        nkeys = a.N;
    } else {
        const int32_t *toff = a.tile_offsets + (size_t)bh * (a.Cq + 1);
        const int x = blockIdx.x;
        if (x >= toff[a.Cq])
            return;
        int lo = 0, hi = a.Cq;  // last c with toff[c] <= x
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            if (toff[mid] <= x)
                lo = mid;
            else
                hi = mid;
        }
        const int c = lo;
        const int32_t *qoff = a.q_offsets + (size_t)bh * (a.Cq + 1);
        const int start = qoff[c] + (x - toff[c]) * BM;
        nrows = min(BM, qoff[c + 1] - start);
        rowlist = a.q_perm + (size_t)bh * a.N + start;
        const size_t row = (size_t)bh * a.Cq + c;
        nkeys = a.r_c[row];
        keylist = a.key_indices + a.key_offsets[row];
    }
    const int ntiles = (nkeys + BN - 1) / BN;

    // copy roles: 16 threads per row, 8 rows per pass
    const int crow = tid >> 4, cchunk = tid & 15;

    // Q tile
    {
#pragma unroll
        for (int i = 0; i < BM / 8; ++i) {
            int r = crow + 8 * i;
            int rr = min(r, nrows - 1);
            int tok = rowlist ? rowlist[rr] : row0 + rr;
            cp_async16(smem_u32(sQ) + swz(r, cchunk), Qh + (int64_t)tok * a.sn + cchunk * 8);
        }
    }
    int kidx[BN / 8];
    auto load_idx = [&](int t) {
#pragma unroll
        for (int i = 0; i < BN / 8; ++i) {
            int j = min(t * BN + crow + 8 * i, nkeys - 1);
            kidx[i] = keylist ? __ldg(keylist + j) : j;
        }
    };
    auto issue_tile = [&](int stage) {
        const uint32_t dk = smem_u32(sK) + stage * TILE_BYTES, dv = smem_u32(sV) + stage * TILE_BYTES;
#pragma unroll
        for (int i = 0; i < BN / 8; ++i) {
            int r = crow + 8 * i;
            const int64_t o = (int64_t)kidx[i] * a.sn + cchunk * 8;
            cp_async16(dk + swz(r, cchunk), Kh + o);
            cp_async16(dv + swz(r, cchunk), Vh + o);
        }
    };
    load_idx(0);
    issue_tile(0);
    cp_async_commit();
    if (ntiles > 1)
        load_idx(1);

    float o_acc[16][4];
#pragma unroll
    for (int n = 0; n < 16; ++n)
#pragma unroll
        for (int q = 0; q < 4; ++q)
            o_acc[n][q] = 0.f;
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
    uint32_t qf[8][4];
    const float sl2 = a.scale * 1.4426950408889634f;

    for (int t = 0; t < ntiles; ++t) {
        const int stage = t & 1;
        if (t + 1 < ntiles) {
            issue_tile(stage ^ 1);
            cp_async_commit();
            if (t + 2 < ntiles)
                load_idx(t + 2);
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        if (t == 0) {
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
                ldsm_x4(smem_u32(sQ) + swz(warp * 16 + (lane & 15), ks * 2 + (lane >> 4)), qf[ks][0], qf[ks][1],
                        qf[ks][2], qf[ks][3]);
        }
        const uint32_t kb = smem_u32(sK) + stage * TILE_BYTES, vb = smem_u32(sV) + stage * TILE_BYTES;

        // S = Q K^T
        float s[8][4];
#pragma unroll
        for (int n = 0; n < 8; ++n)
#pragma unroll
            for (int q = 0; q < 4; ++q)
                s[n][q] = 0.f;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                uint32_t b0, b1, b2, b3;
                int key = np * 16 + (lane & 7) + ((lane >> 4) << 3);
                int chunk = ks * 2 + ((lane >> 3) & 1);
                ldsm_x4(kb + swz(key, chunk), b0, b1, b2, b3);
                mma_bf16(s[2 * np], qf[ks], b0, b1);
                mma_bf16(s[2 * np + 1], qf[ks], b2, b3);
            }
        }
        // mask keys past the end of the list (last tile only)
        const int kvalid = nkeys - t * BN;
        if (kvalid < BN) {
#pragma unroll
            for (int n = 0; n < 8; ++n) {
                int col = n * 8 + (lane & 3) * 2;
                if (col >= kvalid)
                    s[n][0] = s[n][2] = -INFINITY;
                if (col + 1 >= kvalid)
                    s[n][1] = s[n][3] = -INFINITY;
            }
        }
        // online softmax (rows lane/4 and lane/4 + 8 of the warp's 16)
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int n = 0; n < 8; ++n) {
            mx[0] = fmaxf(mx[0], fmaxf(s[n][0], s[n][1]));
            mx[1] = fmaxf(mx[1], fmaxf(s[n][2], s[n][3]));
        }
        float alpha[2], msc[2];
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
            mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 1));
            mx[hh] = fmaxf(mx[hh], __shfl_xor_sync(0xffffffffu, mx[hh], 2));
            float mnew = fmaxf(m_run[hh], mx[hh] * sl2);
            alpha[hh] = exp2f(m_run[hh] - mnew);
            m_run[hh] = mnew;
            msc[hh] = mnew;
        }
        float rs[2] = {0.f, 0.f};
        uint32_t pf[4][4];
#pragma unroll
        for (int n = 0; n < 8; ++n) {
            float p0 = exp2f(fmaf(s[n][0], sl2, -msc[0]));
            float p1 = exp2f(fmaf(s[n][1], sl2, -msc[0]));
            float p2 = exp2f(fmaf(s[n][2], sl2, -msc[1]));
            float p3 = exp2f(fmaf(s[n][3], sl2, -msc[1]));
            rs[0] += p0 + p1;
            rs[1] += p2 + p3;
            pf[n >> 1][(n & 1) * 2] = pack_bf16(p0, p1);
            pf[n >> 1][(n & 1) * 2 + 1] = pack_bf16(p2, p3);
        }
#pragma unroll
        for (int hh = 0; hh < 2; ++hh)
            l_run[hh] = l_run[hh] * alpha[hh] + rs[hh];
#pragma unroll
        for (int n = 0; n < 16; ++n) {
            o_acc[n][0] *= alpha[0];
            o_acc[n][1] *= alpha[0];
            o_acc[n][2] *= alpha[1];
            o_acc[n][3] *= alpha[1];
        }
        // O += P V
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
#pragma unroll
            for (int dp = 0; dp < 8; ++dp) {
                uint32_t b0, b1, b2, b3;
                int key = kk * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
                int chunk = dp * 2 + (lane >> 4);
                ldsm_x4_t(vb + swz(key, chunk), b0, b1, b2, b3);
                mma_bf16(o_acc[2 * dp], pf[kk], b0, b1);
                mma_bf16(o_acc[2 * dp + 1], pf[kk], b2, b3);
            }
        }
        __syncthreads();
    }

    // normalise, stage the tile in shared memory, write whole rows
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
        float l = l_run[hh];
        l += __shfl_xor_sync(0xffffffffu, l, 1);
        l += __shfl_xor_sync(0xffffffffu, l, 2);
        l_run[hh] = 1.f / l;
    }
    {
        const int r0 = warp * 16 + (lane >> 2);
#pragma unroll
        for (int n = 0; n < 16; ++n) {
            // n-tile n covers channels 8n..8n+7 = chunk n; this thread holds 2 of them
            uint32_t lo = pack_bf16(o_acc[n][0] * l_run[0], o_acc[n][1] * l_run[0]);
            uint32_t hi = pack_bf16(o_acc[n][2] * l_run[1], o_acc[n][3] * l_run[1]);
            *reinterpret_cast<uint32_t *>(sQ + swz(r0, n) + (lane & 3) * 4) = lo;
            *reinterpret_cast<uint32_t *>(sQ + swz(r0 + 8, n) + (lane & 3) * 4) = hi;
        }
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < BM / 8; ++i) {
        int r = crow + 8 * i;
        if (r < nrows) {
            int tok = rowlist ? rowlist[r] : row0 + r;
            uint4 v = *reinterpret_cast<const uint4 *>(sQ + swz(r, cchunk));
            *reinterpret_cast<uint4 *>(Oh + (int64_t)tok * a.sn + cchunk * 8) = v;
        }
    }
}

}  // namespace

void launch_attn(const AttnArgs &a, cudaStream_t st)
{
    const int smem = BM * ROW_BYTES + 4 * TILE_BYTES;
    cudaFuncSetAttribute(sparse_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    dim3 grid(a.max_tiles_per_head, a.B * a.H);
    sparse_attn_kernel<<<grid, NT, smem, st>>>(a);
    count_launch();
}

}  // namespace scope
