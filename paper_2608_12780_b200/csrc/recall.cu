// Recall diagnostics: how much of a query's exact attention (Eq. 1) the key set S_c of its cluster keeps.
// For each sampled query: the softmax mass on S_c (the "attention recall" of the paper's recall figure) and
// the share kept of the keys whose exact logit is at least the T-th largest (the "important" keys of
// the matched-recall protocol in the supplement).  Not on the hot path; everything is fp64.
//
// Logits are the sequential fp64 dot product over the channels (bf16 x bf16 products are exact in fp64, so
// a fused multiply-add rounds exactly like multiply-then-add) times the scale: the same bits a plain CPU
// loop produces, so the integer outputs can be compared exactly.
#include "scope_internal.cuh"

namespace scope {

namespace {

constexpr int RR = 4;  // sampled rows per block of the logit kernel (they share every key read)

__global__ void __launch_bounds__(256) recall_logits_kernel(RecallArgs a)
{
    __shared__ double qs[RR][kHeadDim];
    const int bh = blockIdx.z, r0 = blockIdx.y * RR;
    const int b = bh / a.H, h = bh % a.H;
    const int64_t base = (int64_t)b * a.sb + (int64_t)h * a.sh;
    for (int e = threadIdx.x; e < RR * kHeadDim; e += blockDim.x) {
        const int r = e / kHeadDim, ch = e % kHeadDim;
        double v = 0.0;
        if (r0 + r < a.rows_per_head) {
            const int tok = a.rows[(size_t)bh * a.rows_per_head + r0 + r];
            if (tok >= 0 && tok < a.N)
                v = (double)__bfloat162float(a.Q[base + (int64_t)tok * a.sn + ch]);
        }
        qs[r][ch] = v;
    }
    __syncthreads();
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= a.N)
        return;
    const uint4 *kp = reinterpret_cast<const uint4 *>(a.K + base + (int64_t)j * a.sn);
    double acc[RR];
#pragma unroll
    for (int r = 0; r < RR; ++r)
        acc[r] = 0.0;
    for (int chunk = 0; chunk < kHeadDim / 8; ++chunk) {
        const uint4 raw = __ldg(kp + chunk);
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const double k0 = (double)__uint_as_float(w[q] << 16), k1 = (double)__uint_as_float(w[q] & 0xffff0000u);
#pragma unroll
            for (int r = 0; r < RR; ++r) {
                acc[r] = fma(qs[r][chunk * 8 + 2 * q], k0, acc[r]);
                acc[r] = fma(qs[r][chunk * 8 + 2 * q + 1], k1, acc[r]);
            }
        }
    }
#pragma unroll
    for (int r = 0; r < RR; ++r)
        if (r0 + r < a.rows_per_head)
            a.logits[((size_t)bh * a.rows_per_head + r0 + r) * a.N + j] = acc[r] * (double)a.scale;
}

// ascending unsigned order == ascending double order
__device__ __forceinline__ unsigned long long ordered_key(double x)
{
    const unsigned long long u = (unsigned long long)__double_as_longlong(x);
    return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}

template <typename T, typename Op>
__device__ T block_reduce(T v, Op op, T *scratch /* 32 */, T identity)
{
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1)
        v = op(v, __shfl_xor_sync(0xffffffffu, v, m));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();
    if (lane == 0)
        scratch[warp] = v;
    __syncthreads();
    v = lane < (int)(blockDim.x >> 5) ? scratch[lane] : identity;
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1)
        v = op(v, __shfl_xor_sync(0xffffffffu, v, m));
    return v;  // every thread holds the result
}

constexpr int RBITS = 11, RBINS = 1 << RBITS;

__global__ void __launch_bounds__(512) recall_reduce_kernel(RecallArgs a)
{
    __shared__ double red[32];
    __shared__ long long redi[32];
    __shared__ int hist[RBINS];
    __shared__ unsigned long long s_prefix;
    __shared__ long long s_remaining;
    const int bh = blockIdx.y, row = bh * a.rows_per_head + blockIdx.x;
    const int tok = a.rows[row];
    if (tok < 0 || tok >= a.N) {  // block-uniform
        if (threadIdx.x == 0) {
            a.mass[row] = nan("");
            a.top_recall[row] = nan("");
            atomicCAS(a.status + ST_CODE, 0, (int)SCOPE_ERR_INVALID_ARG);
        }
        return;
    }
    const double *s = a.logits + (size_t)row * a.N;
    const int c = a.g[(size_t)bh * a.N + tok];
    const size_t crow = (size_t)bh * a.Cq + c;
    const int32_t *S = a.key_indices + a.key_offsets[crow];
    const int len = a.r_c[crow];

    auto dmax = [](double x, double y) { return x > y ? x : y; };
    auto dadd = [](double x, double y) { return x + y; };
    auto iadd = [](long long x, long long y) { return x + y; };

    double mx = -INFINITY;
    for (int j = threadIdx.x; j < a.N; j += blockDim.x)
        mx = dmax(mx, s[j]);
    mx = block_reduce(mx, dmax, red, (double)-INFINITY);
    double z = 0.0, kept = 0.0;
    for (int j = threadIdx.x; j < a.N; j += blockDim.x)
        z += exp(s[j] - mx);
    for (int l = threadIdx.x; l < len; l += blockDim.x)
        kept += exp(s[S[l]] - mx);
    z = block_reduce(z, dadd, red, 0.0);
    kept = block_reduce(kept, dadd, red, 0.0);

    // key of the T-th largest logit: radix descent from the top bits, 11 bits a level (9 on the last)
    if (threadIdx.x == 0) {
        s_prefix = 0ull;
        s_remaining = a.top_count;
    }
    for (int shift = 64 - RBITS; ; shift = shift >= RBITS ? shift - RBITS : 0) {
        const int bits = shift == 0 ? (64 % RBITS == 0 ? RBITS : 64 % RBITS) : RBITS;
        for (int e = threadIdx.x; e < RBINS; e += blockDim.x)
            hist[e] = 0;
        __syncthreads();
        const unsigned long long prefix = s_prefix;
        const int hi_shift = shift + bits;  // bits above the level's field must equal the prefix
        for (int j = threadIdx.x; j < a.N; j += blockDim.x) {
            const unsigned long long k = ordered_key(s[j]);
            if (hi_shift >= 64 || (k >> hi_shift) == (prefix >> hi_shift))
                atomicAdd(&hist[(int)((k >> shift) & ((1u << bits) - 1u))], 1);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            long long rem = s_remaining;
            int bin = (1 << bits) - 1;
            for (; bin > 0; --bin) {  // from the largest keys down
                if (hist[bin] >= rem)
                    break;
                rem -= hist[bin];
            }
            s_remaining = rem;
            s_prefix = prefix | ((unsigned long long)bin << shift);
        }
        __syncthreads();
        if (shift == 0)
            break;
    }
    const unsigned long long thr = s_prefix;
    long long important = 0, hit = 0;
    for (int j = threadIdx.x; j < a.N; j += blockDim.x)
        important += ordered_key(s[j]) >= thr;
    for (int l = threadIdx.x; l < len; l += blockDim.x)
        hit += ordered_key(s[S[l]]) >= thr;
    important = block_reduce(important, iadd, redi, 0ll);
    hit = block_reduce(hit, iadd, redi, 0ll);
    if (threadIdx.x == 0) {
        a.mass[row] = kept / z;
        a.top_recall[row] = (double)hit / (double)important;
    }
}

}  // namespace

void launch_recall(const RecallArgs &a, cudaStream_t st)
{
    const int BH = a.B * a.H;
    dim3 g1((a.N + 255) / 256, (a.rows_per_head + RR - 1) / RR, BH);
    recall_logits_kernel<<<g1, 256, 0, st>>>(a);
    dim3 g2(a.rows_per_head, BH);
    recall_reduce_kernel<<<g2, 512, 0, st>>>(a);
    count_launch(2);
}

}  // namespace scope
