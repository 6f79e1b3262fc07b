// Tensor-core assignment step of the k-means stage (Eq. 3 labels + Eq. 2 member sums in one read
// of X), for codebooks that fit shared memory; kmeans.cu holds the general kernel.
//
// x.u for a tile of 128 tokens against every centroid is one tcgen05 MMA chain: A = the X tile
// (bf16, exact), B = the centroids split into three bf16 terms u = hi + mid + lo (exact to 24
// bits), all three chains accumulating into the same fp32 columns of tensor memory.  Each thread
// then owns one token (one TMEM lane), forms |u|^2 - 2 x.u per centroid and keeps the two smallest.
// As in the general kernel the label is final only if the gap between those two exceeds the
// worst-case rounding error of this pass; otherwise the token is re-evaluated in fp64 with the
// plain sum of squared differences.  Member sums are accumulated in fp64.
//
// A block holds the codebook splits once and runs two independent 128-thread pipelines (token
// tiles alternate between them), so the loads / MMA of one overlap the epilogue of the other.
#include "scope_internal.cuh"
#include "sm100.cuh"

namespace scope {

using namespace sm100;

namespace {

constexpr int TM = 128;          // tokens per tile = MMA M
constexpr int GROUPS = 2;        // independent pipelines per block
constexpr int NT = 128 * GROUPS;
constexpr int HALF_BYTES = TM * 128;           // one 64-channel half of a 128-row tile
constexpr int XTILE_BYTES = 2 * HALF_BYTES;    // 32 KB
constexpr int TMEM_COLS_PER_GROUP = 256;

struct TcLayout {
    int cpad[3];       // centroids padded to a multiple of 16
    int col[3];        // first TMEM column of the space inside a group's 256
    int cent_off[3];   // byte offset of the space's split tiles in shared memory
    int un_off[3];     // float offset of the space's norms
    int cent_bytes;    // all split tiles
    int un_floats;
};

__host__ __device__ inline bool tc_layout(const KmArgs &a, TcLayout &L)
{
    int col = 0, off = 0, un = 0;
    for (int s = 0; s < a.nspaces; ++s) {
        int cp = (a.sp[s].C + 15) & ~15;
        if (cp > 256)
            return false;
        L.cpad[s] = cp;
        L.col[s] = col;
        col += (cp + 31) & ~31;
        L.cent_off[s] = off;
        off += 3 * 2 * cp * 128;  // 3 splits x 2 channel halves x cp rows x 128 B
        L.un_off[s] = un;
        un += cp;
    }
    L.cent_bytes = off;
    L.un_floats = un;
    return col <= TMEM_COLS_PER_GROUP;
}

struct GroupShared {
    int asg[3][TM];
    uint32_t sorted[3][TM];
    float x2[3][TM];
    int flagged[3 * TM];
    int nflagged;
    int dead;
    uint64_t mbar;
};

__global__ void __launch_bounds__(NT, 1) kmeans_assign_tc_kernel(KmArgs a, int tiles_per_block, int32_t *status)
{
    extern __shared__ unsigned char smem_dyn[];
    // 1024-byte alignment for the swizzled tiles
    unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);
    TcLayout L;
    tc_layout(a, L);
    unsigned char *s_cent = smem;
    unsigned char *s_x = s_cent + L.cent_bytes;                       // GROUPS tiles
    float *s_un = reinterpret_cast<float *>(s_x + GROUPS * XTILE_BYTES);
    GroupShared *s_g = reinterpret_cast<GroupShared *>(s_un + ((L.un_floats + 3) & ~3));
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_timeout;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int grp = tid >> 7, gt = tid & 127;       // pipeline, thread within it
    const int bh = blockIdx.y;
    const int b = bh / a.H, h = bh % a.H;
    const bf16 *Xh = a.X + (int64_t)b * a.sb + (int64_t)h * a.sh;
    GroupShared &G = s_g[grp];

    if (warp == 0) {
        tmem_alloc(&s_tmem_base, GROUPS * TMEM_COLS_PER_GROUP);
        tmem_relinquish();
    }
    if (tid == 0)
        s_timeout = 0;
    if (gt == 0) {
        G.dead = 0;
        mbar_init(&G.mbar, 1);
        mbar_fence_init();
    }
    // codebook splits and norms -> shared memory (once per block)
    for (int s = 0; s < a.nspaces; ++s) {
        const int cp = L.cpad[s];
        const bf16 *src = a.sp[s].split + (size_t)bh * 3 * cp * kHeadDim;
        const int nchunks = 3 * cp * 16;  // 16-byte chunks
        for (int e = tid; e < nchunks; e += NT) {
            int chunk = e & 15, row = (e >> 4) % cp, p = (e >> 4) / cp;
            uint32_t dst = smem_u32(s_cent) + L.cent_off[s] + (p * 2 + (chunk >> 3)) * cp * 128 + sw128(row, chunk & 7);
            cp_async16(dst, src + ((size_t)p * cp + row) * kHeadDim + chunk * 8);
        }
        for (int e = tid; e < cp; e += NT)
            s_un[L.un_off[s] + e] = e < a.sp[s].C ? a.sp[s].unorm[(size_t)bh * a.sp[s].C + e] : INFINITY;
    }
    cp_async_commit();
    cp_async_wait<0>();
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem_base + grp * TMEM_COLS_PER_GROUP;
    const uint32_t xbase = smem_u32(s_x) + grp * XTILE_BYTES;
    const int ntiles = (a.N + TM - 1) / TM;
    uint32_t phase = 0;
    bool dead = false;

    for (int ti = grp; ti < tiles_per_block; ti += GROUPS) {
        const int tile = blockIdx.x * tiles_per_block + ti;
        if (tile >= ntiles || dead)
            break;
        const int tok0 = tile * TM;
        if (gt == 0)
            G.nflagged = 0;
        // X tile: 128 rows x 16 chunks; rows past N are zero
        for (int e = gt; e < TM * 16; e += 128) {
            int row = e >> 4, chunk = e & 15;
            bool ok = tok0 + row < a.N;
            const bf16 *src = Xh + (int64_t)(ok ? tok0 + row : 0) * a.sn + chunk * 8;
            cp_async16_zfill(xbase + (chunk >> 3) * HALF_BYTES + sw128(row, chunk & 7), src, ok ? 16 : 0);
        }
        cp_async_commit();
        cp_async_wait<0>();
        fence_proxy_async();
        tc_fence_before();
        bar_sync(1 + grp, 128);
        if (gt == 0) {
            tc_fence_after();
            for (int s = 0; s < a.nspaces; ++s) {
                const int cp = L.cpad[s];
                const uint32_t idesc = idesc_bf16(TM, cp, false, false);
                const int k_lo = a.sp[s].ch0 >> 4, k_hi = (a.sp[s].ch0 + a.sp[s].D + 15) >> 4;
                bool first = true;
                for (int p = 0; p < 3; ++p)
                    for (int ks = k_lo; ks < k_hi; ++ks) {
                        uint64_t da = smem_desc_sw128(xbase + (ks >> 2) * HALF_BYTES + (ks & 3) * 32);
                        uint64_t db = smem_desc_sw128(smem_u32(s_cent) + L.cent_off[s] + (p * 2 + (ks >> 2)) * cp * 128 + (ks & 3) * 32);
                        mma_ss(tmem + L.col[s], da, db, idesc, !first);
                        first = false;
                    }
            }
            mma_commit(&G.mbar);
        }
        // squared norm of the token's slice per space while the MMAs run
        {
            float x2[3] = {0.f, 0.f, 0.f};
#pragma unroll
            for (int chunk = 0; chunk < 16; ++chunk) {
                uint4 raw = *reinterpret_cast<const uint4 *>(s_x + grp * XTILE_BYTES + (chunk >> 3) * HALF_BYTES + sw128(gt, chunk & 7));
                const bf16 *e = reinterpret_cast<const bf16 *>(&raw);
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    int ch = chunk * 8 + q;
                    float v = __bfloat162float(e[q]);
                    int s = (a.nspaces == 1 || ch < a.sp[1].ch0) ? 0 : (ch < a.sp[2].ch0 ? 1 : 2);
                    x2[s] = fmaf(v, v, x2[s]);
                }
            }
            for (int s = 0; s < a.nspaces; ++s)
                G.x2[s][gt] = x2[s];
        }
        // a wait that runs out is recorded and ends this pipeline after the next barrier
        const bool ok = __all_sync(0xffffffffu, mbar_wait(&G.mbar, phase));
        if (!ok) {
            *reinterpret_cast<volatile int *>(&G.dead) = 1;
            atomicExch(&s_timeout, 1);
        }
        phase ^= 1;
        tc_fence_after();
        if (ok) {
            for (int s = 0; s < a.nspaces; ++s) {
                const int C = a.sp[s].C;
                const float *un = s_un + L.un_off[s];
                float best = INFINITY, second = INFINITY;
                int arg = 0;
                for (int c0 = 0; c0 < L.cpad[s]; c0 += 16) {
                    uint32_t r[16];
                    tmem_ld16(tmem + ((uint32_t)((warp & 3) * 32) << 16) + L.col[s] + c0, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        float dist = fmaf(-2.f, __uint_as_float(r[j]), un[c0 + j]);  // padding columns carry +inf norms
                        if (dist < best) {
                            second = best;
                            best = dist;
                            arg = c0 + j;
                        } else if (dist < second) {
                            second = dist;
                        }
                    }
                }
                G.asg[s][gt] = arg;
                const int cbeg = a.sp[s].ch0 & ~15, cend = (a.sp[s].ch0 + a.sp[s].D + 15) & ~15;
                // error budget of two tensor-core evaluations of |u|^2 - 2 x.u: the products are exact, each
                // of the 3 * (channels / 16) accumulating MMAs may lose up to two fp32 ulps of the running
                // magnitude (truncating adds), |x.u| <= (|u|^2 + |x|^2) / 2; doubled for margin
                const float kappa = 8.f * (float)(3 * ((cend - cbeg) >> 4) + 2) * 1.1920929e-7f;
                const float tol = kappa * (__ldg(a.sp[s].u2max + bh) + G.x2[s][gt]);
                if (tok0 + gt < a.N && C > 1 && second - best <= tol) {
                    int slot = atomicAdd(&G.nflagged, 1);
                    G.flagged[slot] = (s << 16) | gt;
                }
            }
        }
        tc_fence_before();
        bar_sync(1 + grp, 128);
        dead = *reinterpret_cast<volatile int *>(&G.dead) != 0;

        // fp64 re-evaluation of the close calls: one warp per token, centroids spread over lanes
        {
            const int nf = dead ? 0 : G.nflagged;
            for (int f = (warp & 3); f < nf; f += 4) {
                const int s = G.flagged[f] >> 16, lt = G.flagged[f] & 0xffff;
                const KmSpace &sp = a.sp[s];
                const float *cent = sp.cent + (size_t)bh * sp.C * sp.D;
                const bf16 *x = Xh + (int64_t)(tok0 + lt) * a.sn + sp.ch0;
                double bd = INFINITY;
                int ba = 0x7fffffff;
                for (int c = lane; c < sp.C; c += 32) {
                    const float *u = cent + (size_t)c * sp.D;
                    double dist = 0.0;
                    for (int ch = 0; ch < sp.D; ++ch) {
                        double diff = __dsub_rn((double)__bfloat162float(x[ch]), (double)u[ch]);
                        dist = __dadd_rn(dist, __dmul_rn(diff, diff));
                    }
                    if (dist < bd) {
                        bd = dist;
                        ba = c;
                    }
                }
#pragma unroll
                for (int m = 16; m >= 1; m >>= 1) {
                    double od = __shfl_xor_sync(0xffffffffu, bd, m);
                    int oa = __shfl_xor_sync(0xffffffffu, ba, m);
                    if (od < bd || (od == bd && oa < ba)) {
                        bd = od;
                        ba = oa;
                    }
                }
                if (lane == 0)
                    G.asg[s][lt] = ba;
            }
        }
        bar_sync(1 + grp, 128);
        if (dead)
            break;

        // labels out
        if (tok0 + gt < a.N) {
            if (a.nspaces == 1)
                a.assign[(size_t)bh * a.N + tok0 + gt] = G.asg[0][gt];
            else
                a.codes[(size_t)bh * a.N + tok0 + gt] = (uint32_t)G.asg[0][gt] | ((uint32_t)G.asg[1][gt] << kCodeBits) |
                                                        ((uint32_t)G.asg[2][gt] << (2 * kCodeBits));
        }
        // order the tile's tokens by label (rank by counting), then add each run of equal labels once
        for (int s = 0; s < a.nspaces; ++s) {
            uint32_t key = (tok0 + gt < a.N ? (uint32_t)G.asg[s][gt] : (uint32_t)kMaxClusters) << 8 | (uint32_t)gt;
            int rank = 0;
            for (int o = 0; o < TM; ++o) {
                uint32_t ok = (tok0 + o < a.N ? (uint32_t)G.asg[s][o] : (uint32_t)kMaxClusters) << 8 | (uint32_t)o;
                rank += ok < key;
            }
            G.sorted[s][rank] = key;
        }
        bar_sync(1 + grp, 128);
        {
            const int ch = gt;
            int s = 0;
            while (s + 1 < a.nspaces && ch >= a.sp[s].ch0 + a.sp[s].D)
                ++s;
            const KmSpace &sp = a.sp[s];
            const int rel = ch - sp.ch0;
            double *sums = sp.sums + (size_t)bh * sp.C * sp.D;
            int32_t *counts = sp.counts + (size_t)bh * sp.C;
            const unsigned char *xcol = s_x + grp * XTILE_BYTES + (ch >> 6) * HALF_BYTES + (ch & 7) * 2;
            const int chunk = (ch & 63) >> 3;
            int cur = -1, run = 0;
            double acc = 0.0;
            for (int l = 0; l < TM; ++l) {
                uint32_t key = G.sorted[s][l];
                int cl = (int)(key >> 8), lt = (int)(key & 255u);
                if (cl >= kMaxClusters)
                    break;
                if (cl != cur) {
                    if (cur >= 0) {
                        atomicAdd(sums + (size_t)cur * sp.D + rel, acc);
                        if (rel == 0)
                            atomicAdd(counts + cur, run);
                    }
                    cur = cl;
                    acc = 0.0;
                    run = 0;
                }
                acc += (double)__bfloat162float(*reinterpret_cast<const bf16 *>(xcol + sw128(lt, chunk)));
                ++run;
            }
            if (cur >= 0) {
                atomicAdd(sums + (size_t)cur * sp.D + rel, acc);
                if (rel == 0)
                    atomicAdd(counts + cur, run);
            }
        }
        bar_sync(1 + grp, 128);  // the X tile and the label arrays are reused by the next tile
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0)
        tmem_dealloc(s_tmem_base, GROUPS * TMEM_COLS_PER_GROUP);
    if (tid == 0 && s_timeout)
        atomicCAS(status + ST_CODE, 0, (int)SCOPE_ERR_TIMEOUT);
}

}  // namespace

bool kmeans_tc_supported(const KmArgs &a, size_t *smem_bytes)
{
    TcLayout L;
    if (!tc_layout(a, L))
        return false;
    for (int s = 0; s < a.nspaces; ++s)
        if (!a.sp[s].split)
            return false;
    size_t need = 1024 + (size_t)L.cent_bytes + GROUPS * XTILE_BYTES + ((L.un_floats + 3) & ~3) * sizeof(float) +
                  GROUPS * sizeof(GroupShared) + 64;
    if (smem_bytes)
        *smem_bytes = need;
    return need <= 220 * 1024;
}

void launch_kmeans_assign_tc(const KmArgs &a, int32_t *status, cudaStream_t st)
{
    size_t smem = 0;
    kmeans_tc_supported(a, &smem);
    // a block must own its SM (it allocates all 512 TMEM columns): ask for more than half the shared memory
    if (smem < 120 * 1024)
        smem = 120 * 1024;
    cudaFuncSetAttribute(kmeans_assign_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    const int ntiles = (a.N + TM - 1) / TM;
    const int tiles_per_block = 8;
    dim3 grid((ntiles + tiles_per_block - 1) / tiles_per_block, a.B * a.H);
    kmeans_assign_tc_kernel<<<grid, NT, smem, st>>>(a, tiles_per_block, status);
    count_launch();
}

}  // namespace scope
