// K1 (SIMT part): router logits + softmax + top-k, and the plain projection/mix used by the
// fp32 path and by decode.  (Router softmax equation and top-k rule; Theorem 1, mixed streams.)
#include "internal.h"

namespace swimba {

// Router: a block handles chunks of `chunk` consecutive tokens, one warp TPW tokens at a time;
// the router matrix is staged in shared memory once per block (when it fits) so that every token
// costs one pass over its own features.
//
// Logit summation order (fixed, so results are reproducible run to run): lane l accumulates
// features f = 256*c + 8*l + i (c ascending, i = 0..7) with fused multiply-adds; the 32 partial
// sums of each (token, expert) are then combined by a halving butterfly over lane distances
// 16, 8, 4, 2, 1 in which each step also halves the number of values a lane still carries, so
// that afterwards every lane owns the complete logit of one (token, expert) pair (or of V/32
// adjacent experts when V = TPW*EP exceeds 32).  bf16 products are exact in fp32, so the only
// rounding is in the additions.  Softmax and top-k then run across the lanes of a token's group.
//
// Grouping by expert is done here as well: entry (t, j) goes to its expert's list,
// perm[e * cap + pos] = t*k + j.  Positions are handed out per chunk: a shared-memory histogram
// gives every entry its rank inside the chunk, one global atomic per (chunk, expert) on counts[e]
// (zeroed by the caller) reserves the chunk's range.  The order inside a list is arbitrary; every
// output row is computed independently of its position, so results do not depend on it.
constexpr int ROUTER_MAX_CHUNK = 512;

template <typename T, int EP, int TPW>
__global__ void __launch_bounds__(256)
router_topk_kernel(const T *__restrict__ u, const T *__restrict__ W_r, int64_t Ttok, int F, int E,
                   int k, int32_t *__restrict__ idx, float *__restrict__ w, int *__restrict__ counts,
                   int *__restrict__ perm, int64_t cap, int stage_w, int chunk,
                   uint4 *__restrict__ zero_out, int zero_vec_per_token, int router_blocks,
                   const ScalarsArgs scalars)
{
    grid_dep_launch();      // the projection kernel may set itself up under this kernel's tail
    if ((int)blockIdx.x >= router_blocks) {
        // extra blocks: SSD step sizes and tile log-decays, two (tile, head, sequence) units each
        __shared__ float s_tot[2][4];
        const int half = threadIdx.x >> 7;
        const int64_t unit = ((int64_t)blockIdx.x - router_blocks) * 2 + half;
        ssd_scalars_unit(scalars, unit, unit < scalars_units(scalars), threadIdx.x & 127, s_tot[half]);
        return;
    }
    constexpr int V = TPW * EP;                 // values per lane before the butterfly
    constexpr int R = V > 32 ? V / 32 : 1;      // values per lane after it (adjacent experts)
    constexpr int DUP = V >= 32 ? 1 : 32 / V;   // lanes holding the same value after it
    constexpr int GW = 32 / TPW;                // lanes per token group
    static_assert(V >= 2 && (V & (V - 1)) == 0 && R <= EP, "unsupported router shape");
    extern __shared__ __align__(16) unsigned char router_smem[];
    __shared__ int s_cnt[SWIMBA_MAX_EXPERTS], s_base[SWIMBA_MAX_EXPERTS];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
    int *s_ent = reinterpret_cast<int *>(router_smem);              // [chunk * k] expert | rank << 8
    const T *Wsrc = W_r;
    if (stage_w) {
        T *sW = reinterpret_cast<T *>(router_smem + (size_t)ROUTER_MAX_CHUNK * SWIMBA_MAX_TOPK * sizeof(int));
        const int nvec = (int)(((int64_t)E * F * sizeof(T)) >> 4);
        const uint4 *src = reinterpret_cast<const uint4 *>(W_r);
        uint4 *dst = reinterpret_cast<uint4 *>(sW);
        for (int i = threadIdx.x; i < nvec; i += blockDim.x) dst[i] = src[i];
        Wsrc = sW;
    }
    // after the butterfly this lane owns experts e0 .. e0+R-1 of token q_own of the pass
    const int q_own = lane / GW;
    const int e0 = ((lane % GW) / DUP) * R;
    const int64_t nchunks = ceil_div64(Ttok, chunk);
    for (int64_t c = blockIdx.x; c < nchunks; c += router_blocks) {
        const int64_t tbeg = c * chunk;
        const int64_t tend = (tbeg + chunk < Ttok) ? tbeg + chunk : Ttok;
        if (threadIdx.x < SWIMBA_MAX_EXPERTS) s_cnt[threadIdx.x] = 0;
        if (zero_out) {
            // the mixed-stream rows of this chunk start at zero: the projection adds its slots
            const int64_t nz = (tend - tbeg) * zero_vec_per_token;
            uint4 *z = zero_out + tbeg * zero_vec_per_token;
            for (int64_t i = threadIdx.x; i < nz; i += blockDim.x) z[i] = make_uint4(0u, 0u, 0u, 0u);
        }
        __syncthreads();
        // The feature loads run one step ahead of the arithmetic, across passes too: `raw` always
        // holds the next 8-feature slice of the next TPW tokens.
        typename Raw8<T>::type raw[TPW];
        auto prefetch = [&](int64_t tt0, int ff) {
#pragma unroll
            for (int q = 0; q < TPW; ++q) {
                const int64_t t = (tt0 + q < tend) ? tt0 + q : tt0;
                load_raw8(u + t * F + ff, raw[q]);
            }
        };
        if (tbeg + warp * TPW < tend && lane * 8 < F) prefetch(tbeg + warp * TPW, lane * 8);
        for (int64_t t0 = tbeg + warp * TPW; t0 < tend; t0 += nwarp * TPW) {
            float g[V];                                  // g[q * EP + e]
#pragma unroll
            for (int i = 0; i < V; ++i) g[i] = 0.f;
#pragma unroll 1
            for (int f = lane * 8; f < F; f += 256) {
                float uv[TPW][8];
#pragma unroll
                for (int q = 0; q < TPW; ++q) unpack8(raw[q], uv[q]);
                if (f + 256 < F) prefetch(t0, f + 256);
                else if (t0 + nwarp * TPW < tend) prefetch(t0 + nwarp * TPW, lane * 8);
#pragma unroll
                for (int e = 0; e < EP; ++e) {
                    if (e < E) {
                        float wv[8];
                        load8(Wsrc + (int64_t)e * F + f, wv);
#pragma unroll
                        for (int q = 0; q < TPW; ++q)
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                g[q * EP + e] = fmaf(wv[i], uv[q][i], g[q * EP + e]);
                    }
                }
            }
            // halving butterfly: V values on 32 lanes -> R values on this lane
            {
                int n = V;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    if (n > R) {
                        n >>= 1;
                        const bool up = (lane & o) != 0;
#pragma unroll
                        for (int i = 0; i < V / 2; ++i) {
                            if (i < n) {
                                const float send = up ? g[i] : g[i + n];
                                const float keep = up ? g[i + n] : g[i];
                                g[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
                            }
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < R; ++i) g[i] += __shfl_xor_sync(0xffffffffu, g[i], o);
                    }
                }
            }
            // softmax over ALL experts of the token (padding experts count as -inf)
            float gv[R], pv[R];
            float m = -INFINITY;
#pragma unroll
            for (int i = 0; i < R; ++i) {
                gv[i] = (e0 + i < E) ? g[i] : -INFINITY;
                m = fmaxf(m, gv[i]);
            }
#pragma unroll
            for (int o = GW / 2; o >= DUP; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            float z = 0.f;
#pragma unroll
            for (int i = 0; i < R; ++i) {
                pv[i] = expf(gv[i] - m);
                z += pv[i];
            }
#pragma unroll
            for (int o = GW / 2; o >= DUP; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
            // k rounds of "largest remaining logit, lowest index on ties"; weights are NOT
            // renormalised
            const int64_t t = t0 + q_own;
            for (int j = 0; j < k; ++j) {
                float bg = gv[0], bp = pv[0];
                int be = e0;
#pragma unroll
                for (int i = 1; i < R; ++i)
                    if (gv[i] > bg) { bg = gv[i]; bp = pv[i]; be = e0 + i; }
#pragma unroll
                for (int o = GW / 2; o >= DUP; o >>= 1) {
                    const float og = __shfl_xor_sync(0xffffffffu, bg, o);
                    const float op = __shfl_xor_sync(0xffffffffu, bp, o);
                    const int oe = __shfl_xor_sync(0xffffffffu, be, o);
                    if (og > bg || (og == bg && oe < be)) { bg = og; bp = op; be = oe; }
                }
#pragma unroll
                for (int i = 0; i < R; ++i) if (e0 + i == be) gv[i] = -INFINITY;
                if (lane % GW == 0 && t < tend) {
                    idx[t * k + j] = be;
                    w[t * k + j] = bp / z;
                    if (counts) {
                        const int rank = atomicAdd(&s_cnt[be], 1);
                        s_ent[(int)(t - tbeg) * k + j] = be | (rank << 8);
                    }
                }
            }
        }
        if (counts) {
            __syncthreads();
            if (threadIdx.x < E) s_base[threadIdx.x] = atomicAdd(&counts[threadIdx.x], s_cnt[threadIdx.x]);
            __syncthreads();
            const int n_ent = (int)(tend - tbeg) * k;
            for (int i = threadIdx.x; i < n_ent; i += blockDim.x) {
                const int ent = s_ent[i], e = ent & 255;
                perm[(int64_t)e * cap + s_base[e] + (ent >> 8)] = (int)(tbeg * k + i);
            }
        }
        __syncthreads();
    }
}

// One expert: the softmax is identically 1 and every token is routed to expert 0.
__global__ void __launch_bounds__(256)
router_single_expert_kernel(int64_t Ttok, int32_t *__restrict__ idx, float *__restrict__ w,
                            int *__restrict__ counts, int *__restrict__ perm)
{
    grid_dep_launch();
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < Ttok;
         t += (int64_t)gridDim.x * blockDim.x) {
        idx[t] = 0;
        w[t] = 1.f;
        if (counts) perm[t] = (int)t;
    }
    if (counts && blockIdx.x == 0 && threadIdx.x == 0) counts[0] = (int)Ttok;
}

template <typename T>
static int launch_router_t(LaunchCtx &ctx, const T *u, const T *W_r, int64_t Ttok, int F, int E,
                           int k, int32_t *idx, float *w, int *counts, int *perm, int64_t cap,
                           int sm_count, void *zero_out, int zero_bytes_per_token,
                           const ScalarsArgs &scalars)
{
    const int warps = 8;
    if (E == 1) {
        int64_t blocks = ceil_div64(Ttok, 256);
        if (blocks > (int64_t)sm_count * 8) blocks = (int64_t)sm_count * 8;
        ctx.begin(STAGE_ROUTER);
        router_single_expert_kernel<<<(unsigned)blocks, 256, 0, ctx.stream>>>(Ttok, idx, w, counts, perm);
        ctx.end();
        return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
    }
    const size_t w_bytes = (size_t)E * F * sizeof(T);
    const int stage_w = (w_bytes <= 64 * 1024 && (w_bytes & 15) == 0) ? 1 : 0;
    const size_t smem = (size_t)ROUTER_MAX_CHUNK * SWIMBA_MAX_TOPK * sizeof(int) + (stage_w ? w_bytes : 0);
    // chunk: enough chunks to give every SM four blocks, between 32 and ROUTER_MAX_CHUNK tokens
    int chunk = (int)(Ttok / (4 * (int64_t)sm_count));
    chunk = (chunk + 31) / 32 * 32;
    if (chunk < 32) chunk = 32;
    if (chunk > ROUTER_MAX_CHUNK) chunk = ROUTER_MAX_CHUNK;
    ctx.begin(STAGE_ROUTER);
#define SWIMBA_ROUTER_CASE(EPV, TPWV)                                                          \
    do {                                                                                       \
        auto kern = router_topk_kernel<T, EPV, TPWV>;                                          \
        if (smem > 32 * 1024 &&  /* static shared memory counts toward the 48 KB default */    \
            cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,            \
                                 (int)smem) != cudaSuccess)                                    \
            return SWIMBA_ERR_CUDA;                                                            \
        int64_t blocks = ceil_div64(Ttok, chunk);                                              \
        const int64_t cap_blocks = (int64_t)sm_count * (smem > 40 * 1024 ? 2 : 4);             \
        if (blocks > cap_blocks) blocks = cap_blocks;                                          \
        const int64_t extra = (scalars_units(scalars) + 1) / 2;                                \
        kern<<<(unsigned)(blocks + extra), warps * 32, smem, ctx.stream>>>(                    \
            u, W_r, Ttok, F, E, k, idx, w, counts, perm, cap, stage_w, chunk, (uint4 *)zero_out, \
            zero_bytes_per_token / 16, (int)blocks, scalars);                                  \
    } while (0)
    if (E <= 2) SWIMBA_ROUTER_CASE(2, 8);
    else if (E <= 4) SWIMBA_ROUTER_CASE(4, 8);
    else if (E <= 8) SWIMBA_ROUTER_CASE(8, 4);
    else if (E <= 16) SWIMBA_ROUTER_CASE(16, 2);
    else if (E <= 32) SWIMBA_ROUTER_CASE(32, 1);
    else SWIMBA_ROUTER_CASE(64, 1);
#undef SWIMBA_ROUTER_CASE
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

int launch_router(LaunchCtx &ctx, int dtype, const void *u, const void *W_r, int64_t T, int F,
                  int E, int k, int32_t *idx, float *w, int *counts, int *perm, int64_t cap,
                  int sm_count, void *zero_out, int zero_bytes_per_token, const ScalarsArgs &scalars)
{
    if (T <= 0) return SWIMBA_OK;
    if (dtype == SWIMBA_DTYPE_FP32)
        return launch_router_t<float>(ctx, (const float *)u, (const float *)W_r, T, F, E, k, idx, w,
                                      counts, perm, cap, sm_count, zero_out, zero_bytes_per_token, scalars);
    return launch_router_t<__nv_bfloat16>(ctx, (const __nv_bfloat16 *)u,
                                          (const __nv_bfloat16 *)W_r, T, F, E, k, idx, w, counts,
                                          perm, cap, sm_count, zero_out, zero_bytes_per_token, scalars);
}

// One warp per (token, block of RW stream rows): BC[t, r] = sum_j w_j <W_e[e_j, r, :], u_t>.
// Only the k selected experts are touched.
template <typename T, typename TO, int RW>
__global__ void __launch_bounds__(256)
project_mix_simt_kernel(const T *__restrict__ u, const T *__restrict__ W_e,
                        const int32_t *__restrict__ idx, const float *__restrict__ w, int64_t Ttok,
                        int F, int S, int k, TO *__restrict__ BC)
{
    const int lane = threadIdx.x & 31;
    const int nblk = ceil_div(S, RW);
    const int64_t wid = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (wid >= Ttok * nblk) return;
    const int64_t t = wid / nblk;
    const int r0 = (int)(wid % nblk) * RW;
    int ej[SWIMBA_MAX_TOPK];
    float wj[SWIMBA_MAX_TOPK];
#pragma unroll
    for (int j = 0; j < SWIMBA_MAX_TOPK; ++j) {
        ej[j] = (j < k) ? idx[t * k + j] : 0;
        wj[j] = (j < k) ? w[t * k + j] : 0.f;
    }
    float acc[RW];
#pragma unroll
    for (int r = 0; r < RW; ++r) acc[r] = 0.f;
    const T *urow = u + t * F;
    for (int f = lane * 8; f < F; f += 256) {
        float uv[8];
        load8(urow + f, uv);
#pragma unroll
        for (int j = 0; j < SWIMBA_MAX_TOPK; ++j) {
            if (j < k) {
                float us[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) us[i] = wj[j] * uv[i];
                const T *wbase = W_e + ((int64_t)ej[j] * S + r0) * F + f;
#pragma unroll
                for (int r = 0; r < RW; ++r) {
                    if (r0 + r < S) {
                        float wv[8];
                        load8(wbase + (int64_t)r * F, wv);
#pragma unroll
                        for (int i = 0; i < 8; ++i) acc[r] = fmaf(wv[i], us[i], acc[r]);
                    }
                }
            }
        }
    }
    float mine = 0.f;
#pragma unroll
    for (int r = 0; r < RW; ++r) {
        const float s = warp_sum(acc[r]);
        if (lane == r) mine = s;
    }
    if (lane < RW && r0 + lane < S) BC[t * S + r0 + lane] = from_f32<TO>(mine);
}

template <typename T, typename TO>
static int launch_pm(LaunchCtx &ctx, const void *u, const void *W_e, const int32_t *idx,
                     const float *w, int64_t T_, int F, int S, int k, void *BC)
{
    constexpr int RW = 16;
    const int warps = 8;
    const int64_t nw = T_ * ceil_div(S, RW);
    dim3 grid((unsigned)ceil_div64(nw, warps)), block(warps * 32);
    ctx.begin(STAGE_PROJECT_SIMT);
    project_mix_simt_kernel<T, TO, RW><<<grid, block, 0, ctx.stream>>>(
        (const T *)u, (const T *)W_e, idx, w, T_, F, S, k, (TO *)BC);
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

int launch_project_mix_simt(LaunchCtx &ctx, int dtype, const void *u, const void *W_e,
                            const int32_t *idx, const float *w, int64_t T, int F, int S, int E,
                            int k, void *BC, bool bc_fp32)
{
    (void)E;
    if (T <= 0) return SWIMBA_OK;
    if (dtype == SWIMBA_DTYPE_FP32) return launch_pm<float, float>(ctx, u, W_e, idx, w, T, F, S, k, BC);
    if (bc_fp32) return launch_pm<__nv_bfloat16, float>(ctx, u, W_e, idx, w, T, F, S, k, BC);
    return launch_pm<__nv_bfloat16, __nv_bfloat16>(ctx, u, W_e, idx, w, T, F, S, k, BC);
}

}  // namespace swimba
