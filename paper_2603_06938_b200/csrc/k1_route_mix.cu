// K1 (SIMT part): router logits + softmax + top-k, and the plain projection/mix used by the
// fp32 path and by decode.  (Router softmax equation and top-k rule; Theorem 1, mixed streams.)
#include "internal.h"

namespace swimba {

// One warp per token.  Logit summation order (fixed, so results are reproducible run to run):
// lane l accumulates features f = 256*c + 8*l + i (c ascending, i = 0..7) with fused
// multiply-adds, then the 32 partial sums are combined by an xor butterfly (16,8,4,2,1).
// bf16 products are exact in fp32, so the only rounding is in the additions.
template <typename T, int EP>
__global__ void __launch_bounds__(256)
router_topk_kernel(const T *__restrict__ u, const T *__restrict__ W_r, int64_t Ttok, int F, int E,
                   int k, int32_t *__restrict__ idx, float *__restrict__ w, int *__restrict__ counts)
{
    const int lane = threadIdx.x & 31;
    const int64_t t = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= Ttok) return;
    float g[EP];
#pragma unroll
    for (int e = 0; e < EP; ++e) g[e] = 0.f;
    const T *urow = u + t * F;
    for (int f = lane * 8; f < F; f += 256) {
        float uv[8];
        load8(urow + f, uv);
#pragma unroll
        for (int e = 0; e < EP; ++e) {
            if (e < E) {
                float wv[8];
                load8(W_r + (int64_t)e * F + f, wv);
#pragma unroll
                for (int i = 0; i < 8; ++i) g[e] = fmaf(wv[i], uv[i], g[e]);
            }
        }
    }
#pragma unroll
    for (int e = 0; e < EP; ++e) g[e] = warp_sum(g[e]);
    // softmax over ALL experts, ascending expert order
    float m = g[0];
#pragma unroll
    for (int e = 1; e < EP; ++e) if (e < E) m = fmaxf(m, g[e]);
    float z = 0.f;
    float p[EP];
#pragma unroll
    for (int e = 0; e < EP; ++e) {
        p[e] = (e < E) ? expf(g[e] - m) : 0.f;
        z += p[e];
    }
    // k rounds of "largest remaining logit, lowest index on ties"; weights are NOT renormalised
    unsigned long long taken = 0ull;
    for (int j = 0; j < k; ++j) {
        int best = -1;
        float bestg = 0.f, bestp = 0.f;
#pragma unroll
        for (int e = 0; e < EP; ++e) {
            if (e < E && !((taken >> e) & 1ull) && (best < 0 || g[e] > bestg)) {
                best = e; bestg = g[e]; bestp = p[e];
            }
        }
        taken |= 1ull << best;
        if (lane == 0) {
            idx[t * k + j] = best;
            w[t * k + j] = bestp / z;
            if (counts) atomicAdd(&counts[best], 1);
        }
    }
}

template <typename T>
static int launch_router_t(LaunchCtx &ctx, const T *u, const T *W_r, int64_t Ttok, int F, int E,
                           int k, int32_t *idx, float *w, int *counts)
{
    const int warps = 8;
    dim3 grid((unsigned)ceil_div64(Ttok, warps)), block(warps * 32);
    ctx.begin(STAGE_ROUTER);
#define SWIMBA_ROUTER_CASE(EPV)                                                              \
    router_topk_kernel<T, EPV><<<grid, block, 0, ctx.stream>>>(u, W_r, Ttok, F, E, k, idx, w, counts)
    if (E <= 1) SWIMBA_ROUTER_CASE(1);
    else if (E <= 2) SWIMBA_ROUTER_CASE(2);
    else if (E <= 4) SWIMBA_ROUTER_CASE(4);
    else if (E <= 8) SWIMBA_ROUTER_CASE(8);
    else if (E <= 16) SWIMBA_ROUTER_CASE(16);
    else if (E <= 32) SWIMBA_ROUTER_CASE(32);
    else SWIMBA_ROUTER_CASE(64);
#undef SWIMBA_ROUTER_CASE
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

int launch_router(LaunchCtx &ctx, int dtype, const void *u, const void *W_r, int64_t T, int F,
                  int E, int k, int32_t *idx, float *w, int *counts)
{
    if (T <= 0) return SWIMBA_OK;
    if (dtype == SWIMBA_DTYPE_FP32)
        return launch_router_t<float>(ctx, (const float *)u, (const float *)W_r, T, F, E, k, idx, w, counts);
    return launch_router_t<__nv_bfloat16>(ctx, (const __nv_bfloat16 *)u,
                                          (const __nv_bfloat16 *)W_r, T, F, E, k, idx, w, counts);
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
