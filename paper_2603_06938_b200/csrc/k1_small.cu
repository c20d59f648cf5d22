// K1 for a handful of tokens (the decode step: one token per sequence).  With at most a few
// hundred tokens the routing / projection stage moves almost nothing besides the expert matrices
// (Theorem 2: only the active experts are touched), so what counts is latency: no histogram, no
// per-expert lists in global memory, no tile table, two short kernels chained by programmatic
// dependent launch.
//   router_small_kernel   four warps per token: logits in fp32 with a fixed summation order, softmax
//                         over all E, the k largest kept with their softmax values, NOT renormalised
//                         (router softmax equation and the sentence after it); clears the token's
//                         row of the fp32 mixed streams.
//   project_small_kernel  one CTA per (expert, 16 rows of its matrix): finds the tokens routed to
//                         its expert by scanning the k * T routing entries, streams its 16 x F slice
//                         of W_e once, multiplies it with those tokens' features on the tensor cores
//                         (mma.sync m16n8k16, features split over the eight warps and added in a
//                         fixed order) and adds pi_{t,e} times the result into the token's row of
//                         the mixed streams (Theorem 1).  With k <= 2 a row receives at most two
//                         additions onto zero, so the sum does not depend on their order.
#include "internal.h"

namespace swimba {

namespace {
constexpr int SM_MAX_E = 16;        // experts the small router holds in registers
constexpr int SM_MAX_T = 256;       // tokens per call
constexpr int SM_ROWS = 16;         // rows of W_e per CTA (the M of m16n8k16)
constexpr int SM_WARPS = 8;
constexpr int SM_NT = 4;            // 8-token column tiles worked per pass
}  // namespace

__global__ void __launch_bounds__(256)
router_small_kernel(const __nv_bfloat16 *__restrict__ u, const __nv_bfloat16 *__restrict__ W_r, int Ttok,
                    int F, int E, int k, int32_t *__restrict__ idx, float *__restrict__ w,
                    float4 *__restrict__ bc_zero, int bc_vec_per_token)
{
    // two tokens per block, four warps per token (a quarter of the features each, partial logits
    // added in warp order)
    __shared__ float s_part[2][4][SM_MAX_E];
    grid_dep_wait();        // the previous step's update may still be reading the mixed streams
    grid_dep_launch();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int tl = warp >> 2, part = warp & 3;
    const int t = blockIdx.x * 2 + tl;
    const bool live = t < Ttok;
    float acc[SM_MAX_E];
#pragma unroll
    for (int e = 0; e < SM_MAX_E; ++e) acc[e] = 0.f;
    if (live) {
        for (int v = part * 32 + lane; v < bc_vec_per_token; v += 128)
            bc_zero[(int64_t)t * bc_vec_per_token + v] = make_float4(0.f, 0.f, 0.f, 0.f);
        const __nv_bfloat16 *urow = u + (int64_t)t * F;
        const int fq = F / 4;                               // (a multiple of 64)
#pragma unroll 2
        for (int f = part * fq + lane * 8; f < (part + 1) * fq; f += 256) {
            float uv[8];
            load8(urow + f, uv);
#pragma unroll
            for (int e = 0; e < SM_MAX_E; ++e) {
                if (e < E) {
                    float wv[8];
                    load8(W_r + (int64_t)e * F + f, wv);
#pragma unroll
                    for (int i = 0; i < 8; ++i) acc[e] = fmaf(wv[i], uv[i], acc[e]);
                }
            }
        }
    }
#pragma unroll
    for (int e = 0; e < SM_MAX_E; ++e) {
        const float v = warp_sum(acc[e]);
        if (lane == 0) s_part[tl][part][e] = v;
    }
    __syncthreads();
    if (!live || part != 0) return;
#pragma unroll
    for (int e = 0; e < SM_MAX_E; ++e)
        acc[e] = e < E ? ((s_part[tl][0][e] + s_part[tl][1][e]) + s_part[tl][2][e]) + s_part[tl][3][e] : -INFINITY;
    // softmax over all E, then k rounds of arg-max (ties to the lower index); every lane holds the
    // same values, lane 0 writes
    float m = acc[0];
#pragma unroll
    for (int e = 1; e < SM_MAX_E; ++e) m = fmaxf(m, acc[e]);
    float den = 0.f, pe[SM_MAX_E];
#pragma unroll
    for (int e = 0; e < SM_MAX_E; ++e) {
        pe[e] = e < E ? expf(acc[e] - m) : 0.f;
        den += pe[e];
    }
    const float inv = 1.f / den;
    unsigned taken = 0u;
    for (int j = 0; j < k; ++j) {
        int best = -1;
        float bv = -INFINITY;
#pragma unroll
        for (int e = 0; e < SM_MAX_E; ++e) {
            if (e < E && !((taken >> e) & 1u) && acc[e] > bv) { bv = acc[e]; best = e; }
        }
        taken |= 1u << best;
        float pb = 0.f;
#pragma unroll
        for (int e = 0; e < SM_MAX_E; ++e) if (e == best) pb = pe[e];
        if (lane == 0) {
            idx[(int64_t)t * k + j] = best;
            w[(int64_t)t * k + j] = pb * inv;
        }
    }
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                               uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__global__ void __launch_bounds__(256)
project_small_kernel(const __nv_bfloat16 *__restrict__ u, const __nv_bfloat16 *__restrict__ W_e,
                     const int32_t *__restrict__ idx, const float *__restrict__ w, int Ttok, int F, int S,
                     int E, int k, float *__restrict__ BC, int check, int *d_status)
{
    __shared__ int s_tok[SM_MAX_T];
    __shared__ float s_wgt[SM_MAX_T];
    __shared__ int s_count;
    __shared__ float s_red[SM_WARPS][SM_ROWS][8 * SM_NT];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int e = blockIdx.y, row0 = blockIdx.x * SM_ROWS;
    if (tid == 0) s_count = 0;
    __syncthreads();
    grid_dep_launch();
    // The matrix slice does not depend on the routing: when a warp's share fits in registers (F up to
    // 2048) it is fetched before the wait, under the router kernel's tail, and serves every pass.
    const int g = lane >> 2, tq = lane & 3;
    const int kslice = F / SM_WARPS;                       // features per warp (a multiple of 32)
    const __nv_bfloat16 *wrow0 = W_e + ((int64_t)e * S + row0 + g) * F + warp * kslice + tq * 8;
    const __nv_bfloat16 *wrow1 = wrow0 + (int64_t)8 * F;
    const bool resident = kslice <= 256;
    uint4 a0[8], a1[8];
    if (resident) {
#pragma unroll
        for (int st = 0; st < 8; ++st) {
            if (st * 32 < kslice) {
                a0[st] = *reinterpret_cast<const uint4 *>(wrow0 + st * 32);
                a1[st] = *reinterpret_cast<const uint4 *>(wrow1 + st * 32);
            }
        }
    }
    grid_dep_wait();        // routing entries come from the router kernel
    // tokens routed to this expert (a token picks an expert at most once); the order of the list
    // does not matter: every entry ends in its own output row
    for (int i = tid; i < Ttok * k; i += blockDim.x) {
        const int ei = idx[i];
        if (check && (ei < 0 || ei >= E)) atomicCAS(d_status, 0, SWIMBA_ERR_DEVICE_BOUNDS);
        if (ei == e) {
            const int slot = atomicAdd(&s_count, 1);
            if (slot < SM_MAX_T) {
                s_tok[slot] = i / k;
                s_wgt[slot] = w[i];
            }
        }
    }
    __syncthreads();
    const int count = min(s_count, SM_MAX_T);
    if (count == 0) return;
    for (int n0 = 0; n0 < count; n0 += 8 * SM_NT) {
        float acc[SM_NT][4];
#pragma unroll
        for (int q = 0; q < SM_NT; ++q)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[q][i] = 0.f;
        // 32 features per step, up to eight steps in flight: a lane holds 8 consecutive features of
        // its two matrix rows and of its token of every column tile; the first four feed one
        // m16n8k16, the last four the next (the contraction may run over the features in any
        // order, as long as both operands agree)
        for (int f0 = 0; f0 < kslice; f0 += 256) {
            const int nst = min(8, (kslice - f0) >> 5);
#pragma unroll
            for (int st = 0; st < 8; ++st) {
                if (!resident && st < nst) {
                    a0[st] = *reinterpret_cast<const uint4 *>(wrow0 + f0 + st * 32);
                    a1[st] = *reinterpret_cast<const uint4 *>(wrow1 + f0 + st * 32);
                }
            }
#pragma unroll
            for (int q = 0; q < SM_NT; ++q) {
                if (n0 + q * 8 < count) {                  // (warp-uniform)
                    const int n = n0 + q * 8 + g;
                    const __nv_bfloat16 *urow = n < count ? u + (int64_t)s_tok[n] * F + warp * kslice + tq * 8 + f0 : nullptr;
                    uint4 bv[8];
#pragma unroll
                    for (int st = 0; st < 8; ++st)
                        bv[st] = (urow && st < nst) ? *reinterpret_cast<const uint4 *>(urow + st * 32)
                                                    : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                    for (int st = 0; st < 8; ++st) {
                        if (st < nst) {
                            mma_bf16_16816(acc[q], a0[st].x, a1[st].x, a0[st].y, a1[st].y, bv[st].x, bv[st].y);
                            mma_bf16_16816(acc[q], a0[st].z, a1[st].z, a0[st].w, a1[st].w, bv[st].z, bv[st].w);
                        }
                    }
                }
            }
        }
        // partial sums of the eight feature slices -> shared memory, added in warp order
#pragma unroll
        for (int q = 0; q < SM_NT; ++q) {
            s_red[warp][g][q * 8 + 2 * tq] = acc[q][0];
            s_red[warp][g][q * 8 + 2 * tq + 1] = acc[q][1];
            s_red[warp][g + 8][q * 8 + 2 * tq] = acc[q][2];
            s_red[warp][g + 8][q * 8 + 2 * tq + 1] = acc[q][3];
        }
        __syncthreads();
        for (int o = tid; o < SM_ROWS * 8 * SM_NT; o += blockDim.x) {
            const int r = o / (8 * SM_NT), c = o % (8 * SM_NT);
            const int n = n0 + c;
            if (n < count) {
                float v = 0.f;
#pragma unroll
                for (int q = 0; q < SM_WARPS; ++q) v += s_red[q][r][c];
                atomicAdd(&BC[(int64_t)s_tok[n] * S + row0 + r], s_wgt[n] * v);
            }
        }
        __syncthreads();
    }
}

bool front_small_supported(int dtype, int64_t T, int F, int S, int E, int k)
{
    return dtype == SWIMBA_DTYPE_BF16 && T <= SM_MAX_T && E <= SM_MAX_E && k <= 2 && S % SM_ROWS == 0 &&
           F % (32 * SM_WARPS) == 0;
}

// idx [T,k], w [T,k] out; BC [T,S] fp32 out.
int launch_front_small(LaunchCtx &ctx, const void *u, const void *W_r, const void *W_e, int64_t T, int F,
                       int S, int E, int k, int32_t *idx, float *w, float *BC)
{
    if (T <= 0) return SWIMBA_OK;
    ctx.begin(STAGE_ROUTER);
    launch_kernel(router_small_kernel, dim3((unsigned)ceil_div64(T, 2)), dim3(256), 0, ctx.stream, true,
                  (const __nv_bfloat16 *)u, (const __nv_bfloat16 *)W_r, (int)T, F, E, k, idx, w, (float4 *)BC,
                  S / 4);
    ctx.end();
    ctx.begin(STAGE_PROJECT_SMALL);
    launch_kernel(project_small_kernel, dim3((unsigned)(S / SM_ROWS), (unsigned)E), dim3(256), 0, ctx.stream,
                  true, (const __nv_bfloat16 *)u, (const __nv_bfloat16 *)W_e, (const int32_t *)idx,
                  (const float *)w, (int)T, F, S, E, k, BC, ctx.check_indices ? 1 : 0, ctx.d_status);
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

}  // namespace swimba
