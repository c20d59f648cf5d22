// Gradients of  sum(dy * y)  with respect to the router matrix W_r and the expert matrices W_e
// (Section "Training": the router and the expert parameters are what the conversion trains; the
// rest of the layer is frozen), by reverse-mode differentiation of the forward's steps:
//   recurrence (Theorem 1)   lambda_t = a_{t+1} lambda_{t+1} + dy_t Ctilde_t^T
//                            dCtilde_t[n] = sum_{h,p} dy_t[h,p] h_t[h,p,n]
//                            dBtilde_t[n] = Delta_t sum_{h,p} x_t[h,p] lambda_t[h,p,n]
//   mix (parameter-space mixing)   dpi_{t,j} = <dBC_t, W_e[e_j] u_t>,  dW_e[e_j] += pi_{t,e_j} dBC_t u_t^T
//   softmax (router equation)      dg_{t,i} = pi_{t,i} ([i in K_t] dpi_{t,i} - sum_{j in K_t} pi_{t,j} dpi_{t,j})
//   logits                         dW_r += dg_t u_t^T
// The active sets are constants; the kept weights are softmax values over all E (no
// renormalisation) and are differentiated as such.  Plain CUDA-core kernels, fp32 accumulation.
#include "internal.h"
#include "tc05.cuh"

namespace swimba {

namespace {
constexpr int ADJ_TS = 16;   // tokens staged in shared memory per round
constexpr int ADJ_PT = 16;   // channels per thread

// One pass of the recurrence for one (sequence, head), state in registers: thread (n, ps) owns
// state entries [p = ps*ADJ_PT + i][n].  Per token:  st = a st + inj_p V_n,  out_n = sum_p rd_p st.
//   forward in time (REVERSE = false): inj = Delta x, rd = dy, V = Btilde, a = a_t: out = dCtilde
//   backward in time (REVERSE = true): inj = dy, rd = Delta x, V = Ctilde, a = a_{t+1}: out = dBtilde
// out is added to dBC[t, column block of V's partner] with atomics (heads of a group share columns).
template <typename T, bool REVERSE>
__global__ void __launch_bounds__(1024)
ssd_adjoint_kernel(const T *__restrict__ x, const T *__restrict__ dy, const T *__restrict__ BC,
                   const float *__restrict__ dt, const float *__restrict__ A, const float *__restrict__ dt_bias,
                   const float *__restrict__ h0, int L, int H, int P, int N, int G, int PS,
                   float *__restrict__ dBC)
{
    extern __shared__ float smem[];
    const int Ppad = PS * ADJ_PT;
    float *sV = smem;                       // [TS][N]
    float *sInj = sV + ADJ_TS * N;          // [TS][Ppad]
    float *sRd = sInj + ADJ_TS * Ppad;      // [TS][Ppad]
    float *sOut = sRd + ADJ_TS * Ppad;      // [TS][N]
    float *sA = sOut + ADJ_TS * N;          // [TS]

    const int b = blockIdx.x / H, h = blockIdx.x % H;
    const int g = h / (H / G);
    const int S = 2 * G * N;
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int n = tid / PS, ps = tid % PS;
    const float Ah = A[h], bias = dt_bias[h];
    const unsigned amask = __activemask();
    const int vcol = REVERSE ? (G + g) * N : g * N;          // columns of V in BC
    const int ocol = REVERSE ? g * N : (G + g) * N;          // columns of dBC that receive out

    float st[ADJ_PT];
#pragma unroll
    for (int i = 0; i < ADJ_PT; ++i) {
        const int p = ps * ADJ_PT + i;
        st[i] = (!REVERSE && h0 && p < P) ? h0[(((int64_t)b * H + h) * P + p) * N + n] : 0.f;
    }
    float a_carry = 0.f;        // REVERSE: decay of the token after the current one

    const int nrounds = (L + ADJ_TS - 1) / ADJ_TS;
    for (int rd = 0; rd < nrounds; ++rd) {
        const int t0 = (REVERSE ? nrounds - 1 - rd : rd) * ADJ_TS;
        const int nt = min(ADJ_TS, L - t0);
        for (int i = tid; i < nt * N; i += nthr) {
            const int tt = i / N, nn = i % N;
            sV[tt * N + nn] = to_f32<T>(BC[((int64_t)b * L + t0 + tt) * S + vcol + nn]);
        }
        for (int i = tid; i < nt; i += nthr) {
            const float raw = dt ? dt[((int64_t)b * L + t0 + i) * H + h] : 0.f;
            sA[i] = softplus_f(raw + bias);          // Delta for now
        }
        __syncthreads();
        for (int i = tid; i < nt * Ppad; i += nthr) {
            const int tt = i / Ppad, pp = i % Ppad;
            float xv = 0.f, dv = 0.f;
            if (pp < P) {
                const int64_t at = (((int64_t)b * L + t0 + tt) * H + h) * P + pp;
                xv = to_f32<T>(x[at]) * sA[tt];
                dv = to_f32<T>(dy[at]);
            }
            sInj[tt * Ppad + pp] = REVERSE ? dv : xv;
            sRd[tt * Ppad + pp] = REVERSE ? xv : dv;
        }
        __syncthreads();
        for (int i = tid; i < nt; i += nthr) sA[i] = expf(sA[i] * Ah);
        __syncthreads();
        for (int q = 0; q < nt; ++q) {
            const int tt = REVERSE ? nt - 1 - q : q;
            const float a = REVERSE ? a_carry : sA[tt];
            const float v = sV[tt * N + n];
            const float4 *inj4 = reinterpret_cast<const float4 *>(sInj + tt * Ppad + ps * ADJ_PT);
            const float4 *rd4 = reinterpret_cast<const float4 *>(sRd + tt * Ppad + ps * ADJ_PT);
            float acc = 0.f;
#pragma unroll
            for (int c = 0; c < ADJ_PT / 4; ++c) {
                const float4 iv = inj4[c], rv = rd4[c];
                st[4 * c + 0] = fmaf(a, st[4 * c + 0], iv.x * v);
                st[4 * c + 1] = fmaf(a, st[4 * c + 1], iv.y * v);
                st[4 * c + 2] = fmaf(a, st[4 * c + 2], iv.z * v);
                st[4 * c + 3] = fmaf(a, st[4 * c + 3], iv.w * v);
                acc = fmaf(rv.x, st[4 * c + 0], acc);
                acc = fmaf(rv.y, st[4 * c + 1], acc);
                acc = fmaf(rv.z, st[4 * c + 2], acc);
                acc = fmaf(rv.w, st[4 * c + 3], acc);
            }
            for (int o = PS >> 1; o > 0; o >>= 1) acc += __shfl_xor_sync(amask, acc, o);
            if (ps == 0) sOut[tt * N + n] = acc;
            if (REVERSE) a_carry = sA[tt];
        }
        __syncthreads();
        for (int i = tid; i < nt * N; i += nthr) {
            const int tt = i / N, nn = i % N;
            atomicAdd(dBC + ((int64_t)b * L + t0 + tt) * S + ocol + nn, sOut[tt * N + nn]);
        }
        __syncthreads();
    }
}

// Softmax over all E of the router logits, one warp per token: pi[T,E].
template <typename T>
__global__ void __launch_bounds__(256)
router_softmax_kernel(const T *__restrict__ u, const T *__restrict__ W_r, int64_t Tn, int F, int E,
                      float *__restrict__ pi)
{
    const int lane = threadIdx.x & 31;
    const int64_t t = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= Tn) return;
    float g[SWIMBA_MAX_EXPERTS];
    float m = -INFINITY;
    for (int e = 0; e < E; ++e) {
        float acc = 0.f;
        for (int f = lane; f < F; f += 32) acc = fmaf(to_f32<T>(W_r[(int64_t)e * F + f]), to_f32<T>(u[t * F + f]), acc);
        acc = warp_sum(acc);
        g[e] = acc;
        m = fmaxf(m, acc);
    }
    float z = 0.f;
    for (int e = 0; e < E; ++e) { g[e] = expf(g[e] - m); z += g[e]; }
    const float inv = 1.f / z;
    for (int e = lane; e < E; e += 32) pi[t * E + e] = g[e] * inv;
}

// dpi and dg, one warp per token.  slots[t*k + j, :] = W_e[idx[t,j]] u_t (unscaled).
template <typename T>
__global__ void __launch_bounds__(256)
dpi_dg_kernel(const float *__restrict__ dBC, const T *__restrict__ slots, const int32_t *__restrict__ idx,
              const float *__restrict__ w, const float *__restrict__ pi, int64_t Tn, int S, int E, int k,
              float *__restrict__ dg)
{
    const int lane = threadIdx.x & 31;
    const int64_t t = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= Tn) return;
    float inner = 0.f;
    float dpi[SWIMBA_MAX_TOPK];
    for (int j = 0; j < k; ++j) {
        float acc = 0.f;
        const T *row = slots + (t * k + j) * (int64_t)S;
        for (int s = lane; s < S; s += 32) acc = fmaf(dBC[t * S + s], to_f32<T>(row[s]), acc);
        acc = warp_sum(acc);
        dpi[j] = acc;
        inner = fmaf(w[t * k + j], acc, inner);
    }
    for (int e = lane; e < E; e += 32) {
        float v = -pi[t * E + e] * inner;
        for (int j = 0; j < k; ++j)
            if (idx[t * k + j] == e) v = fmaf(w[t * k + j], dpi[j], v);
        dg[t * E + e] = v;
    }
}

// dW_r[e,f] += sum_t dg[t,e] u[t,f] over the block's run of tokens; thread = one feature f,
// eight experts at a time.
constexpr int DWR_TOK = 512;
template <typename T>
__global__ void __launch_bounds__(256)
dw_router_kernel(const T *__restrict__ u, const float *__restrict__ dg, int64_t Tn, int F, int E,
                 float *__restrict__ dW_r)
{
    __shared__ float sdg[64][8];
    const int f = blockIdx.y * blockDim.x + threadIdx.x;
    const int64_t t0 = (int64_t)blockIdx.x * DWR_TOK;
    const int nt = (int)min((int64_t)DWR_TOK, Tn - t0);
    for (int e0 = 0; e0 < E; e0 += 8) {
        float acc[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) acc[q] = 0.f;
        for (int c0 = 0; c0 < nt; c0 += 64) {
            const int nc = min(64, nt - c0);
            __syncthreads();
            for (int i = threadIdx.x; i < nc * 8; i += blockDim.x) {
                const int tt = i >> 3, q = i & 7;
                sdg[tt][q] = e0 + q < E ? dg[(t0 + c0 + tt) * E + e0 + q] : 0.f;
            }
            __syncthreads();
            if (f < F) {
                for (int tt = 0; tt < nc; ++tt) {
                    const float uv = to_f32<T>(u[(t0 + c0 + tt) * F + f]);
#pragma unroll
                    for (int q = 0; q < 8; ++q) acc[q] = fmaf(sdg[tt][q], uv, acc[q]);
                }
            }
        }
        if (f < F) {
#pragma unroll
            for (int q = 0; q < 8; ++q)
                if (e0 + q < E) atomicAdd(dW_r + (int64_t)(e0 + q) * F + f, acc[q]);
        }
    }
}

// dW_e[e][s,f] += sum over the (token, slot) entries routed to e inside the block's run of tokens
// of  w dBC[t,s] u[t,f]:  a 64 x 64 tile of one expert's matrix per block, 4 x 4 per thread, the
// entries taken 16 at a time through shared memory.
constexpr int DWE_TOK = 2048;    // tokens per run (the run's entries of one expert are listed in shared memory)
template <typename T>
__global__ void __launch_bounds__(256)
dw_expert_kernel(const T *__restrict__ u, const float *__restrict__ dBC, const int32_t *__restrict__ idx,
                 const float *__restrict__ w, int64_t Tn, int F, int S, int E, int k, int nruns,
                 float *__restrict__ dW_e)
{
    __shared__ int list[DWE_TOK];
    __shared__ int list_n;
    __shared__ __align__(16) float sA[16][64];
    __shared__ __align__(16) float sB[16][64];
    const int e = blockIdx.z / nruns, run = blockIdx.z % nruns;
    const int s0 = blockIdx.x * 64, f0 = blockIdx.y * 64;
    const int64_t t0 = (int64_t)run * DWE_TOK;
    const int nt = (int)min((int64_t)DWE_TOK, Tn - t0);
    const int tid = threadIdx.x;
    if (tid == 0) list_n = 0;
    __syncthreads();
    // entries r = t*k + j of this run routed to e (at most one per token: a token's experts are distinct)
    for (int i = tid; i < nt * k; i += blockDim.x) {
        const int64_t r = t0 * k + i;
        if (idx[r] == e) list[atomicAdd(&list_n, 1)] = i;
    }
    __syncthreads();
    const int cnt = list_n;
    if (cnt == 0) return;
    const int ty = tid >> 4, tx = tid & 15;          // rows s0 + 4 ty .., columns f0 + 4 tx ..
    float acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[a][c] = 0.f;
    for (int c0 = 0; c0 < cnt; c0 += 16) {
        const int nc = min(16, cnt - c0);
        __syncthreads();
        for (int i = tid; i < 16 * 64; i += blockDim.x) {
            const int kk = i >> 6, col = i & 63;
            float av = 0.f, bv = 0.f;
            if (kk < nc) {
                const int64_t r = t0 * k + list[c0 + kk];
                const int64_t t = r / k;
                if (s0 + col < S) av = w[r] * dBC[t * S + s0 + col];
                if (f0 + col < F) bv = to_f32<T>(u[t * F + f0 + col]);
            }
            sA[kk][col] = av;
            sB[kk][col] = bv;
        }
        __syncthreads();
#pragma unroll 4
        for (int kk = 0; kk < 16; ++kk) {
            const float4 a4 = *reinterpret_cast<const float4 *>(&sA[kk][4 * ty]);
            const float4 b4 = *reinterpret_cast<const float4 *>(&sB[kk][4 * tx]);
            const float av[4] = {a4.x, a4.y, a4.z, a4.w}, bv[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int c = 0; c < 4; ++c) acc[a][c] = fmaf(av[a], bv[c], acc[a][c]);
        }
    }
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int s = s0 + 4 * ty + a, f = f0 + 4 * tx + c;
            if (s < S && f < F) atomicAdd(dW_e + ((int64_t)e * S + s) * F + f, acc[a][c]);
        }
}

__global__ void fill_kernel(float *p, int64_t n, float v)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) p[i] = v;
}

int adjoint_ps(int P)
{
    int ps = 1;
    while (ps * ADJ_PT < P) ps <<= 1;
    return ps;
}

template <typename T>
int launch_adjoint_t(LaunchCtx &ctx, const void *x, const void *dy, const void *BC, const float *dt, const float *A,
                     const float *dt_bias, const float *h0, int B, int L, int H, int P, int N, int G, float *dBC)
{
    const int PS = adjoint_ps(P);
    const int Ppad = PS * ADJ_PT;
    const size_t smem = sizeof(float) * (size_t)(2 * ADJ_TS * N + 2 * ADJ_TS * Ppad + ADJ_TS);
    auto kf = ssd_adjoint_kernel<T, false>;
    auto kr = ssd_adjoint_kernel<T, true>;
    if (smem > 48 * 1024 &&
        (!ensure_dynamic_smem((const void *)kf, smem) || !ensure_dynamic_smem((const void *)kr, smem)))
        return SWIMBA_ERR_CUDA;
    ctx.begin(STAGE_SSD_ADJOINT);
    kf<<<B * H, N * PS, smem, ctx.stream>>>((const T *)x, (const T *)dy, (const T *)BC, dt, A, dt_bias, h0, L, H, P, N,
                                           G, PS, dBC);
    ctx.end();
    ctx.begin(STAGE_SSD_ADJOINT);
    kr<<<B * H, N * PS, smem, ctx.stream>>>((const T *)x, (const T *)dy, (const T *)BC, dt, A, dt_bias, h0, L, H, P, N,
                                           G, PS, dBC);
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

template <typename T>
int launch_weight_grads_t(LaunchCtx &ctx, const void *u, const void *W_r, const void *slots, const int32_t *idx,
                          const float *w, const float *dBC, int64_t Tn, int F, int S, int E, int k, float *pi,
                          float *dg, float *dW_r, float *dW_e)
{
    const unsigned tok_blocks = (unsigned)ceil_div64(Tn, 8);
    ctx.begin(STAGE_ROUTER_SOFTMAX);
    router_softmax_kernel<T><<<tok_blocks, 256, 0, ctx.stream>>>((const T *)u, (const T *)W_r, Tn, F, E, pi);
    ctx.end();
    ctx.begin(STAGE_DPI_DG);
    dpi_dg_kernel<T><<<tok_blocks, 256, 0, ctx.stream>>>(dBC, (const T *)slots, idx, w, pi, Tn, S, E, k, dg);
    ctx.end();
    if (dW_r) {
        ctx.begin(STAGE_DW_ROUTER);
        dw_router_kernel<T><<<dim3((unsigned)ceil_div64(Tn, DWR_TOK), (unsigned)ceil_div(F, 256)), 256, 0, ctx.stream>>>(
            (const T *)u, dg, Tn, F, E, dW_r);
        ctx.end();
    }
    const int nruns = (int)ceil_div64(Tn, DWE_TOK);
    ctx.begin(STAGE_DW_EXPERT);
    dw_expert_kernel<T><<<dim3((unsigned)ceil_div(S, 64), (unsigned)ceil_div(F, 64), (unsigned)(E * nruns)), 256, 0,
                          ctx.stream>>>((const T *)u, dBC, idx, w, Tn, F, S, E, k, nruns, dW_e);
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}
}  // namespace

bool ssd_adjoint_supported(int P, int N)
{
    return N * adjoint_ps(P) <= 1024 && N >= 1;
}

int launch_fill(LaunchCtx &ctx, float *p, int64_t n, float v)
{
    if (n <= 0) return SWIMBA_OK;
    fill_kernel<<<(unsigned)ceil_div64(n, 256), 256, 0, ctx.stream>>>(p, n, v);
    ctx.launches++;
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

int launch_ssd_adjoint(LaunchCtx &ctx, int dtype, const void *x, const void *dy, const void *BC, const float *dt,
                       const float *A, const float *dt_bias, const float *h0, int B, int L, int H, int P, int N,
                       int G, float *dBC)
{
    if (B <= 0 || L <= 0) return SWIMBA_OK;
    if (dtype == SWIMBA_DTYPE_FP32)
        return launch_adjoint_t<float>(ctx, x, dy, BC, dt, A, dt_bias, h0, B, L, H, P, N, G, dBC);
    return launch_adjoint_t<__nv_bfloat16>(ctx, x, dy, BC, dt, A, dt_bias, h0, B, L, H, P, N, G, dBC);
}

int launch_weight_grads(LaunchCtx &ctx, int dtype, const void *u, const void *W_r, const void *slots,
                        const int32_t *idx, const float *w, const float *dBC, int64_t Tn, int F, int S, int E,
                        int k, float *pi, float *dg, float *dW_r, float *dW_e)
{
    if (Tn <= 0) return SWIMBA_OK;
    if (dtype == SWIMBA_DTYPE_FP32)
        return launch_weight_grads_t<float>(ctx, u, W_r, slots, idx, w, dBC, Tn, F, S, E, k, pi, dg, dW_r, dW_e);
    return launch_weight_grads_t<__nv_bfloat16>(ctx, u, W_r, slots, idx, w, dBC, Tn, F, S, E, k, pi, dg, dW_r, dW_e);
}

}  // namespace swimba
