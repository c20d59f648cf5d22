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

// Softmax over all E of the router logits, one warp per token: pi[T,E].  A lane takes 8 consecutive
// features at a time (one 16- or 32-byte load of u, reused for every expert's row).
template <typename T>
__global__ void __launch_bounds__(256)
router_softmax_kernel(const T *__restrict__ u, const T *__restrict__ W_r, int64_t Tn, int F, int E,
                      float *__restrict__ pi)
{
    const int lane = threadIdx.x & 31;
    const int64_t t = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (t >= Tn) return;
    float g[SWIMBA_MAX_EXPERTS];
    for (int e = 0; e < E; ++e) g[e] = 0.f;
    for (int f0 = lane * 8; f0 < F; f0 += 256) {            // (F is a multiple of 8)
        float uv[8];
        load8(u + t * F + f0, uv);
        for (int e = 0; e < E; ++e) {
            float wv[8];
            load8(W_r + (int64_t)e * F + f0, wv);
            float acc = g[e];
#pragma unroll
            for (int q = 0; q < 8; ++q) acc = fmaf(wv[q], uv[q], acc);
            g[e] = acc;
        }
    }
    float m = -INFINITY;
    for (int e = 0; e < E; ++e) {
        g[e] = warp_sum(g[e]);
        m = fmaxf(m, g[e]);
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

}  // namespace

// ---------------------------------------------------------------------------------------------
// The adjoint through the tile kernel of the forward.  For head h the contribution to dCtilde is
//   dC_t[n] = sum_{s<=t} (prod_{r=s+1..t} a_r) (dy_t[h] . x_s[h]) Delta_s Btilde_s[n]  (+ the h0 term),
// which is the forward's own form  y_t = sum_{s<=t} decay (C_t . B_s) Delta_s x_s  with the roles
//   C := [dy_t[h] | 0],  B := [x_s[h] | 0]  (64 entries padded to the 128 of a state row),
//   x := one 64-wide half c of Btilde_s,
// i.e. a layer of 2H heads (h, c) in H groups.  dBtilde is the same in reversed time,
//   dB_s[n] = Delta_s sum_{t>=s} (prod_{r=s+1..t} a_r) (x_s[h] . dy_t[h]) Ctilde_t[n],
// with position rho = L-1-t carrying the step size of token t+1 (so that the decay between two
// reversed positions is the product the adjoint needs) and x := Ctilde_t half / that step size (the
// kernel multiplies its input by the step size).  The per-head results (bf16) are summed over the
// heads of a group into dBC.  Shapes of the tile kernel only (bf16, P = 64, N = 128).
namespace {
constexpr int VP = 64, VN = 128;

// Operand streams of the virtual layer.  One block per token, thread = (head, 8-element chunk).
template <bool REVERSE>
__global__ void __launch_bounds__(256)
adjoint_pack_kernel(const __nv_bfloat16 *__restrict__ x, const __nv_bfloat16 *__restrict__ dy,
                    const __nv_bfloat16 *__restrict__ BC, const float *__restrict__ dt,
                    const float *__restrict__ dt_bias, int L, int H, int G,
                    __nv_bfloat16 *__restrict__ BCv, __nv_bfloat16 *__restrict__ xv, float *__restrict__ dtv)
{
    const int64_t bt = blockIdx.x;                    // token of the ORIGINAL order
    const int b = (int)(bt / L), t = (int)(bt % L);
    const int64_t ot = REVERSE ? (int64_t)b * L + (L - 1 - t) : bt;      // its position in the virtual layer
    const int S = 2 * G * VN, HG = H / G;
    const int Sv = 2 * H * VN;                        // virtual streams: H groups
    // C / B rows: [x | 0] and [dy | 0] (forward), [dy | 0] and [x | 0] (reverse)
    for (int i = threadIdx.x; i < H * 16; i += blockDim.x) {
        const int h = i >> 4, ch = i & 15;            // 16 chunks of 8 elements per 128-entry row
        uint4 vb = make_uint4(0, 0, 0, 0), vc = make_uint4(0, 0, 0, 0);
        if (ch < 8) {
            const uint4 xr = *reinterpret_cast<const uint4 *>(x + (bt * H + h) * VP + ch * 8);
            const uint4 dr = *reinterpret_cast<const uint4 *>(dy + (bt * H + h) * VP + ch * 8);
            vb = REVERSE ? dr : xr;
            vc = REVERSE ? xr : dr;
        }
        *reinterpret_cast<uint4 *>(BCv + ot * Sv + (int64_t)h * VN + ch * 8) = vb;
        *reinterpret_cast<uint4 *>(BCv + ot * Sv + (int64_t)(H + h) * VN + ch * 8) = vc;
    }
    // step sizes of the virtual heads and their inputs
    for (int i = threadIdx.x; i < 2 * H * 8; i += blockDim.x) {
        const int vh = i >> 3, ch = i & 7;
        const int h = vh >> 1, c = vh & 1, g = h / HG;
        float raw;
        if (REVERSE) raw = (t + 1 < L && dt) ? dt[(bt + 1) * H + h] : 0.f;
        else raw = dt ? dt[bt * H + h] : 0.f;
        if (ch == 0) dtv[ot * 2 * H + vh] = raw;
        const __nv_bfloat16 *src = BC + bt * S + (int64_t)(REVERSE ? G + g : g) * VN + c * 64 + ch * 8;
        uint4 v = *reinterpret_cast<const uint4 *>(src);
        if (REVERSE) {
            const float inv = 1.f / softplus_f(raw + dt_bias[h]);
            uint32_t wv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float lo = __uint_as_float(wv[q] << 16) * inv, hi = __uint_as_float(wv[q] & 0xffff0000u) * inv;
                const __nv_bfloat162 pr = __floats2bfloat162_rn(lo, hi);
                wv[q] = *reinterpret_cast<const uint32_t *>(&pr);
            }
            v = make_uint4(wv[0], wv[1], wv[2], wv[3]);
        }
        *reinterpret_cast<uint4 *>(xv + (ot * 2 * H + vh) * VP + ch * 8) = v;
    }
}

// A, dt_bias of the virtual heads and the transposed initial state (forward pass only):
// h0v[b, (h,c), p', n'] = h0[b, h, p = n', n = 64 c + p'] for n' < 64, else 0.
__global__ void __launch_bounds__(256)
adjoint_params_kernel(const float *__restrict__ A, const float *__restrict__ dt_bias, const float *__restrict__ h0,
                      int B, int H, float *__restrict__ Av, float *__restrict__ biasv, float *__restrict__ h0v)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < 2 * H) {
        Av[i] = A[i >> 1];
        biasv[i] = dt_bias[i >> 1];
    }
    const int64_t total = (int64_t)B * 2 * H * VP * VN;
    if (h0v && i < total) {
        const int np = (int)(i % VN), pp = (int)((i / VN) % VP);
        const int vh = (int)((i / ((int64_t)VN * VP)) % (2 * H));
        const int64_t b = i / ((int64_t)VN * VP * 2 * H);
        const int h = vh >> 1, c = vh & 1;
        h0v[i] = (np < VP && h0) ? h0[((b * H + h) * VP + np) * VN + 64 * c + pp] : 0.f;
    }
}

// dBC[t, column block] = sum over the heads of the group of the virtual layer's outputs (times the
// head's own step size in the reverse pass).  One block per token, thread = column n.
template <bool REVERSE>
__global__ void __launch_bounds__(128)
adjoint_reduce_kernel(const __nv_bfloat16 *__restrict__ yv, const float *__restrict__ dt,
                      const float *__restrict__ dt_bias, int L, int H, int G, float *__restrict__ dBC)
{
    const int64_t bt = blockIdx.x;
    const int b = (int)(bt / L), t = (int)(bt % L);
    const int64_t ot = REVERSE ? (int64_t)b * L + (L - 1 - t) : bt;
    const int S = 2 * G * VN, HG = H / G;
    const int n = threadIdx.x, c = n >> 6, pp = n & 63;
    __shared__ float s_delta[1024];                       // the token's step sizes, one per head
    if (REVERSE) {
        for (int h = threadIdx.x; h < H; h += blockDim.x)
            s_delta[h] = softplus_f((dt ? dt[bt * H + h] : 0.f) + dt_bias[h]);
        __syncthreads();
    }
    for (int g = 0; g < G; ++g) {
        float acc = 0.f;
        for (int hh = 0; hh < HG; ++hh) {
            const int h = g * HG + hh;
            float v = __bfloat162float(yv[(ot * 2 * H + 2 * h + c) * VP + pp]);
            if (REVERSE) v *= s_delta[h];
            acc += v;
        }
        dBC[bt * S + (int64_t)(REVERSE ? g : G + g) * VN + n] = acc;
    }
}

struct AdjLayout {
    size_t bcv, xv, yv, dtv, av, biasv, h0v, ssd, total;
};
AdjLayout adj_layout(int B, int L, int H, int chunk, int sm_count)
{
    auto up = [](size_t v) { return (v + 255) / 256 * 256; };
    const size_t T = (size_t)B * L;
    AdjLayout l;
    size_t off = 0;
    l.bcv = off;   off += up(T * 2 * H * VN * 2);
    l.xv = off;    off += up(T * 2 * H * VP * 2);
    l.yv = off;    off += up(T * 2 * H * VP * 2);
    l.dtv = off;   off += up(T * 2 * H * sizeof(float));
    l.av = off;    off += up(2 * (size_t)H * sizeof(float));
    l.biasv = off; off += up(2 * (size_t)H * sizeof(float));
    l.h0v = off;   off += up((size_t)B * 2 * H * VP * VN * sizeof(float));
    l.ssd = off;   off += up(ssd_workspace_bytes(B, L, 2 * H, H, chunk, sm_count));
    l.total = off;
    return l;
}
}  // namespace

size_t ssd_adjoint_tiles_workspace_bytes(int B, int L, int H, int chunk, int sm_count)
{
    return adj_layout(B, L, H, chunk, sm_count).total;
}

int launch_ssd_adjoint_tiles(LaunchCtx &ctx, const void *x, const void *dy, const void *BC, const float *dt,
                             const float *A, const float *dt_bias, const float *h0, int B, int L, int H, int G,
                             int chunk, int sm_count, float *dBC, void *workspace)
{
    if (B <= 0 || L <= 0) return SWIMBA_OK;
    const AdjLayout lay = adj_layout(B, L, H, chunk, sm_count);
    char *ws = (char *)workspace;
    __nv_bfloat16 *BCv = (__nv_bfloat16 *)(ws + lay.bcv), *xv = (__nv_bfloat16 *)(ws + lay.xv);
    __nv_bfloat16 *yv = (__nv_bfloat16 *)(ws + lay.yv);
    float *dtv = (float *)(ws + lay.dtv), *Av = (float *)(ws + lay.av), *biasv = (float *)(ws + lay.biasv);
    float *h0v = (float *)(ws + lay.h0v);
    const int64_t T = (int64_t)B * L;
    const int64_t nparam = (int64_t)B * 2 * H * VP * VN;
    ctx.begin(STAGE_ADJOINT_PACK);
    adjoint_params_kernel<<<(unsigned)ceil_div64(h0 ? nparam : 2 * H, 256), 256, 0, ctx.stream>>>(
        A, dt_bias, h0, B, H, Av, biasv, h0 ? h0v : nullptr);
    ctx.end();
    for (int pass = 0; pass < 2; ++pass) {
        const bool rev = pass == 1;
        ctx.begin(STAGE_ADJOINT_PACK);
        if (rev)
            adjoint_pack_kernel<true><<<(unsigned)T, 256, 0, ctx.stream>>>(
                (const __nv_bfloat16 *)x, (const __nv_bfloat16 *)dy, (const __nv_bfloat16 *)BC, dt, dt_bias, L, H, G,
                BCv, xv, dtv);
        else
            adjoint_pack_kernel<false><<<(unsigned)T, 256, 0, ctx.stream>>>(
                (const __nv_bfloat16 *)x, (const __nv_bfloat16 *)dy, (const __nv_bfloat16 *)BC, dt, dt_bias, L, H, G,
                BCv, xv, dtv);
        ctx.end();
        if (cudaGetLastError() != cudaSuccess) return SWIMBA_ERR_CUDA;
        const int rc = launch_ssd_tiles(ctx, xv, BCv, dtv, Av, biasv, nullptr, (!rev && h0) ? h0v : nullptr, B, L, 2 * H,
                                        H, chunk, sm_count, yv, nullptr, ws + lay.ssd, false);
        if (rc != SWIMBA_OK) return rc;
        ctx.begin(STAGE_ADJOINT_PACK);
        if (rev)
            adjoint_reduce_kernel<true><<<(unsigned)T, 128, 0, ctx.stream>>>(yv, dt, dt_bias, L, H, G, dBC);
        else
            adjoint_reduce_kernel<false><<<(unsigned)T, 128, 0, ctx.stream>>>(yv, dt, dt_bias, L, H, G, dBC);
        ctx.end();
    }
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

namespace {
// The same sum on tensor cores (bf16 features): a 128 x 128 tile of one expert's matrix per block,
// eight warps of 32 (s) x 64 (f), the entries taken 32 at a time.  Both operands sit in shared memory
// with the contraction index (the entry) as the row, so every fragment is a transposing ldmatrix:
//   A[m = s][k = entry]  from sA[entry][s],   B[k = entry][n = f]  from sB[entry][f].
// w dBC is rounded to bf16 once; accumulation in fp32; split over runs of tokens with atomics.
constexpr int DWM_TOK = 4096, DWM_K = 32, DWM_LD = 136;      // row pitch 272 B: conflict-free ldmatrix
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__global__ void __launch_bounds__(256)
dw_expert_mma_kernel(const __nv_bfloat16 *__restrict__ u, const float *__restrict__ dBC,
                     const int32_t *__restrict__ idx, const float *__restrict__ w, int64_t Tn, int F, int S,
                     int E, int k, int nruns, float *__restrict__ dW_e)
{
    __shared__ int list[DWM_TOK];
    __shared__ int list_n;
    __shared__ __align__(16) __nv_bfloat16 sA[DWM_K][DWM_LD];
    __shared__ __align__(16) __nv_bfloat16 sB[DWM_K][DWM_LD];
    const int e = blockIdx.z / nruns, run = blockIdx.z % nruns;
    const int s0 = blockIdx.x * 128, f0 = blockIdx.y * 128;
    const int64_t t0 = (int64_t)run * DWM_TOK;
    const int nt = (int)min((int64_t)DWM_TOK, Tn - t0);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) list_n = 0;
    __syncthreads();
    for (int i = tid; i < nt * k; i += blockDim.x)
        if (idx[t0 * k + i] == e) list[atomicAdd(&list_n, 1)] = i;
    __syncthreads();
    const int cnt = list_n;
    if (cnt == 0) return;
    const int wm = (warp & 3) * 32, wn = (warp >> 2) * 64;       // the warp's corner inside the tile
    float acc[2][8][4];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int c = 0; c < 8; ++c)
#pragma unroll
            for (int q = 0; q < 4; ++q) acc[a][c][q] = 0.f;
    const int lj = lane >> 3, lr = lane & 7;
    for (int c0 = 0; c0 < cnt; c0 += DWM_K) {
        const int nc = min(DWM_K, cnt - c0);
        __syncthreads();
        // 32 entries x 128 columns of each operand, eight columns per thread and step
        for (int i = tid; i < DWM_K * 16; i += blockDim.x) {
            const int kk = i >> 4, col = (i & 15) * 8;
            uint4 av = make_uint4(0, 0, 0, 0), bv = make_uint4(0, 0, 0, 0);
            if (kk < nc) {
                const int64_t r = t0 * k + list[c0 + kk];
                const int64_t t = r / k;
                const float wr = w[r];
                if (s0 + col < S) {          // (S and F are multiples of 8)
                    const float4 d0 = *reinterpret_cast<const float4 *>(dBC + t * S + s0 + col);
                    const float4 d1 = *reinterpret_cast<const float4 *>(dBC + t * S + s0 + col + 4);
                    const __nv_bfloat162 p0 = __floats2bfloat162_rn(wr * d0.x, wr * d0.y), p1 = __floats2bfloat162_rn(wr * d0.z, wr * d0.w);
                    const __nv_bfloat162 p2 = __floats2bfloat162_rn(wr * d1.x, wr * d1.y), p3 = __floats2bfloat162_rn(wr * d1.z, wr * d1.w);
                    av = make_uint4(*reinterpret_cast<const uint32_t *>(&p0), *reinterpret_cast<const uint32_t *>(&p1),
                                    *reinterpret_cast<const uint32_t *>(&p2), *reinterpret_cast<const uint32_t *>(&p3));
                }
                if (f0 + col < F) bv = *reinterpret_cast<const uint4 *>(u + t * F + f0 + col);
            }
            *reinterpret_cast<uint4 *>(&sA[kk][col]) = av;
            *reinterpret_cast<uint4 *>(&sB[kk][col]) = bv;
        }
        __syncthreads();
#pragma unroll
        for (int k0 = 0; k0 < DWM_K; k0 += 16) {
            uint32_t af[2][4];
#pragma unroll
            for (int a = 0; a < 2; ++a)
                ldmatrix_x4_trans(af[a], (uint32_t)__cvta_generic_to_shared(
                                             &sA[k0 + (lj >> 1) * 8 + lr][wm + 16 * a + (lj & 1) * 8]));
#pragma unroll
            for (int c2 = 0; c2 < 4; ++c2) {
                uint32_t bf[4];
                ldmatrix_x4_trans(bf, (uint32_t)__cvta_generic_to_shared(
                                          &sB[k0 + (lj & 1) * 8 + lr][wn + 16 * c2 + (lj >> 1) * 8]));
#pragma unroll
                for (int a = 0; a < 2; ++a) {
                    mma_16816(acc[a][2 * c2], af[a], bf[0], bf[1]);
                    mma_16816(acc[a][2 * c2 + 1], af[a], bf[2], bf[3]);
                }
            }
        }
    }
    const int g = lane >> 2, q2 = (lane & 3) * 2;
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int c = 0; c < 8; ++c)
#pragma unroll
            for (int hrow = 0; hrow < 2; ++hrow) {
                const int srow = s0 + wm + 16 * a + g + 8 * hrow;
                const int f = f0 + wn + 8 * c + q2;
                if (srow < S && f < F) {            // (F is even)
                    float *dst = dW_e + ((int64_t)e * S + srow) * F + f;
                    atomicAdd(dst, acc[a][c][2 * hrow]);
                    atomicAdd(dst + 1, acc[a][c][2 * hrow + 1]);
                }
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
    ctx.begin(STAGE_DW_EXPERT);
    if (sizeof(T) == 2 && F % 8 == 0 && S % 8 == 0) {
        const int nruns = (int)ceil_div64(Tn, DWM_TOK);
        dw_expert_mma_kernel<<<dim3((unsigned)ceil_div(S, 128), (unsigned)ceil_div(F, 128), (unsigned)(E * nruns)), 256, 0,
                               ctx.stream>>>((const __nv_bfloat16 *)u, dBC, idx, w, Tn, F, S, E, k, nruns, dW_e);
    } else {
        const int nruns = (int)ceil_div64(Tn, DWE_TOK);
        dw_expert_kernel<T><<<dim3((unsigned)ceil_div(S, 64), (unsigned)ceil_div(F, 64), (unsigned)(E * nruns)), 256, 0,
                              ctx.stream>>>((const T *)u, dBC, idx, w, Tn, F, S, E, k, nruns, dW_e);
    }
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
