// Per-timestep evaluation of the single selective-SSM recurrence (selective-SSM equation with
// the channelwise convention; Theorem 1) with the state held in registers: the fp32 path of the
// forward, and K4, the one-token decode update.
#include "internal.h"
#include "tc05.cuh"

namespace swimba {

constexpr int SEQ_TS = 32;   // tokens staged in shared memory per round
constexpr int SEQ_NT = 16;   // state entries per thread

// Block = one (sequence, head).  Thread (p, ns) owns state entries n = ns + i*NS of channel p.
template <typename T, typename TBC>
__global__ void __launch_bounds__(1024)
ssd_sequential_kernel(const T *__restrict__ x, const TBC *__restrict__ BC,
                      const float *__restrict__ dt, const float *__restrict__ A,
                      const float *__restrict__ dt_bias, const float *__restrict__ D,
                      const float *__restrict__ h0, int L, int H, int P, int N, int G, int NS,
                      T *__restrict__ y, float *__restrict__ h_final, const int4 *__restrict__ seq_tab)
{
    extern __shared__ float smem[];
    float *sB = smem;                    // [TS][N]
    float *sC = sB + SEQ_TS * N;         // [TS][N]
    float *sx = sC + SEQ_TS * N;         // [TS][P]
    float *sy = sx + SEQ_TS * P;         // [TS][P]
    float *sdl = sy + SEQ_TS * P;        // [TS] Delta
    float *sa = sdl + SEQ_TS;            // [TS] exp(Delta*A)

    int b = blockIdx.x / H;
    const int h = blockIdx.x % H;
    // seq_tab (packed batches): entry i = (first token, tokens, sequence index) of the i-th listed
    // sequence; tokens are rows of the packed arrays, the states are indexed by the sequence
    int64_t tok_base = (int64_t)b * L;
    if (seq_tab) {
        const int4 e = seq_tab[b];
        tok_base = e.x;
        L = e.y;
        b = e.z;
    }
    const int g = h / (H / G);
    const int S = 2 * G * N;
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int p = tid / NS, ns = tid % NS;
    const float Ah = A[h], bias = dt_bias[h], Dh = D ? D[h] : 0.f;
    const unsigned amask = __activemask();   // the block size need not be a multiple of 32

    float st[SEQ_NT];
#pragma unroll
    for (int i = 0; i < SEQ_NT; ++i) {
        const int n = ns + i * NS;
        st[i] = (h0 && n < N) ? h0[(((int64_t)b * H + h) * P + p) * N + n] : 0.f;
    }

    for (int t0 = 0; t0 < L; t0 += SEQ_TS) {
        const int nt = min(SEQ_TS, L - t0);
        for (int i = tid; i < nt * N; i += nthr) {
            const int tt = i / N, n = i % N;
            const TBC *row = BC + (tok_base + t0 + tt) * S;
            sB[tt * N + n] = to_f32<TBC>(row[g * N + n]);
            sC[tt * N + n] = to_f32<TBC>(row[(G + g) * N + n]);
        }
        for (int i = tid; i < nt * P; i += nthr) {
            const int tt = i / P, pp = i % P;
            sx[tt * P + pp] = to_f32<T>(x[((tok_base + t0 + tt) * H + h) * P + pp]);
        }
        for (int i = tid; i < nt; i += nthr) {        // (blocks may have fewer than SEQ_TS threads)
            const float raw = dt ? dt[(tok_base + t0 + i) * H + h] : 0.f;
            const float delta = softplus_f(raw + bias);
            sdl[i] = delta;
            sa[i] = expf(delta * Ah);
        }
        __syncthreads();
        for (int tt = 0; tt < nt; ++tt) {
            const float xv = sx[tt * P + p];
            const float dx = sdl[tt] * xv, a = sa[tt];
            float acc = 0.f;
#pragma unroll
            for (int i = 0; i < SEQ_NT; ++i) {
                const int n = ns + i * NS;
                if (n < N) {
                    st[i] = fmaf(a, st[i], dx * sB[tt * N + n]);
                    acc = fmaf(sC[tt * N + n], st[i], acc);
                }
            }
            for (int o = NS >> 1; o > 0; o >>= 1) acc += __shfl_xor_sync(amask, acc, o);
            if (ns == 0) sy[tt * P + p] = acc + Dh * xv;
        }
        __syncthreads();
        for (int i = tid; i < nt * P; i += nthr) {
            const int tt = i / P, pp = i % P;
            y[((tok_base + t0 + tt) * H + h) * P + pp] = from_f32<T>(sy[tt * P + pp]);
        }
        __syncthreads();
    }
    if (h_final) {
#pragma unroll
        for (int i = 0; i < SEQ_NT; ++i) {
            const int n = ns + i * NS;
            if (n < N) h_final[(((int64_t)b * H + h) * P + p) * N + n] = st[i];
        }
    }
}

static int seq_ns(int N)
{
    int ns = 1;
    while (ns * SEQ_NT < N) ns <<= 1;
    return ns;
}

template <typename T, typename TBC>
static int launch_seq_t(LaunchCtx &ctx, const void *x, const void *BC, const float *dt,
                        const float *A, const float *dt_bias, const float *D, const float *h0,
                        int B, int L, int H, int P, int N, int G, void *y, float *h_final,
                        const int4 *seq_tab = nullptr)
{
    const int NS = seq_ns(N);
    const size_t smem = sizeof(float) * (size_t)(2 * SEQ_TS * N + 2 * SEQ_TS * P + 2 * SEQ_TS);
    auto kern = ssd_sequential_kernel<T, TBC>;
    if (smem > 48 * 1024 && !ensure_dynamic_smem((const void *)kern, smem)) return SWIMBA_ERR_CUDA;
    ctx.begin(STAGE_SSD_SEQUENTIAL);
    kern<<<B * H, P * NS, smem, ctx.stream>>>((const T *)x, (const TBC *)BC, dt, A, dt_bias, D, h0,
                                             L, H, P, N, G, NS, (T *)y, h_final, seq_tab);
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

int launch_ssd_sequential(LaunchCtx &ctx, int dtype, const void *x, const void *BC, bool bc_fp32,
                          const float *dt, const float *A, const float *dt_bias, const float *D,
                          const float *h0, int B, int L, int H, int P, int N, int G, void *y,
                          float *h_final)
{
    if (B <= 0 || L <= 0) return SWIMBA_OK;
    if (dtype == SWIMBA_DTYPE_FP32)
        return launch_seq_t<float, float>(ctx, x, BC, dt, A, dt_bias, D, h0, B, L, H, P, N, G, y, h_final);
    if (bc_fp32)
        return launch_seq_t<__nv_bfloat16, float>(ctx, x, BC, dt, A, dt_bias, D, h0, B, L, H, P, N, G, y, h_final);
    return launch_seq_t<__nv_bfloat16, __nv_bfloat16>(ctx, x, BC, dt, A, dt_bias, D, h0, B, L, H, P, N, G, y, h_final);
}

// The same over a list of sequences of a packed batch (device table of n entries: first token,
// tokens, sequence index); bf16 streams.  Used for the sequences of a packed batch that are only a
// few tokens long (decode tokens riding in a prefill batch): one block per (sequence, head) reads
// the state, steps through the tokens and writes the state, instead of a 128-token tile each.
int launch_ssd_sequential_listed(LaunchCtx &ctx, const void *x, const void *BC, const float *dt, const float *A,
                                 const float *dt_bias, const float *D, const float *h0, const int4 *seq_tab, int n,
                                 int H, int P, int N, int G, void *y, float *h_final)
{
    if (n <= 0) return SWIMBA_OK;
    return launch_seq_t<__nv_bfloat16, __nv_bfloat16>(ctx, x, BC, dt, A, dt_bias, D, h0, n, 0, H, P, N, G, y, h_final,
                                                      seq_tab);
}

// ------------------------------------------------------------------------------------------
// K4: decode.  The state [B,H,P,N] fp32 is read and written exactly once: the kernel is a pure
// HBM stream.  One warp owns ROWS consecutive channels p of one (b,h); a row is N floats read
// as float4 per lane, all ROWS loads are issued before any use.
// ------------------------------------------------------------------------------------------
constexpr int DEC_ROWS = 8;

__device__ __forceinline__ float4 load_bc4(const float *p, int v)
{
    return reinterpret_cast<const float4 *>(p)[v];
}
__device__ __forceinline__ float4 load_bc4(const __nv_bfloat16 *p, int v)
{
    const uint2 raw = reinterpret_cast<const uint2 *>(p)[v];
    return make_float4(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xffff0000u),
                       __uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xffff0000u));
}

template <typename T, typename TBC>
__global__ void __launch_bounds__(256)
decode_update_kernel(const T *__restrict__ x, const TBC *__restrict__ BC,
                     const float *__restrict__ dt, const float *__restrict__ A,
                     const float *__restrict__ dt_bias, const float *__restrict__ D,
                     float *__restrict__ state, int B, int H, int P, int N, int G,
                     T *__restrict__ y)
{
    grid_dep_wait();      // the mixed streams come from the projection kernel
    const int lane = threadIdx.x & 31;
    const int S = 2 * G * N;
    const int pgroups = ceil_div(P, DEC_ROWS);
    const int64_t nwork = (int64_t)B * H * pgroups;
    const int64_t nwarps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int nv = N >> 2;   // groups of 4 state entries per row
    for (int64_t wk = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); wk < nwork;
         wk += nwarps) {
        const int pg = (int)(wk % pgroups);
        const int64_t bh = wk / pgroups;
        const int h = (int)(bh % H), b = (int)(bh / H);
        const int g = h / (H / G);
        const float delta = softplus_f((dt ? dt[bh] : 0.f) + dt_bias[h]);
        const float a = expf(delta * A[h]);
        const float Dh = D ? D[h] : 0.f;
        const TBC *Bp = BC + (int64_t)b * S + g * N;
        const TBC *Cp = BC + (int64_t)b * S + (G + g) * N;
        float xv[DEC_ROWS], acc[DEC_ROWS];
#pragma unroll
        for (int r = 0; r < DEC_ROWS; ++r) {
            const int p = pg * DEC_ROWS + r;
            xv[r] = (p < P) ? to_f32<T>(x[bh * P + p]) : 0.f;
            acc[r] = 0.f;
        }
        for (int v = lane; v < nv; v += 32) {
            float4 s[DEC_ROWS];
#pragma unroll
            for (int r = 0; r < DEC_ROWS; ++r) {
                const int p = pg * DEC_ROWS + r;
                if (p < P)
                    s[r] = __ldcs(reinterpret_cast<const float4 *>(state + (bh * P + p) * N) + v);
            }
            const float4 bb = load_bc4(Bp, v), cc = load_bc4(Cp, v);
#pragma unroll
            for (int r = 0; r < DEC_ROWS; ++r) {
                const int p = pg * DEC_ROWS + r;
                if (p < P) {
                    const float dx = delta * xv[r];
                    s[r].x = fmaf(a, s[r].x, dx * bb.x);
                    s[r].y = fmaf(a, s[r].y, dx * bb.y);
                    s[r].z = fmaf(a, s[r].z, dx * bb.z);
                    s[r].w = fmaf(a, s[r].w, dx * bb.w);
                    acc[r] = fmaf(cc.x, s[r].x, acc[r]);
                    acc[r] = fmaf(cc.y, s[r].y, acc[r]);
                    acc[r] = fmaf(cc.z, s[r].z, acc[r]);
                    acc[r] = fmaf(cc.w, s[r].w, acc[r]);
                    __stcs(reinterpret_cast<float4 *>(state + (bh * P + p) * N) + v, s[r]);
                }
            }
        }
#pragma unroll
        for (int r = 0; r < DEC_ROWS; ++r) {
            const float tot = warp_sum(acc[r]);
            const int p = pg * DEC_ROWS + r;
            if (lane == r && p < P) y[bh * P + p] = from_f32<T>(tot + Dh * xv[r]);
        }
    }
}

int launch_decode_update(LaunchCtx &ctx, int dtype, const void *x, const void *BC, bool bc_fp32,
                         const float *dt, const float *A, const float *dt_bias, const float *D,
                         float *state, int B, int H, int P, int N, int G, int sm_count, void *y)
{
    if (B <= 0) return SWIMBA_OK;
    const int64_t nwork = (int64_t)B * H * ceil_div(P, DEC_ROWS);
    const int warps = 8;
    int64_t blocks = ceil_div64(nwork, warps);
    const int64_t cap = (int64_t)sm_count * 8;
    if (blocks > cap) blocks = cap;
    ctx.begin(STAGE_DECODE_UPDATE);
    const dim3 grid((unsigned)blocks), block(warps * 32);
    if (dtype == SWIMBA_DTYPE_FP32)
        launch_kernel(decode_update_kernel<float, float>, grid, block, 0, ctx.stream, true,
                      (const float *)x, (const float *)BC, dt, A, dt_bias, D, state, B, H, P, N, G,
                      (float *)y);
    else if (bc_fp32)
        launch_kernel(decode_update_kernel<__nv_bfloat16, float>, grid, block, 0, ctx.stream, true,
                      (const __nv_bfloat16 *)x, (const float *)BC, dt, A, dt_bias, D, state, B, H, P, N,
                      G, (__nv_bfloat16 *)y);
    else
        launch_kernel(decode_update_kernel<__nv_bfloat16, __nv_bfloat16>, grid, block, 0, ctx.stream,
                      true, (const __nv_bfloat16 *)x, (const __nv_bfloat16 *)BC, dt, A, dt_bias, D,
                      state, B, H, P, N, G, (__nv_bfloat16 *)y);
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

}  // namespace swimba
