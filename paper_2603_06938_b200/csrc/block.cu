// The rest of the block around the mixer (Section "Swimba layer": the in-projection becomes a
// mixture of experts and the rest of the Mamba-2 layer is kept unchanged): causal depthwise
// convolution + SiLU on the [x | B | C] stream, the gated RMS norm rmsnorm(y * silu(z)) * weight,
// and the conversion of the step-size columns of the shared in-projection to fp32.  All three are
// streaming kernels (every element read and written once).
#include "internal.h"

namespace swimba {

namespace {
constexpr int CV_K = 4;        // widest convolution window
constexpr int CV_STRIP = 8;    // tokens per thread

__device__ __forceinline__ float silu_f(float v) { return v / (1.f + __expf(-v)); }

template <typename T> __device__ __forceinline__ void store8(T *p, const float (&v)[8]);
template <> __device__ __forceinline__ void store8<float>(float *p, const float (&v)[8]) {
    *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4 *>(p + 4) = make_float4(v[4], v[5], v[6], v[7]);
}
template <> __device__ __forceinline__ void store8<__nv_bfloat16>(__nv_bfloat16 *p, const float (&v)[8]) {
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat162 q = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
        o[i] = *reinterpret_cast<const uint32_t *>(&q);
    }
    *reinterpret_cast<uint4 *>(p) = make_uint4(o[0], o[1], o[2], o[3]);
}
}  // namespace

// out[b,t,c] = silu(bias[c] + sum_{i<K} w[c,i] in[b, t-(K-1)+i, c]) over the channels c of
// [x' (D, rows of stride ldx) | B'C' (S)]; tokens before the call come from state_in[b,K-1,C]
// (zeros when null).  A thread owns 8 channels and a strip of CV_STRIP tokens and slides its
// window along the strip; the thread of a sequence's last strip also writes state_out.
template <typename T>
__global__ void __launch_bounds__(256, 2)
conv_silu_kernel(const T *__restrict__ xp, int64_t ldx, const T *__restrict__ bcp, const float *__restrict__ cw,
                 const float *__restrict__ cb, const T *__restrict__ state_in, int B, int L, int D, int S,
                 int K, T *__restrict__ x, T *__restrict__ bc, T *__restrict__ state_out)
{
    grid_dep_wait();
    const int C = D + S, ngrp = C / 8;
    const int nstrip = ceil_div(L, CV_STRIP);
    const int64_t item = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (item >= (int64_t)B * nstrip * ngrp) return;
    const int grp = (int)(item % ngrp);
    const int strip = (int)((item / ngrp) % nstrip);
    const int b = (int)(item / ((int64_t)ngrp * nstrip));
    const int c0 = grp * 8;
    const bool from_x = c0 < D;
    const T *src = from_x ? xp + c0 : bcp + (c0 - D);
    const int64_t lds = from_x ? ldx : (int64_t)S;
    T *dst = from_x ? x + c0 : bc + (c0 - D);
    const int64_t ldd = from_x ? (int64_t)D : (int64_t)S;
    // taps aligned to the end of a window of CV_K: tap j multiplies the token CV_K-1-j steps back
    float wt[CV_K][8], bias[8];
    if (cb) {
        load8(cb + c0, bias);
    } else {
#pragma unroll
        for (int q = 0; q < 8; ++q) bias[q] = 0.f;
    }
    if (K == CV_K) {
        // one 16-byte load per channel: its four taps
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float4 t4 = *reinterpret_cast<const float4 *>(cw + (int64_t)(c0 + q) * CV_K);
            wt[0][q] = t4.x; wt[1][q] = t4.y; wt[2][q] = t4.z; wt[3][q] = t4.w;
        }
    } else {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
#pragma unroll
            for (int j = 0; j < CV_K; ++j) {
                const int i = j - (CV_K - K);
                wt[j][q] = i >= 0 ? cw[(int64_t)(c0 + q) * K + i] : 0.f;
            }
        }
    }
    const int t0 = strip * CV_STRIP;
    // token at position tt of this sequence (tt may be negative: before the call)
    auto fetch = [&](int tt, float (&v)[8]) {
        if (tt >= 0) {
            load8(src + ((int64_t)b * L + tt) * lds, v);
        } else if (state_in && tt >= -(K - 1)) {
            load8(state_in + ((int64_t)b * (K - 1) + (K - 1 + tt)) * C + c0, v);
        } else {
#pragma unroll
            for (int q = 0; q < 8; ++q) v[q] = 0.f;
        }
    };
    // all rows of the strip and its history are loaded first (raw, so that they are in flight
    // together), then widened one by one into the sliding window
    typename Raw8<T>::type raw[CV_STRIP];
    const int t1 = min(L, t0 + CV_STRIP);
#pragma unroll
    for (int r = 0; r < CV_STRIP; ++r)
        if (t0 + r < t1) load_raw8(src + ((int64_t)b * L + t0 + r) * lds, raw[r]);
    float win[CV_K][8];
#pragma unroll
    for (int j = 0; j < CV_K - 1; ++j) fetch(t0 - (CV_K - 1) + j, win[j]);
#pragma unroll
    for (int r = 0; r < CV_STRIP; ++r) {
        if (t0 + r >= t1) break;
        unpack8(raw[r], win[(r + CV_K - 1) % CV_K]);
        float o[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            float acc = bias[q];
#pragma unroll
            for (int j = 0; j < CV_K; ++j) acc = fmaf(wt[j][q], win[(r + j) % CV_K][q], acc);
            o[q] = silu_f(acc);
        }
        store8<T>(dst + ((int64_t)b * L + t0 + r) * ldd, o);
    }
    if (state_out && strip == nstrip - 1) {
        for (int i = 0; i < K - 1; ++i) {
            float v[8];
            fetch(L - (K - 1) + i, v);
            store8<T>(state_out + ((int64_t)b * (K - 1) + i) * C + c0, v);
        }
    }
}

// out[t, g-th group] = v / sqrt(mean(v^2) + eps) * weight,  v = y * silu(z); one block per
// (token, group), two passes over the group (the second hits in cache).
template <typename T>
__global__ void __launch_bounds__(128)
gated_rmsnorm_kernel(const T *__restrict__ y, const T *__restrict__ z, int64_t ldz, const float *__restrict__ wt,
                     int D, int ngroups, float eps, T *__restrict__ out)
{
    grid_dep_wait();
    __shared__ float s_part[4];
    const int gs = D / ngroups;
    const int64_t t = blockIdx.x / ngroups;
    const int g = blockIdx.x % ngroups;
    const T *yr = y + t * D + g * gs;
    const T *zr = z + t * ldz + g * gs;
    float ss = 0.f;
    for (int c = threadIdx.x * 8; c < gs; c += 128 * 8) {
        float yv[8], zv[8];
        load8(yr + c, yv);
        load8(zr + c, zv);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float v = yv[q] * silu_f(zv[q]);
            ss = fmaf(v, v, ss);
        }
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
    __syncthreads();
    const float tot = (s_part[0] + s_part[1]) + (s_part[2] + s_part[3]);
    const float r = rsqrtf(tot / gs + eps);
    for (int c = threadIdx.x * 8; c < gs; c += 128 * 8) {
        float yv[8], zv[8], o[8];
        load8(yr + c, yv);
        load8(zr + c, zv);
#pragma unroll
        for (int q = 0; q < 8; ++q) o[q] = yv[q] * silu_f(zv[q]) * r * wt[g * gs + c + q];
        store8<T>(out + t * D + g * gs + c, o);
    }
}

// dt[t, h] (float) = zxdt[t, off + h]
template <typename T>
__global__ void __launch_bounds__(256)
dt_columns_kernel(const T *__restrict__ zxdt, int64_t ld, int off, int64_t Ttok, int H, float *__restrict__ dt)
{
    grid_dep_wait();
    const int64_t n = Ttok * H;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        dt[i] = to_f32<T>(zxdt[(i / H) * ld + off + (int)(i % H)]);
}

int launch_conv_silu(LaunchCtx &ctx, int dtype, const void *xp, int64_t ldx, const void *bcp, const float *cw,
                     const float *cb, const void *state_in, int B, int L, int D, int S, int K, void *x,
                     void *bc, void *state_out)
{
    if (B <= 0 || L <= 0) return SWIMBA_OK;
    const int64_t items = (int64_t)B * ceil_div(L, CV_STRIP) * ((D + S) / 8);
    const dim3 grid((unsigned)ceil_div64(items, 256)), block(256);
    ctx.begin(STAGE_CONV);
    if (dtype == SWIMBA_DTYPE_FP32)
        conv_silu_kernel<float><<<grid, block, 0, ctx.stream>>>((const float *)xp, ldx, (const float *)bcp, cw, cb,
                                                                 (const float *)state_in, B, L, D, S, K, (float *)x,
                                                                 (float *)bc, (float *)state_out);
    else
        conv_silu_kernel<__nv_bfloat16><<<grid, block, 0, ctx.stream>>>(
            (const __nv_bfloat16 *)xp, ldx, (const __nv_bfloat16 *)bcp, cw, cb, (const __nv_bfloat16 *)state_in, B, L,
            D, S, K, (__nv_bfloat16 *)x, (__nv_bfloat16 *)bc, (__nv_bfloat16 *)state_out);
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

int launch_gated_rmsnorm(LaunchCtx &ctx, int dtype, const void *y, const void *z, int64_t ldz, const float *wt,
                         int64_t T, int D, int ngroups, float eps, void *out)
{
    if (T <= 0) return SWIMBA_OK;
    const dim3 grid((unsigned)(T * ngroups)), block(128);
    ctx.begin(STAGE_GATED_NORM);
    if (dtype == SWIMBA_DTYPE_FP32)
        gated_rmsnorm_kernel<float><<<grid, block, 0, ctx.stream>>>((const float *)y, (const float *)z, ldz, wt, D,
                                                                     ngroups, eps, (float *)out);
    else
        gated_rmsnorm_kernel<__nv_bfloat16><<<grid, block, 0, ctx.stream>>>(
            (const __nv_bfloat16 *)y, (const __nv_bfloat16 *)z, ldz, wt, D, ngroups, eps, (__nv_bfloat16 *)out);
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

int launch_dt_columns(LaunchCtx &ctx, int dtype, const void *zxdt, int64_t ld, int off, int64_t T, int H, float *dt)
{
    if (T <= 0) return SWIMBA_OK;
    int64_t blocks = ceil_div64(T * H, 256);
    if (blocks > 148 * 8) blocks = 148 * 8;
    ctx.begin(STAGE_DT_COLUMNS);
    if (dtype == SWIMBA_DTYPE_FP32)
        dt_columns_kernel<float><<<(unsigned)blocks, 256, 0, ctx.stream>>>((const float *)zxdt, ld, off, T, H, dt);
    else
        dt_columns_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, ctx.stream>>>((const __nv_bfloat16 *)zxdt, ld, off, T, H, dt);
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

}  // namespace swimba
