// Step sizes and tile log-decays of the SSD evaluation (Background, "Mamba-2 and SSD"; the
// transition is shared by all experts: shared-A equation):
//   Delta_t = softplus(dt_t + dt_bias_h),
//   dl[(b*H + h)*Lpad + t] = (Delta_t, sum_{r <= t, r in t's 128-token tile} Delta_r A_h log2 e);
// positions past L carry Delta = 0, so the last entry of a tile is always the tile's total.
// The work depends on dt only, so it runs either as a kernel of its own or as extra blocks of
// the router kernel.
#pragma once
#include "common.cuh"

namespace swimba {

constexpr int SCALARS_TILE = 128;

struct ScalarsArgs {
    const float *dt, *A, *dt_bias;
    float2 *dl;           // null: nothing to do
    int L, Lpad, H, B;
};

__host__ __device__ inline int64_t scalars_units(const ScalarsArgs &a)
{
    return a.dl ? (int64_t)(a.Lpad / SCALARS_TILE) * a.H * a.B : 0;
}


// NU consecutive (tile, head, sequence) units, worked by one warp without any block-level
// synchronisation: lane l owns tokens 4l .. 4l+3 of a tile; the loads of all NU units are issued
// before the first use.  The tile's running log-decay is summed token by token inside a lane and
// by a shuffle scan across lanes.
template <int NU>
__device__ __forceinline__ void ssd_scalars_warp(const ScalarsArgs &a, int64_t unit0, int lane)
{
    const int ntile = a.Lpad / SCALARS_TILE;
    const int64_t nunits = scalars_units(a);
    float raw[NU][4];
    int hh[NU], tt[NU];
    int64_t out[NU];
#pragma unroll
    for (int q = 0; q < NU; ++q) {
        const int64_t unit = unit0 + q;
        const bool act = unit < nunits;
        const int tile = act ? (int)(unit % ntile) : 0;
        const int h = act ? (int)((unit / ntile) % a.H) : 0;
        const int64_t b = act ? unit / ((int64_t)ntile * a.H) : 0;
        const int t = tile * SCALARS_TILE + lane * 4;
        hh[q] = h;
        tt[q] = t;
        out[q] = act ? (b * a.H + h) * a.Lpad + t : -1;
#pragma unroll
        for (int i = 0; i < 4; ++i)
            raw[q][i] = (act && a.dt && t + i < a.L) ? a.dt[(b * a.L + t + i) * a.H + h] : 0.f;
    }
#pragma unroll
    for (int q = 0; q < NU; ++q) {
        if (out[q] < 0) continue;                       // (uniform over the warp)
        const float bias = a.dt_bias[hh[q]];
        const float a2 = a.A[hh[q]] * 1.4426950408889634f;
        float d[4], p[4], run = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            d[i] = tt[q] + i < a.L ? softplus_f(raw[q][i] + bias) : 0.f;
            run += d[i] * a2;
            p[i] = run;
        }
        float incl = run;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float nb = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += nb;
        }
        const float excl = incl - run;
        float4 *dst = reinterpret_cast<float4 *>(a.dl + out[q]);
        dst[0] = make_float4(d[0], excl + p[0], d[1], excl + p[1]);
        dst[1] = make_float4(d[2], excl + p[2], d[3], excl + p[3]);
    }
}

// The block's share: two units per warp, blocks of any whole number of warps.
__device__ __forceinline__ void ssd_scalars_block(const ScalarsArgs &a, int64_t block)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarp = blockDim.x >> 5;
    ssd_scalars_warp<2>(a, (block * nwarp + warp) * 2, lane);
}

// Blocks of `threads` threads that cover all units.
__host__ __device__ inline int64_t scalars_blocks(const ScalarsArgs &a, int threads)
{
    const int per_block = (threads >> 5) * 2;
    return (scalars_units(a) + per_block - 1) / per_block;
}

}  // namespace swimba
