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

// One (tile, head, sequence) unit, worked by 128 consecutive threads (i = 0..127 inside the unit).
// Every thread of the block must call this (it holds a __syncthreads); threads whose unit is out
// of range pass active = false.  s_tot: four floats of shared memory private to the unit.
__device__ __forceinline__ void ssd_scalars_unit(const ScalarsArgs &a, int64_t unit, bool active, int i,
                                                 float *s_tot)
{
    const int ntile = a.Lpad / SCALARS_TILE;
    const int lane = i & 31, wq = i >> 5;
    const int tile = (int)(unit % ntile);
    const int h = (int)((unit / ntile) % a.H);
    const int b = (int)(unit / ((int64_t)ntile * a.H));
    const int t = tile * SCALARS_TILE + i;
    float delta = 0.f, l2 = 0.f;
    if (active) {
        const float raw = (a.dt && t < a.L) ? a.dt[((int64_t)b * a.L + t) * a.H + h] : 0.f;
        delta = t < a.L ? softplus_f(raw + a.dt_bias[h]) : 0.f;
        l2 = delta * (a.A[h] * 1.4426950408889634f);
    }
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float nb = __shfl_up_sync(0xffffffffu, l2, o);
        if (lane >= o) l2 += nb;
    }
    if (lane == 31) s_tot[wq] = l2;
    __syncthreads();
    for (int w = 0; w < wq; ++w) l2 += s_tot[w];
    if (active) a.dl[((int64_t)b * a.H + h) * a.Lpad + t] = make_float2(delta, l2);
}

}  // namespace swimba
