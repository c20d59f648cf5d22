// Step sizes and tile log-decays of the SSD evaluation (Background, "Mamba-2 and SSD"; the
// transition is shared by all experts: shared-A equation).  Per token t of head h, with
// Delta_t = softplus(dt_t + dt_bias_h) and l_t = sum_{r <= t, r in t's 128-token tile} Delta_r A_h log2 e,
// two arrays are produced:
//   l2[(b*H + h)*Lpad + t] = l_t
//   rec[((b*H + h)*ntile + tile)] = one record per 128-token tile, copied to shared memory as a block:
//       wp[128]  W(Delta_t 2^(l_last - l_t))      weight of token t in the tile's end state
//       cb[128]  Delta_t 2^(l_blockend - l_t)     weight of token t at the end of its 32-token block
//       ends[4]  l at the end of each 32-token block (ends[3] = l_last)
// Every exponent is <= 0.  W(w) is w as a two-term bf16 sum packed in one word (high part in the low
// half, remainder in the high half): round(w_hi x + round(w_lo x)) is w x rounded once for a bf16 x,
// up to a term of relative size 2^-17.  Positions past L carry Delta = 0.
// The work depends on dt only, so it runs either as a kernel of its own or as extra blocks of
// the router kernel.
#pragma once
#include "common.cuh"

namespace swimba {

constexpr int SCALARS_TILE = 128;

struct TileScalars {            // (the shared-memory image as well)
    uint32_t wp[SCALARS_TILE];
    float cb[SCALARS_TILE];
    float ends[4];
};
static_assert(sizeof(TileScalars) % 16 == 0, "tile records are moved by 16-byte bulk copies");

struct ScalarsArgs {
    const float *dt, *A, *dt_bias;
    float *l2;            // null: nothing to do
    TileScalars *rec;
    int L, Lpad, H, B;
    // packed batch (sequences of different lengths back to back): per 128-token tile of the batch,
    // (first token, valid tokens); tiles start at sequence starts.  dt is then [T, H], the arrays
    // are laid out [H, tiles] and Lpad = 128 * tiles, B = 1.  Null: dense [B, L].
    const int2 *tile_tab = nullptr;
};

__host__ __device__ inline int64_t scalars_units(const ScalarsArgs &a)
{
    return a.l2 ? (int64_t)(a.Lpad / SCALARS_TILE) * a.H * a.B : 0;
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
    int hh[NU], nleft[NU];
    int64_t out[NU];
#pragma unroll
    for (int q = 0; q < NU; ++q) {
        const int64_t unit = unit0 + q;
        const bool act = unit < nunits;
        const int tile = act ? (int)(unit % ntile) : 0;
        const int h = act ? (int)((unit / ntile) % a.H) : 0;
        const int64_t b = act ? unit / ((int64_t)ntile * a.H) : 0;
        // first token of the lane's four in dt, and tokens of the tile that exist from there on
        int64_t tok = b * a.L + tile * SCALARS_TILE + lane * 4;
        int left = a.L - (tile * SCALARS_TILE + lane * 4);
        if (a.tile_tab && act) {
            const int2 tt2 = a.tile_tab[tile];
            tok = (int64_t)tt2.x + lane * 4;
            left = tt2.y - lane * 4;
        }
        hh[q] = h;
        nleft[q] = left;
        out[q] = act ? (b * a.H + h) * ntile + tile : -1;        // record index
#pragma unroll
        for (int i = 0; i < 4; ++i)
            raw[q][i] = (act && a.dt && i < left) ? a.dt[(tok + i) * a.H + h] : 0.f;
    }
#pragma unroll
    for (int q = 0; q < NU; ++q) {
        if (out[q] < 0) continue;                       // (uniform over the warp)
        const float bias = a.dt_bias[hh[q]];
        const float a2 = a.A[hh[q]] * 1.4426950408889634f;
        float d[4], p[4], run = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            d[i] = i < nleft[q] ? softplus_f(raw[q][i] + bias) : 0.f;
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
        const float l_last = __shfl_sync(0xffffffffu, incl, 31);
        const float l_blk = __shfl_sync(0xffffffffu, incl, lane | 7);   // 8 lanes = one 32-token block
        float lv[4], cb[4];
        uint32_t wp[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            lv[i] = excl + p[i];
            const float w = d[i] * exp2f(l_last - lv[i]);
            const __nv_bfloat16 w_hi = __float2bfloat16_rn(w);
            wp[i] = (uint32_t)__bfloat16_as_ushort(w_hi) |
                    ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(w - __bfloat162float(w_hi))) << 16);
            cb[i] = d[i] * exp2f(l_blk - lv[i]);
        }
        TileScalars *rec = a.rec + out[q];
        reinterpret_cast<float4 *>(a.l2 + out[q] * SCALARS_TILE)[lane] = make_float4(lv[0], lv[1], lv[2], lv[3]);
        reinterpret_cast<uint4 *>(rec->wp)[lane] = make_uint4(wp[0], wp[1], wp[2], wp[3]);
        reinterpret_cast<float4 *>(rec->cb)[lane] = make_float4(cb[0], cb[1], cb[2], cb[3]);
        if ((lane & 7) == 7) rec->ends[lane >> 3] = incl;
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
