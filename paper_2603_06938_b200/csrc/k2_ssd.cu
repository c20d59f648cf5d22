// K2/K3: chunked SSD evaluation of the single selective SSM on tcgen05 tensor cores
// (Background, "Mamba-2 and SSD": matrix products inside chunks, a linear recurrence between
// chunks; the recurrence itself is Theorem 1's h_t = a_t h_{t-1} + Delta_t Btilde_t x_t^T,
// y_t = Ctilde_t^T h_t + D x_t).
//
// A small kernel first turns dt into Delta and the log-decay accumulated inside each 128-token
// tile.  Then one CTA owns one (sequence, pair of heads of one B/C group, segment) and walks its
// segment in tiles of 128 tokens.  With l_i = sum_{r<=i} Delta_r A (inside the tile), per tile:
//   G      = Ctilde Btilde^T                      [128 x 128]  (MMA 1, once for both heads)
// and for each of the two heads
//   Y      = Ctilde H_prev^T                      [128 x 64]   (MMA 3), then scaled in place by
//            exp(l_i) on the CUDA cores
//   M[i,s] = G[i,s] exp(l_i - l_s) Delta_s  for s <= i, else 0      (CUDA cores -> TMEM, bf16)
//   Y     += M X                                               (MMA 2, A operand from TMEM)
//   y_i    = Y_i + D x_i                                       (staged in shared memory, TMA store)
//   dH^T   = Btilde^T (w . X),  w_s = exp(l_last - l_s) Delta_s  [128 x 64]  (MMA 4)
//   H      = exp(l_last) H_prev + dH                           (fp32, registers)
// The carried state never leaves the SM inside a segment: the inter-chunk recurrence is fused.
// Each head has eight compute warps (a thread owns one token row / state index and one half of
// the head dimension) and its own MMA-issuing warp, so that one head's tensor-core and memory
// latencies are covered by the other warps' CUDA-core work.
//
// The decay mask needs exp(l_i - l_s) for every kept (i, s).  Only the four 32x32 blocks on the
// diagonal evaluate it entry by entry.  A block strictly below the diagonal (rows in block w,
// columns in block b < w) factors as
//   exp(l_i - L_w) * exp(L_w - L_{b+1}) * exp(L_{b+1} - l_s),     L_w = l at the end of block w-1,
// every exponent being <= 0 (no overflow, underflow only where the true value underflows), so
// that it costs two multiplications per entry.
//
// Long sequences with few (sequence, head) pairs are cut into segments: a first pass of this
// kernel computes every segment's local end state (MMA 4 only), segment_scan_kernel (K3) chains
// them, and a second pass evaluates each segment from its true incoming state.
#include <vector>

#include "internal.h"
#include "ssd_scalars.cuh"
#include "tc05.cuh"

namespace swimba {

namespace {
constexpr int ST = 128;                 // tokens per tile
constexpr int SP = 64;                  // head dim this kernel is built for
constexpr int SN = 128;                 // state size this kernel is built for
constexpr int NHD = 2;                  // heads per CTA
constexpr int NCW = 8 * NHD;            // compute warps
// warps 0-7: head 0 compute, 8-15: head 1 compute (warp = 8 head + 4 half + row block),
// 16: TMA, 17: MMA issuer head 0 (+ MMA 1), 18: MMA issuer head 1
constexpr int WARP_TMA = NCW, WARP_MMA0 = NCW + 1;
constexpr int SSD_THREADS = 32 * (NCW + 1 + NHD);
constexpr int HEAD_THREADS = 256;
constexpr uint32_t SLAB = 16384;        // 128 rows x 128 bytes

// shared memory map (bytes from the 1024-aligned base)
constexpr uint32_t SM_CB = 0;                        // C0 C1 B0 B1 slabs (single stage)
constexpr uint32_t SM_HEAD = 4 * SLAB;               // per head: X[2] XP HB YS
constexpr uint32_t SM_HEAD_BYTES = 5 * SLAB;
constexpr uint32_t SM_SMALL = SM_HEAD + NHD * SM_HEAD_BYTES;

// TMEM columns: G, then Y, dH and M (bf16 A operand), each 64 columns per head with the two heads
// side by side (one MMA of N = 128 can then write both heads' Y or dH)
constexpr uint32_t TM_G = 0, TM_HEAD = 0, TM_HEAD_COLS = 64, TM_COLS = 512;
constexpr uint32_t TM_Y = 128, TM_DH = 256, TM_M = 384;

enum { MODE_FULL = 0, MODE_STATE_ONLY = 1 };

struct SeqDesc {            // one sequence of a packed batch
    int tok0, len;          // first token in the packed arrays, tokens
    int tile0, seg0;        // first 128-token tile / first segment of the sequence in the batch-wide lists
};

struct SsdParams {
    const float *l2;        // [B,H,Lpad] log2-decay accumulated inside the 128-token tile
    const TileScalars *rec; // [B,H,Lpad/128] per-tile weights and block ends
    const float *D;
    const float *h_in;      // initial states: [B,H,P,N] (nseg == 1) or [B,nseg,H,P,N]; may be null
    float *h_out;           // MODE_FULL: h_final [B,H,P,N] (last segment writes) or null
                            // MODE_STATE_ONLY: local end states [B,nseg,H,P,N]
    float *seg_decay;       // MODE_STATE_ONLY: [B,nseg,H] product of a_t over the segment
    int L, Lpad, H, G, nseg, seg_len, mode;
    int split_tiles;        // > 0 (MODE_FULL, nseg == 1): every (sequence, head pair) is worked by two
                            // CTAs, see ssd_tiles_kernel
    int *d_status;
    // Packed batch (sequences of different lengths back to back in one [T, ...] array): seqs has one
    // entry per sequence plus a closing one, items lists the (sequence, segment) pairs of this launch
    // (grid.x), the scalar arrays are laid out [H, tiles of the batch], and the per-segment state
    // arrays are indexed by seqs[b].seg0 + segment.  seg_states: h_in / state-only h_out are those
    // per-segment arrays (else h_in is [sequences, H, P, N]).  y: base of the output (ragged last
    // tiles are stored row by row).  Null seqs: dense [B, L].
    const SeqDesc *seqs;
    const int2 *items;
    int ntile_total, seg_states;
    void *y;
};

struct __align__(8) HeadBars {
    uint64_t x_full[2], x_free[2];
    uint64_t yoff_full, m_full, yd_full, xp_full, dh_full, h_ready, y_free, y_staged, sc_full;
};
struct __align__(8) SsdBars {
    uint64_t cb_full, cb_empty, g_full, g_free;
    HeadBars hd[NHD];
};

struct __align__(16) SsdSmall {
    TileScalars sc[NHD];     // the current tile's weights and block ends, copied in by the TMA warp
    SsdBars bars;
    uint32_t tmem_slot;
    int abort_flag;
};

// pairs of heads never straddle a B/C group
__host__ __device__ inline int pairs_per_group(int H, int G) { return (H / G + NHD - 1) / NHD; }
}  // namespace

// Stand-alone launch of the step sizes and tile log-decays.
__global__ void __launch_bounds__(256)
ssd_scalars_kernel(const ScalarsArgs args)
{
    // Everything earlier in the stream has completed once the wait returns; only then may the
    // kernel behind this one (the streaming router, which writes without waiting) be let in.
    grid_dep_wait();
    grid_dep_launch();
    ssd_scalars_block(args, blockIdx.x);
}

// Self-test of the bounded wait every tensor-core kernel here relies on: one warp waits, with the
// given cycle limit, on a barrier that nothing ever signals.  The wait must give up, record
// SWIMBA_ERR_DEVICE_TIMEOUT and raise the CTA's abort flag; a second wait must then return at once.
// out[0] = 1 if the first wait reported failure, out[1] = 1 if the second did, out[2] = cycles the
// second wait took.
__global__ void __launch_bounds__(32)
wait_selftest_kernel(int *d_status, long long limit_cycles, long long *out)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        tc::mbar_init(&bar, 1);
        abort_flag = 0;
        tc::fence_mbar_init();
    }
    __syncwarp();
    const bool first = tc::mbar_wait(&bar, 0, &abort_flag, d_status, limit_cycles);
    __syncwarp();
    const long long t0 = clock64();
    const bool second = tc::mbar_wait(&bar, 0, &abort_flag, d_status, limit_cycles);
    const long long t1 = clock64();
    if (threadIdx.x == 0) {
        out[0] = first ? 0 : 1;
        out[1] = second ? 0 : 1;
        out[2] = t1 - t0;
    }
}

int launch_wait_selftest(LaunchCtx &ctx, long long limit_cycles, long long *out_dev)
{
    wait_selftest_kernel<<<1, 32, 0, ctx.stream>>>(ctx.d_status, limit_cycles, out_dev);
    ctx.launches++;
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

// w . X for units [UB, UE) of one lane's 16 (row block, 16-byte chunk) units of its half of the
// head dim: x' = w x with the weight given as a two-term bf16 sum (rounded once).  The unit range
// is known at compile time, so that all loads are issued before the first use.
template <int UB, int UE>
__device__ __forceinline__ void scale_units(const uint8_t *s_x, uint8_t *s_xp, const uint32_t *s_wp, int lane, int hf)
{
    uint4 xr[UE - UB];
    uint32_t wp[UE - UB];
#pragma unroll
    for (int un = UB; un < UE; ++un) {
        const int r = (un >> 2) * 32 + lane;
        wp[un - UB] = s_wp[r];
        xr[un - UB] = *reinterpret_cast<const uint4 *>(s_x + tc::sw128_offset(r, 4 * hf + (un & 3)));
    }
#pragma unroll
    for (int un = UB; un < UE; ++un) {
        const int r = (un >> 2) * 32 + lane;
        const uint32_t hi_u = __byte_perm(wp[un - UB], 0, 0x1010), lo_u = __byte_perm(wp[un - UB], 0, 0x3232);
        const __nv_bfloat162 w_hi2 = *reinterpret_cast<const __nv_bfloat162 *>(&hi_u);
        const __nv_bfloat162 w_lo2 = *reinterpret_cast<const __nv_bfloat162 *>(&lo_u);
        const uint32_t wv[4] = {xr[un - UB].x, xr[un - UB].y, xr[un - UB].z, xr[un - UB].w};
        uint32_t o[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const __nv_bfloat162 xv = *reinterpret_cast<const __nv_bfloat162 *>(&wv[q]);
            const __nv_bfloat162 pr = __hfma2(w_hi2, xv, __hmul2(w_lo2, xv));
            o[q] = *reinterpret_cast<const uint32_t *>(&pr);
        }
        *reinterpret_cast<uint4 *>(s_xp + tc::sw128_offset(r, 4 * hf + (un & 3))) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// The same for the four units of the thread's own row (state-only tiles), with the row's weight
// multiplied by `f` first: w' = w f is split again into two bf16 terms.
__device__ __forceinline__ void scale_own_row(const uint8_t *s_x, uint8_t *s_xp, uint32_t wp, float f, int i, int hf)
{
    const float w = (__uint_as_float(wp << 16) + __uint_as_float(wp & 0xffff0000u)) * f;
    const __nv_bfloat16 w_hi = __float2bfloat16_rn(w);
    const __nv_bfloat16 w_lo = __float2bfloat16_rn(w - __bfloat162float(w_hi));
    const __nv_bfloat162 w_hi2 = __halves2bfloat162(w_hi, w_hi), w_lo2 = __halves2bfloat162(w_lo, w_lo);
    uint4 xr[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) xr[c] = *reinterpret_cast<const uint4 *>(s_x + tc::sw128_offset(i, 4 * hf + c));
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const uint32_t wv[4] = {xr[c].x, xr[c].y, xr[c].z, xr[c].w};
        uint32_t o[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const __nv_bfloat162 xv = *reinterpret_cast<const __nv_bfloat162 *>(&wv[q]);
            const __nv_bfloat162 pr = __hfma2(w_hi2, xv, __hmul2(w_lo2, xv));
            o[q] = *reinterpret_cast<const uint32_t *>(&pr);
        }
        *reinterpret_cast<uint4 *>(s_xp + tc::sw128_offset(i, 4 * hf + c)) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

template <bool SPLIT>
__global__ void __launch_bounds__(SSD_THREADS, 1)
ssd_tiles_kernel(const __grid_constant__ CUtensorMap tmap_bc, const __grid_constant__ CUtensorMap tmap_x,
                 const __grid_constant__ CUtensorMap tmap_y, const SsdParams prm)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    SsdSmall *sm = (SsdSmall *)(smem + SM_SMALL);
    SsdBars *bars = &sm->bars;
    int *abort_flag = &sm->abort_flag;
    int *d_status = prm.d_status;
    if ((tc::smem_u32(smem) & 1023u) != 0) {      // the swizzled tiles need a 1024-byte aligned base
        if (threadIdx.x == 0) atomicCAS(d_status, 0, SWIMBA_ERR_DEVICE_BOUNDS);
        return;
    }

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // Split launch (grid = [B, head pairs, 2]; used when one CTA per (sequence, head pair) would
    // leave a third of the SMs idle): the CTAs of the first z-plane, which start first, walk the whole
    // sequence but evaluate the first split_tiles tiles for their end state only (about half the
    // cost of a full tile) and produce y from there on; the CTAs of the second plane produce y of
    // those first tiles.  No CTA waits for another.
    constexpr bool split = SPLIT;                                // (prm.split_tiles > 0)
    const bool head_part = split && blockIdx.z == 1;             // y of the leading tiles only
    const bool packed = !SPLIT && prm.seqs != nullptr;
    int seg = split ? 0 : blockIdx.x, b = split ? blockIdx.x : blockIdx.z;
    int L = prm.L, nseg = prm.nseg, tok0 = 0, bco = b;
    const int H = prm.H;
    int seg_base = b * prm.nseg;                     // index of the sequence's first segment
    int64_t rec_base = (int64_t)b * H * (prm.Lpad / ST);   // tile record of head 0, tile 0: + h * rec_hstride
    int rec_hstride = prm.Lpad / ST;
    if (packed) {
        const int2 it = prm.items[blockIdx.x];
        b = it.x; seg = it.y;
        const SeqDesc sd = prm.seqs[b];
        L = sd.len; tok0 = sd.tok0; bco = 0;
        seg_base = sd.seg0;
        nseg = prm.seqs[b + 1].seg0 - sd.seg0;
        rec_base = sd.tile0;
        rec_hstride = prm.ntile_total;
    }
    const int HG = H / prm.G, ppg = pairs_per_group(H, prm.G);
    const int g = blockIdx.y / ppg, pr = blockIdx.y % ppg;
    const int head0 = g * HG + pr * NHD;
    const int nh = min(NHD, HG - pr * NHD);          // heads this CTA really has
    const int t_begin = seg * prm.seg_len;
    const int t_end = head_part ? min(L, prm.split_tiles * ST) : min(L, t_begin + prm.seg_len);
    const int ntiles = (t_end - t_begin + ST - 1) / ST;
    const bool kfull = prm.mode == MODE_FULL;
    // leading tiles that only carry the state forward (tile j is a full tile iff kfull && j >= n_pre;
    // barriers that only full tiles use count their phases in full tiles, jf = j - n_pre)
    const int n_pre = split ? (head_part ? 0 : min(prm.split_tiles, ntiles)) : 0;

    if (tid == 0) {
        tc::mbar_init(&bars->cb_full, 1);
        tc::mbar_init(&bars->cb_empty, 1);
        tc::mbar_init(&bars->g_full, 1);
        tc::mbar_init(&bars->g_free, HEAD_THREADS * nh);
        for (int hd = 0; hd < NHD; ++hd) {
            HeadBars *hb = &bars->hd[hd];
            for (int s = 0; s < 2; ++s) {
                tc::mbar_init(&hb->x_full[s], 1);
                tc::mbar_init(&hb->x_free[s], HEAD_THREADS + 1);
            }
            tc::mbar_init(&hb->yoff_full, 1);
            tc::mbar_init(&hb->m_full, HEAD_THREADS);
            tc::mbar_init(&hb->yd_full, 1);
            tc::mbar_init(&hb->xp_full, HEAD_THREADS);
            tc::mbar_init(&hb->dh_full, 1);
            tc::mbar_init(&hb->h_ready, HEAD_THREADS);
            tc::mbar_init(&hb->y_free, HEAD_THREADS);
            tc::mbar_init(&hb->y_staged, HEAD_THREADS);
            tc::mbar_init(&hb->sc_full, 1);
        }
        *abort_flag = 0;
        tc::fence_mbar_init();
    }
    if (warp == WARP_MMA0) {
        tc::tmem_alloc(&sm->tmem_slot, TM_COLS);
        tc::tmem_relinquish();
    }
    if (warp == WARP_TMA && lane == 0) {
        tc::prefetch_tmap(&tmap_bc);
        tc::prefetch_tmap(&tmap_x);
        tc::prefetch_tmap(&tmap_y);
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = sm->tmem_slot;
    // Everything above needs nothing from earlier kernels and may run under their tail; the
    // mixed streams and the step sizes are read from here on.
    grid_dep_launch();
    grid_dep_wait();

    // Warp index as a value the compiler knows to be warp-uniform.
    const int uwarp = __shfl_sync(0xffffffffu, warp, 0);
    if (uwarp == WARP_TMA) {
        // ------------------------------------------------------------------ TMA producer
        // (the whole warp runs the loop; one elected lane issues the copies)
        const bool leader = tc::elect_one();
        // record of tile t_begin / ST + j of head head0 + hd
        auto scal_rec = [&](int hd, int j) {
            return prm.rec + rec_base + (int64_t)(head0 + hd) * rec_hstride + t_begin / ST + j;
        };
        if (leader && ntiles > 0) {
            for (int hd = 0; hd < nh; ++hd) {               // X and scalars of tile 0
                HeadBars *hb = &bars->hd[hd];
                tc::mbar_arrive_expect_tx(&hb->x_full[0], SLAB);
                tc::tma_load_4d(smem + SM_HEAD + hd * SM_HEAD_BYTES, &tmap_x, &hb->x_full[0], 0,
                                head0 + hd, tok0 + t_begin, bco);
                tc::mbar_arrive_expect_tx(&hb->sc_full, (uint32_t)sizeof(TileScalars));
                tc::bulk_load(&sm->sc[hd], scal_rec(hd, 0), (uint32_t)sizeof(TileScalars), &hb->sc_full);
            }
        }
        for (int j = 0; j < ntiles; ++j) {
            const int t0 = tok0 + t_begin + j * ST;
            const bool full = SPLIT ? (kfull && j >= n_pre) : kfull;
            tc::mbar_wait(&bars->cb_empty, (j & 1) ^ 1, abort_flag, d_status);
            if (leader) {
                tc::mbar_arrive_expect_tx(&bars->cb_full, full ? 4 * SLAB : 2 * SLAB);
                if (full) {
                    tc::tma_load_3d(smem + SM_CB + 0 * SLAB, &tmap_bc, &bars->cb_full, (prm.G + g) * SN, t0, bco);
                    tc::tma_load_3d(smem + SM_CB + 1 * SLAB, &tmap_bc, &bars->cb_full, (prm.G + g) * SN + 64, t0, bco);
                }
                tc::tma_load_3d(smem + SM_CB + 2 * SLAB, &tmap_bc, &bars->cb_full, g * SN, t0, bco);
                tc::tma_load_3d(smem + SM_CB + 3 * SLAB, &tmap_bc, &bars->cb_full, g * SN + 64, t0, bco);
            }
            if (j + 1 < ntiles) {                            // X one tile ahead
                const int jn = j + 1, sx = jn & 1;
                for (int hd = 0; hd < nh; ++hd) {
                    HeadBars *hb = &bars->hd[hd];
                    tc::mbar_wait(&hb->x_free[sx], ((jn >> 1) & 1) ^ 1, abort_flag, d_status);
                    if (leader) {
                        tc::mbar_arrive_expect_tx(&hb->x_full[sx], SLAB);
                        tc::tma_load_4d(smem + SM_HEAD + hd * SM_HEAD_BYTES + sx * SLAB, &tmap_x,
                                        &hb->x_full[sx], 0, head0 + hd, t0 + ST, bco);
                    }
                }
                // scalars of the next tile: the record buffer is single; its last readers are the
                // mask (full pass) or the w.X scaling (state-only pass) of this tile
                for (int hd = 0; hd < nh; ++hd) {
                    HeadBars *hb = &bars->hd[hd];
                    if (full) tc::mbar_wait(&hb->m_full, (SPLIT ? j - n_pre : j) & 1, abort_flag, d_status);
                    else tc::mbar_wait(&hb->xp_full, j & 1, abort_flag, d_status);
                    if (leader) {
                        tc::mbar_arrive_expect_tx(&hb->sc_full, (uint32_t)sizeof(TileScalars));
                        tc::bulk_load(&sm->sc[hd], scal_rec(hd, jn), (uint32_t)sizeof(TileScalars), &hb->sc_full);
                    }
                }
            }
            __syncwarp();
        }
    } else if (uwarp >= WARP_MMA0) {
        // ------------------------------------------------------------------ MMA issuers
        // The whole warp runs the loop and the waits; one elected lane issues the MMAs, the
        // commits and the y stores.
        const int hd = uwarp - WARP_MMA0;
        const bool leader = tc::elect_one();
        if (hd < nh) {
            // The products against the shared Ctilde / Btilde tiles (MMA 1, 3, 4) are issued by the
            // first issuer for both heads at once: with N = 128 the shared operand is read from
            // shared memory once instead of once per head.  MMA 2 and the y store stay per head.
            constexpr uint32_t id_g = tc::idesc_bf16(128, 128, 0, 0);     // C (K-major) x B (K-major)
            constexpr uint32_t id_y = tc::idesc_bf16(128, 64, 0, 1);      // K-major / TMEM A, MN-major B
            const uint32_t id_yn = nh == 2 ? tc::idesc_bf16(128, 128, 0, 1) : id_y;
            const uint32_t id_hn = nh == 2 ? tc::idesc_bf16(128, 128, 1, 1) : tc::idesc_bf16(128, 64, 1, 1);
            HeadBars *hb = &bars->hd[hd];
            const uint32_t c_addr = tc::smem_u32(smem + SM_CB), b_addr = c_addr + 2 * SLAB;
            const uint32_t head0_addr = tc::smem_u32(smem + SM_HEAD);
            const uint32_t head_addr = head0_addr + hd * SM_HEAD_BYTES;
            const uint8_t *s_y = smem + SM_HEAD + hd * SM_HEAD_BYTES + 4 * SLAB;
            const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem, 0);
            const uint32_t tm = tmem_u + TM_HEAD + hd * TM_HEAD_COLS;
            // descriptors of the first K step; later steps advance the address field
            const uint64_t dC = tc::smem_desc_sw128(c_addr, 16, 1024);          // K-major
            const uint64_t dB = tc::smem_desc_sw128(b_addr, 16, 1024);          // K-major
            const uint64_t dBt = tc::smem_desc_sw128(b_addr, SLAB, 1024);       // MN-major
            // MN-major operands over both heads: the second head's 64 columns lie one head region on
            const uint64_t dH = tc::smem_desc_sw128(head0_addr + 3 * SLAB, SM_HEAD_BYTES, 1024);
            const uint64_t dXp = tc::smem_desc_sw128(head0_addr + 2 * SLAB, SM_HEAD_BYTES, 1024);
            const uint64_t dX0 = tc::smem_desc_sw128(head_addr, SLAB, 1024);    // MN-major
            // MMA 1 of tile jj: G = Ctilde Btilde^T (K = state index), shared by both heads
            auto issue_g = [&](int jj) {
                tc::mbar_wait(&bars->cb_full, jj & 1, abort_flag, d_status);
                const int jjf = SPLIT ? jj - n_pre : jj;
                if (jjf > 0) tc::mbar_wait(&bars->g_free, (jjf - 1) & 1, abort_flag, d_status);
                tc::tc_fence_after();
                if (leader) {
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        const uint32_t off = (kk >> 2) * SLAB + (kk & 3) * 32;
                        tc::mma_ss(tmem_u + TM_G, tc::smem_desc_advance(dC, off),
                                   tc::smem_desc_advance(dB, off), id_g, kk > 0);
                    }
                    tc::mma_commit(&bars->g_full);
                }
                __syncwarp();
            };
            for (int j = 0; j < ntiles; ++j) {
                const int sx = j & 1;
                const bool full = SPLIT ? (kfull && j >= n_pre) : kfull;
                const int jf = SPLIT ? j - n_pre : j;
                if (hd == 0) {
                    tc::mbar_wait(&bars->cb_full, j & 1, abort_flag, d_status);
                    tc::tc_fence_after();
                    if (full) {
                        // MMA 3: Y = Ctilde Hprev^T  (K = state index; B = bf16 states, rows = n)
                        for (int q = 0; q < nh; ++q) {
                            tc::mbar_wait(&bars->hd[q].h_ready, jf & 1, abort_flag, d_status);
                            if (jf > 0) tc::mbar_wait(&bars->hd[q].y_free, (jf - 1) & 1, abort_flag, d_status);
                        }
                        tc::tc_fence_after();
                        if (leader) {
#pragma unroll
                            for (int kk = 0; kk < 8; ++kk) {
                                const uint32_t off = (kk >> 2) * SLAB + (kk & 3) * 32;
                                tc::mma_ss(tmem_u + TM_Y, tc::smem_desc_advance(dC, off),
                                           tc::smem_desc_advance(dH, kk * 2048), id_yn, kk > 0);
                            }
                            for (int q = 0; q < nh; ++q) tc::mma_commit(&bars->hd[q].yoff_full);
                        }
                        __syncwarp();
                        // MMA 1 of this tile goes behind MMA 3 in the tensor pipe: the product with
                        // the carried state is needed first (it is scaled before the mask is built)
                        issue_g(j);
                    }
                    // MMA 4: dH^T[n,p] = sum_s Btilde[s,n] (w_s x_s[p])   (K = token)
                    for (int q = 0; q < nh; ++q)
                        tc::mbar_wait(&bars->hd[q].xp_full, j & 1, abort_flag, d_status);
                    tc::tc_fence_after();
                    if (leader) {
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk)     // (the tiles of a state-only run accumulate)
                            tc::mma_ss(tmem_u + TM_DH, tc::smem_desc_advance(dBt, kk * 2048),
                                       tc::smem_desc_advance(dXp, kk * 2048), id_hn, (kk > 0) || (!full && j > 0));
                        for (int q = 0; q < nh; ++q) tc::mma_commit(&bars->hd[q].dh_full);
                        tc::mma_commit(&bars->cb_empty);     // C and B tiles are no longer needed
                    }
                    __syncwarp();
                }
                if (full) {
                    // MMA 2: Y += M X  (A = masked tile in TMEM, 8 columns per 16 tokens of K)
                    tc::mbar_wait(&hb->m_full, jf & 1, abort_flag, d_status);
                    tc::tc_fence_after();
                    const uint64_t dX = tc::smem_desc_advance(dX0, sx * SLAB);
                    if (leader) {
                        tc::bulk_wait_read_all();        // previous y tile has left its staging buffer
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk)
                            tc::mma_ts(tm + TM_Y, tm + TM_M + kk * 8, tc::smem_desc_advance(dX, kk * 2048),
                                       id_y, 1);
                        tc::mma_commit(&hb->yd_full);
                    }
                }
                // (state-only pass: the second issuer has no product of its own; it follows the
                // tile loop at the pace of its head's w.X scaling, whose end frees the X slot)
                if (!full && hd > 0) tc::mbar_wait(&hb->xp_full, j & 1, abort_flag, d_status);
                if (leader) tc::mma_commit(&hb->x_free[sx]);
                __syncwarp();
                if (full) {
                    // the staged y tile goes out as one TMA store (rows past the end of the
                    // sequence are clipped by the tensor map)
                    // (packed batch: a tile that runs past the end of its sequence is stored row by row
                    // by the compute warps, the rows behind it belong to the next sequence)
                    tc::mbar_wait(&hb->y_staged, jf & 1, abort_flag, d_status);
                    if (leader && !(packed && t_begin + (j + 1) * ST > L)) {
                        tc::tma_store_4d(&tmap_y, s_y, 0, head0 + hd, tok0 + t_begin + j * ST, bco);
                        tc::bulk_commit_group();
                    }
                    __syncwarp();
                }
            }
            if (kfull && leader) tc::bulk_wait_read_all();
        }
    } else if ((uwarp >> 3) < nh) {
        // ------------------------------------------------------------------ compute warps
        const int hd = warp >> 3, hf = (warp >> 2) & 1, wq = warp & 3;
        const int h = head0 + hd;
        const int i = wq * 32 + lane;                        // token row in the tile == state index n
        const int p0 = 32 * hf;                              // this thread's half of the head dim
        HeadBars *hb = &bars->hd[hd];
        uint8_t *s_head = smem + SM_HEAD + hd * SM_HEAD_BYTES;
        uint8_t *s_xp = s_head + 2 * SLAB, *s_hb = s_head + 3 * SLAB, *s_y = s_head + 4 * SLAB;
        const uint32_t *s_wp = sm->sc[hd].wp;
        const float *s_cb = sm->sc[hd].cb, *s_ends = sm->sc[hd].ends;
        const uint32_t lane_base = (uint32_t)(wq * 32) << 16;
        const uint32_t tm = tmem + TM_HEAD + hd * TM_HEAD_COLS + lane_base;
        const float Dh = prm.D ? prm.D[h] : 0.f;
        // fp32 master copy of the state: this thread holds H[n = i][p = p0 .. p0+31]
        float Hst[32];
        {
            const float *h_in = prm.h_in;
            if (h_in && kfull) {
                const int64_t base = prm.seg_states
                    ? ((((int64_t)seg_base + seg) * H + h) * SP) * SN
                    : (((int64_t)b * H + h) * SP) * SN;
#pragma unroll
                for (int q = 0; q < 32; ++q) Hst[q] = h_in[base + (int64_t)(p0 + q) * SN + i];
            } else {
#pragma unroll
                for (int q = 0; q < 32; ++q) Hst[q] = 0.f;
            }
            if (kfull && n_pre == 0) {
                // bf16 copy of the state the first tile starts from
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint4 v = make_uint4(tc::pack_bf16x2(Hst[8 * ch + 0], Hst[8 * ch + 1]),
                                         tc::pack_bf16x2(Hst[8 * ch + 2], Hst[8 * ch + 3]),
                                         tc::pack_bf16x2(Hst[8 * ch + 4], Hst[8 * ch + 5]),
                                         tc::pack_bf16x2(Hst[8 * ch + 6], Hst[8 * ch + 7]));
                    *reinterpret_cast<uint4 *>(s_hb + tc::sw128_offset(i, 4 * hf + ch)) = v;
                }
                tc::fence_proxy_async_smem();
                tc::mbar_arrive(&hb->h_ready);
            }
            if (kfull) {
                // blocks of M above the diagonal stay zero for the whole kernel
                uint32_t zero[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) zero[q] = 0u;
                for (int c = wq + 1; c < 4; ++c) tc::tmem_st8(tm + TM_M + c * 16 + 8 * hf, zero);
                tc::tmem_st_wait();
            }
        }
        float seg_l2 = 0.f;      // log2 of the product of a_t over the tiles done so far
        const int64_t rec_row = rec_base + (int64_t)h * rec_hstride;     // tile 0 of this (sequence, head)
        const float *l2p = prm.l2 + rec_row * ST + t_begin;
        float l2_next = ntiles > 0 ? l2p[i] : 0.f;
        // A run of state-only tiles (a whole segment in the state-only pass, the lead of a split
        // launch) is one long contraction: with every token weighted by its decay up to the END OF
        // THE RUN (exponent <= 0), Btilde^T (w . X) accumulates over all tiles of the run in tensor
        // memory and the state is touched once, at the run's last tile:
        //   H_end = 2^(sum of l_last over the run) H_in + sum_tiles Btilde^T (w' . X).
        const int run_end = kfull ? n_pre : ntiles;
        float run_total = 0.f;   // log2 decay over the whole run
        {
            const TileScalars *rec0 = prm.rec + rec_row + t_begin / ST;
            for (int jr = 0; jr < run_end; ++jr) run_total += rec0[jr].ends[3];
        }
        float run_done = 0.f;    // ... over the tiles of the run up to and including the current one

        for (int j = 0; j < ntiles; ++j) {
            const int sx = j & 1;
            const bool full = SPLIT ? (kfull && j >= n_pre) : kfull;
            const bool hb_next = SPLIT ? (kfull && j + 1 >= n_pre) : kfull;   // the next tile reads the bf16 state copy
            const int jf = SPLIT ? j - n_pre : j;
            const uint8_t *s_x = s_head + sx * SLAB;
            // ---- per-token scalars: this row's cumulative log2 decay inside the tile (prefetched);
            // the weights of all rows and the block ends arrive in shared memory
            const float l2 = l2_next;
            if (j + 1 < ntiles) l2_next = l2p[(j + 1) * ST + i];
            tc::mbar_wait(&hb->sc_full, j & 1, abort_flag, d_status);
            const float4 ends = *reinterpret_cast<const float4 *>(s_ends);
            const float L1 = ends.x, L2 = ends.y, L3 = ends.z, l2_last = ends.w;
            const float Lw = wq == 0 ? 0.f : (wq == 1 ? L1 : (wq == 2 ? L2 : L3));    // l before my block
            const float Lend = wq == 0 ? L1 : (wq == 1 ? L2 : (wq == 2 ? L3 : l2_last));  // l at its end

            // ---- w . X  (rows of the X slab -> rows of the X' slab, this thread's half of the
            // head dim).  The decay mask below costs row block wq about wq + 1 units of work, so in
            // the full pass the 16 (row block, 16-byte chunk) units of a lane are dealt 6 / 5 / 3 / 2
            // to row blocks 0 .. 3 instead of 4 each; a foreign row's weight is read from shared
            // memory.
            tc::mbar_wait(&hb->x_full[sx], (j >> 1) & 1, abort_flag, d_status);
            if (full) {
                if (wq == 0) scale_units<0, 6>(s_x, s_xp, s_wp, lane, hf);
                else if (wq == 1) scale_units<6, 11>(s_x, s_xp, s_wp, lane, hf);
                else if (wq == 2) scale_units<11, 14>(s_x, s_xp, s_wp, lane, hf);
                else scale_units<14, 16>(s_x, s_xp, s_wp, lane, hf);
            } else {
                // a tile of a run: the X' slab is free once the previous tile's product has read it
                run_done += l2_last;
                const uint32_t wp = s_wp[i];
                if (j > 0) tc::mbar_wait(&hb->dh_full, (j - 1) & 1, abort_flag, d_status);
                scale_own_row(s_x, s_xp, wp, tc::ex2_approx(run_total - run_done), i, hf);
            }
            tc::fence_proxy_async_smem();
            tc::mbar_arrive(&hb->xp_full);

            if (full) {
                // ---- Y = exp(l_i) * (Ctilde Hprev^T), in place
                tc::mbar_wait(&hb->yoff_full, jf & 1, abort_flag, d_status);
                tc::tc_fence_after();
                {
                    const float e_i = tc::ex2_approx(l2);
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        uint32_t yo[16];
                        tc::tmem_ld16(tm + TM_Y + p0 + 16 * hh, yo);
                        tc::tmem_ld_wait();
#pragma unroll
                        for (int q = 0; q < 16; ++q) yo[q] = __float_as_uint(e_i * __uint_as_float(yo[q]));
                        tc::tmem_st16(tm + TM_Y + p0 + 16 * hh, yo);
                    }
                }
                // ---- decay mask: G (fp32, TMEM) -> M (bf16, TMEM); this thread owns row i and
                // columns 16 hf .. 16 hf + 15 of every 32-column block
                tc::mbar_wait(&bars->g_full, jf & 1, abort_flag, d_status);
                tc::tc_fence_after();
                const float r_i = tc::ex2_approx(l2 - Lw);
                const uint32_t g_addr = tmem + lane_base + TM_G + 16 * hf;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    if (c <= wq) {
                        uint32_t cur[16], pk[8];
                        tc::tmem_ld16(g_addr + c * 32, cur);
                        tc::tmem_ld_wait();
                        if (c == wq) {
                            // diagonal block: Delta_j 2^(l_i - l_j) = cb_j 2^(l_i - l_blockend).  The
                            // second factor is >= 1; when the whole block decays by less than
                            // 2^-96 it cannot overflow and is applied as a product, else the
                            // exponent is formed per entry (always <= 0 where j <= i).
                            const float up = l2 - Lend;
                            if (Lw - Lend < 96.f) {
                                const float rf = tc::ex2_approx(up);
#pragma unroll
                                for (int q = 0; q < 8; ++q) {
                                    const float2 cb = *reinterpret_cast<const float2 *>(&s_cb[c * 32 + 16 * hf + 2 * q]);
                                    float m0 = __uint_as_float(cur[2 * q]) * cb.x * rf;
                                    float m1 = __uint_as_float(cur[2 * q + 1]) * cb.y * rf;
                                    if (16 * hf + 2 * q > lane) m0 = 0.f;
                                    if (16 * hf + 2 * q + 1 > lane) m1 = 0.f;
                                    pk[q] = tc::pack_bf16x2(m0, m1);
                                }
                            } else {
#pragma unroll
                                for (int q = 0; q < 8; ++q) {
                                    const float2 cb = *reinterpret_cast<const float2 *>(&s_cb[c * 32 + 16 * hf + 2 * q]);
                                    float m0 = __uint_as_float(cur[2 * q]) * tc::ex2_approx(up + tc::lg2_approx(cb.x));
                                    float m1 = __uint_as_float(cur[2 * q + 1]) * tc::ex2_approx(up + tc::lg2_approx(cb.y));
                                    if (16 * hf + 2 * q > lane) m0 = 0.f;
                                    if (16 * hf + 2 * q + 1 > lane) m1 = 0.f;
                                    pk[q] = tc::pack_bf16x2(m0, m1);
                                }
                            }
                        } else {
                            // l at the end of column block c, relative to the start of my block
                            const float Lc1 = c == 0 ? L1 : (c == 1 ? L2 : L3);
                            const float rowf = r_i * tc::ex2_approx(Lw - Lc1);
#pragma unroll
                            for (int q = 0; q < 8; ++q) {
                                const float2 cb = *reinterpret_cast<const float2 *>(&s_cb[c * 32 + 16 * hf + 2 * q]);
                                pk[q] = tc::pack_bf16x2(__uint_as_float(cur[2 * q]) * cb.x * rowf,
                                                        __uint_as_float(cur[2 * q + 1]) * cb.y * rowf);
                            }
                        }
                        tc::tmem_st8(tm + TM_M + c * 16 + 8 * hf, pk);
                    }
                }
                tc::tmem_st_wait();
                tc::tc_fence_before();
                tc::mbar_arrive(&bars->g_free);
                // (the scalars record read above is refilled by a bulk copy once m_full completes)
                tc::fence_proxy_async_smem();
                tc::mbar_arrive(&hb->m_full);
            }

            // ---- state: H = exp(l_last) H + dH  (thread owns state index n = i, 32 channels); inside a
            // run of state-only tiles only at its last tile, with the decay of the whole run
            seg_l2 += l2_last;
            if (full || j == run_end - 1) {
            tc::mbar_wait(&hb->dh_full, j & 1, abort_flag, d_status);
            tc::tc_fence_after();
            const float dec = tc::ex2_approx(full ? l2_last : run_total);
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                uint32_t dh[16];
                tc::tmem_ld16(tm + TM_DH + p0 + 16 * hh, dh);
                tc::tmem_ld_wait();
#pragma unroll
                for (int q = 0; q < 16; ++q)
                    Hst[16 * hh + q] = fmaf(dec, Hst[16 * hh + q], __uint_as_float(dh[q]));
                if (hb_next) {
#pragma unroll
                    for (int c2 = 0; c2 < 2; ++c2) {
                        const int ch = 2 * hh + c2;
                        uint4 v = make_uint4(tc::pack_bf16x2(Hst[8 * ch + 0], Hst[8 * ch + 1]),
                                             tc::pack_bf16x2(Hst[8 * ch + 2], Hst[8 * ch + 3]),
                                             tc::pack_bf16x2(Hst[8 * ch + 4], Hst[8 * ch + 5]),
                                             tc::pack_bf16x2(Hst[8 * ch + 6], Hst[8 * ch + 7]));
                        *reinterpret_cast<uint4 *>(s_hb + tc::sw128_offset(i, 4 * hf + ch)) = v;
                    }
                }
            }
            if (hb_next) {
                tc::fence_proxy_async_smem();
                tc::tc_fence_before();
                tc::mbar_arrive(&hb->h_ready);
            }
            }
            if (full) {
                // ---- epilogue: y_i = Y_i + D x_i, staged in shared memory for the TMA store
                tc::mbar_wait(&hb->yd_full, jf & 1, abort_flag, d_status);
                tc::tc_fence_after();
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    uint32_t yd[16];
                    tc::tmem_ld16(tm + TM_Y + p0 + 16 * hh, yd);
                    tc::tmem_ld_wait();
#pragma unroll
                    for (int c2 = 0; c2 < 2; ++c2) {
                        const uint32_t off = tc::sw128_offset(i, 4 * hf + 2 * hh + c2);
                        const uint4 xr = *reinterpret_cast<const uint4 *>(s_x + off);
                        const uint32_t xw[4] = {xr.x, xr.y, xr.z, xr.w};
                        uint32_t o[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const int e0 = c2 * 8 + 2 * q;
                            const float x0 = __uint_as_float(xw[q] << 16);
                            const float x1 = __uint_as_float(xw[q] & 0xffff0000u);
                            o[q] = tc::pack_bf16x2(fmaf(Dh, x0, __uint_as_float(yd[e0])),
                                                   fmaf(Dh, x1, __uint_as_float(yd[e0 + 1])));
                        }
                        *reinterpret_cast<uint4 *>(s_y + off) = make_uint4(o[0], o[1], o[2], o[3]);
                        if (packed && t_begin + (j + 1) * ST > L && t_begin + j * ST + i < L) {
                            __nv_bfloat16 *yrow = reinterpret_cast<__nv_bfloat16 *>(prm.y) +
                                ((int64_t)(tok0 + t_begin + j * ST + i) * H + h) * SP;
                            *reinterpret_cast<uint4 *>(yrow + p0 + 16 * hh + 8 * c2) = make_uint4(o[0], o[1], o[2], o[3]);
                        }
                    }
                }
                tc::tc_fence_before();
                tc::mbar_arrive(&hb->y_free);
                tc::fence_proxy_async_smem();
                tc::mbar_arrive(&hb->y_staged);
            } else {
                tc::tc_fence_before();
            }
            tc::mbar_arrive(&hb->x_free[sx]);
        }

        // ---- final state of the segment
        if (kfull) {
            if (prm.h_out && seg == nseg - 1 && !head_part) {
                float *dst = prm.h_out + (((int64_t)b * H + h) * SP) * SN;
#pragma unroll
                for (int q = 0; q < 32; ++q) dst[(int64_t)(p0 + q) * SN + i] = Hst[q];
            }
        } else {
            float *dst = prm.h_out + ((((int64_t)seg_base + seg) * H + h) * SP) * SN;
#pragma unroll
            for (int q = 0; q < 32; ++q) dst[(int64_t)(p0 + q) * SN + i] = Hst[q];
            if (i == 0 && hf == 0) prm.seg_decay[((int64_t)seg_base + seg) * H + h] = tc::ex2_approx(seg_l2);
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == WARP_MMA0) tc::tmem_dealloc(tmem, TM_COLS);
}

// K3: chain the segments.  states[b,s,h,:,:] holds segment s's local end state (computed from a
// zero initial state) on entry and the state ENTERING segment s on exit:
//   H_in(0) = h0,   H_in(s+1) = decay(s) H_in(s) + S(s).
// One thread per 4 consecutive state entries; segments are walked in order.
// (packed batch: sequence b owns segments seqs[b].seg0 .. seqs[b+1].seg0 - 1 of the batch-wide list)
__global__ void __launch_bounds__(256)
segment_scan_kernel(float *__restrict__ states, const float *__restrict__ seg_decay,
                    const float *__restrict__ h0, int nseg, int H, int PN4, const SeqDesc *__restrict__ seqs,
                    float *__restrict__ end_state, float *__restrict__ end_decay)
{
    const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;   // float4 index inside [P*N/4]
    const int h = blockIdx.y, b = blockIdx.z;
    if (v >= PN4) return;
    int64_t sb = (int64_t)b * nseg;
    if (seqs) {
        sb = seqs[b].seg0;
        nseg = seqs[b + 1].seg0 - seqs[b].seg0;
    }
    float4 run = h0 ? reinterpret_cast<const float4 *>(h0)[((int64_t)b * H + h) * PN4 + v]
                    : make_float4(0.f, 0.f, 0.f, 0.f);
    float dtot = 1.f;
    // Local end states exist for all segments but a sequence's last one, unless the caller wants the
    // state after the last segment (a sequence shard's summary): that one was computed too.
    const int nlocal = (end_state || end_decay) ? nseg : nseg - 1;
    // the loads do not depend on the running state: four segments are fetched at a time
    constexpr int U = 4;
    for (int s0 = 0; s0 < nseg; s0 += U) {
        float4 loc[U];
        float d[U];
#pragma unroll
        for (int q = 0; q < U; ++q) {
            const int s = s0 + q;
            if (s < nlocal) {
                loc[q] = reinterpret_cast<const float4 *>(states)[((sb + s) * H + h) * PN4 + v];
                d[q] = seg_decay[(sb + s) * H + h];
            }
        }
#pragma unroll
        for (int q = 0; q < U; ++q) {
            const int s = s0 + q;
            if (s < nseg) {
                reinterpret_cast<float4 *>(states)[((sb + s) * H + h) * PN4 + v] = run;
                if (s >= nlocal) continue;
                run.x = fmaf(d[q], run.x, loc[q].x);
                run.y = fmaf(d[q], run.y, loc[q].y);
                run.z = fmaf(d[q], run.z, loc[q].z);
                run.w = fmaf(d[q], run.w, loc[q].w);
                dtot *= d[q];
            }
        }
    }
    // (dense batches only) the state after the last segment and the decay over all of them
    if (end_state) reinterpret_cast<float4 *>(end_state)[((int64_t)b * H + h) * PN4 + v] = run;
    if (end_decay && v == 0) end_decay[(int64_t)b * H + h] = dtot;
}

// Sequence-sharded evaluation, second half.  Rank r of R holds tokens [r L, (r+1) L) of every
// sequence; all ranks' summaries (end state from a zero entry state, decay over the shard) have been
// gathered: gs [R, B, H, P*N], gd [R, B, H].  The state entering this rank's shard is
//   H_in = scan over ranks r' < rank of  H <- gd[r'] H + gs[r'],  from h0,
// and the states entering its local segments, computed from a zero entry state by the local scan,
// gain the entry state decayed up to the segment's start: states[b,s] += (prod_{s'<s} decay[b,s']) H_in.
__global__ void __launch_bounds__(256)
shard_entry_kernel(float *__restrict__ states, const float *__restrict__ seg_decay, const float *__restrict__ h0,
                   const float *__restrict__ gs, const float *__restrict__ gd, int rank, int B, int nseg, int H,
                   int PN4)
{
    const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int h = blockIdx.y, b = blockIdx.z;
    if (v >= PN4) return;
    float4 run = h0 ? reinterpret_cast<const float4 *>(h0)[((int64_t)b * H + h) * PN4 + v]
                    : make_float4(0.f, 0.f, 0.f, 0.f);
    for (int r = 0; r < rank; ++r) {
        const float d = gd[((int64_t)r * B + b) * H + h];
        const float4 loc = reinterpret_cast<const float4 *>(gs)[(((int64_t)r * B + b) * H + h) * PN4 + v];
        run.x = fmaf(d, run.x, loc.x);
        run.y = fmaf(d, run.y, loc.y);
        run.z = fmaf(d, run.z, loc.z);
        run.w = fmaf(d, run.w, loc.w);
    }
    float cum = 1.f;
    for (int sgi = 0; sgi < nseg; ++sgi) {
        float4 *p = reinterpret_cast<float4 *>(states) + (((int64_t)b * nseg + sgi) * H + h) * PN4 + v;
        float4 cur = *p;
        cur.x = fmaf(cum, run.x, cur.x);
        cur.y = fmaf(cum, run.y, cur.y);
        cur.z = fmaf(cum, run.z, cur.z);
        cur.w = fmaf(cum, run.w, cur.w);
        *p = cur;
        cum *= seg_decay[((int64_t)b * nseg + sgi) * H + h];
    }
}

// ---------------------------------------------------------------------------------------------
// State-only pass on its own: the local end state of a segment from a zero entry state,
//   H_end^T[n,p] = sum_s Btilde_s[n] (w'_s x_s[p]),   w'_s = Delta_s 2^(l(end of segment) - l(s)),
// one long contraction over the segment's tokens accumulated in tensor memory (see the run
// accumulation in ssd_tiles_kernel).  Nothing but Btilde, x and the tile records is read, so one
// CTA takes FOUR heads of a group (the Btilde tile is fetched once for all of them: half the
// shared-operand traffic of a head pair) and the tiles flow through a two-stage ring in which the
// x slabs are scaled IN PLACE: TMA fills a stage, 16 warps (one token row of one head per thread)
// scale, one thread issues a single 128 x 256 x 128 product per tile, its completion frees the
// stage.  The state is read from tensor memory once, at the end.
namespace {
constexpr int NQ = 4;                                   // heads per CTA
constexpr int ST_STAGES = 4;
constexpr int HT = 64;                                  // tokens per ring stage: half a tile
constexpr uint32_t HSLAB = SLAB / 2;                    // 64 rows x 128 bytes
constexpr uint32_t ST_STAGE_BYTES = (2 + NQ) * HSLAB;   // B0 B1 X0 X1 X2 X3
constexpr uint32_t ST_SMALL = ST_STAGES * ST_STAGE_BYTES;
constexpr int ST_THREADS = 32 * (4 * NQ + 2);
constexpr uint32_t ST_TM_COLS = NQ * 64 < 32 ? 32 : NQ * 64;

struct __align__(16) StateSmall {
    TileScalars sc[ST_STAGES][NQ];
    uint64_t full[ST_STAGES], scaled[ST_STAGES], empty[ST_STAGES], done;
    uint32_t tmem_slot;
    int abort_flag;
};

__host__ __device__ inline int quads_per_group(int H, int G) { return (H / G + NQ - 1) / NQ; }
}  // namespace

__global__ void __launch_bounds__(ST_THREADS, 1)
ssd_state_kernel(const __grid_constant__ CUtensorMap tmap_bc, const __grid_constant__ CUtensorMap tmap_x,
                 const SsdParams prm)
{
    extern __shared__ __align__(1024) uint8_t smem[];
    StateSmall *sm = (StateSmall *)(smem + ST_SMALL);
    int *abort_flag = &sm->abort_flag;
    int *d_status = prm.d_status;
    if ((tc::smem_u32(smem) & 1023u) != 0) {
        if (threadIdx.x == 0) atomicCAS(d_status, 0, SWIMBA_ERR_DEVICE_BOUNDS);
        return;
    }
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool packed = prm.seqs != nullptr;
    int seg = blockIdx.x, b = blockIdx.z;
    int L = prm.L, tok0 = 0, bco = b;
    const int H = prm.H;
    int seg_base = b * prm.nseg;
    int64_t rec_base = (int64_t)b * H * (prm.Lpad / ST);
    int rec_hstride = prm.Lpad / ST;
    if (packed) {
        const int2 it = prm.items[blockIdx.x];
        b = it.x; seg = it.y;
        const SeqDesc sd = prm.seqs[b];
        L = sd.len; tok0 = sd.tok0; bco = 0;
        seg_base = sd.seg0;
        rec_base = sd.tile0;
        rec_hstride = prm.ntile_total;
    }
    const int HG = H / prm.G, qpg = quads_per_group(H, prm.G);
    const int g = blockIdx.y / qpg, qd = blockIdx.y % qpg;
    const int head0 = g * HG + qd * NQ;
    const int nh = min(NQ, HG - qd * NQ);
    const int t_begin = seg * prm.seg_len;
    const int t_end = min(L, t_begin + prm.seg_len);
    const int ntiles = (t_end - t_begin + ST - 1) / ST;
    const int nhalves = (t_end - t_begin + HT - 1) / HT;     // ring stages: half tiles that hold tokens

    if (tid == 0) {
        for (int s = 0; s < ST_STAGES; ++s) {
            tc::mbar_init(&sm->full[s], 1);
            tc::mbar_init(&sm->scaled[s], 128 * nh);
            tc::mbar_init(&sm->empty[s], 1);
        }
        tc::mbar_init(&sm->done, 1);
        *abort_flag = 0;
        tc::fence_mbar_init();
    }
    if (warp == 4 * NQ + 1) {
        tc::tmem_alloc(&sm->tmem_slot, ST_TM_COLS);
        tc::tmem_relinquish();
    }
    if (warp == 4 * NQ && lane == 0) {
        tc::prefetch_tmap(&tmap_bc);
        tc::prefetch_tmap(&tmap_x);
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = sm->tmem_slot;
    grid_dep_launch();
    grid_dep_wait();

    const int uwarp = __shfl_sync(0xffffffffu, warp, 0);
    if (uwarp == 4 * NQ) {
        // ------------------------------------------------------------------ TMA producer
        const bool leader = tc::elect_one();
        for (int q = 0; q < nhalves; ++q) {
            const int s = q % ST_STAGES, ph = (q / ST_STAGES) & 1;
            tc::mbar_wait(&sm->empty[s], ph ^ 1, abort_flag, d_status);
            if (leader) {
                uint8_t *stg = smem + s * ST_STAGE_BYTES;
                const int t0 = tok0 + t_begin + q * HT;
                tc::mbar_arrive_expect_tx(&sm->full[s], (2 + nh) * HSLAB + nh * (uint32_t)sizeof(TileScalars));
                tc::tma_load_3d(stg, &tmap_bc, &sm->full[s], g * SN, t0, bco);
                tc::tma_load_3d(stg + HSLAB, &tmap_bc, &sm->full[s], g * SN + 64, t0, bco);
                for (int hd = 0; hd < nh; ++hd) {
                    tc::tma_load_4d(stg + (2 + hd) * HSLAB, &tmap_x, &sm->full[s], 0, head0 + hd, t0, bco);
                    tc::bulk_load(&sm->sc[s][hd],
                                  prm.rec + rec_base + (int64_t)(head0 + hd) * rec_hstride + t_begin / ST + (q >> 1),
                                  (uint32_t)sizeof(TileScalars), &sm->full[s]);
                }
            }
            __syncwarp();
        }
    } else if (uwarp == 4 * NQ + 1) {
        // ------------------------------------------------------------------ MMA issuer
        const bool leader = tc::elect_one();
        const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem, 0);
        const uint32_t id_h = tc::idesc_bf16(128, 64 * nh, 1, 1);        // both operands MN-major
        for (int q = 0; q < nhalves; ++q) {
            const int s = q % ST_STAGES, ph = (q / ST_STAGES) & 1;
            tc::mbar_wait(&sm->scaled[s], ph, abort_flag, d_status);
            tc::tc_fence_after();
            if (leader) {
                const uint32_t base = tc::smem_u32(smem + s * ST_STAGE_BYTES);
                const uint64_t dBt = tc::smem_desc_sw128(base, HSLAB, 1024);
                const uint64_t dXp = tc::smem_desc_sw128(base + 2 * HSLAB, HSLAB, 1024);
#pragma unroll
                for (int kk = 0; kk < HT / 16; ++kk)
                    tc::mma_ss(tmem_u, tc::smem_desc_advance(dBt, kk * 2048), tc::smem_desc_advance(dXp, kk * 2048),
                               id_h, (q > 0) || (kk > 0));
                tc::mma_commit(&sm->empty[s]);
                if (q == nhalves - 1) tc::mma_commit(&sm->done);
            }
            __syncwarp();
        }
    } else if ((uwarp >> 2) < nh) {
        // ------------------------------------------------------------------ compute warps
        const int hd = warp >> 2, wq = warp & 3;
        const int h = head0 + hd;
        const int i = wq * 32 + lane;                    // token row in the tile == state index n
        const int64_t rec_row = rec_base + (int64_t)h * rec_hstride + t_begin / ST;
        float run_total = 0.f;                            // log2 decay over the whole segment
        for (int jr = 0; jr < ntiles; ++jr) run_total += prm.rec[rec_row + jr].ends[3];
        float run_done = 0.f;
        // within a stage: this thread's token row and its half of the row's eight 16-byte chunks
        const int srow = i >> 1, shalf = i & 1;
        for (int q = 0; q < nhalves; ++q) {
            const int s = q % ST_STAGES, ph = (q / ST_STAGES) & 1;
            tc::mbar_wait(&sm->full[s], ph, abort_flag, d_status);
            const TileScalars *sc = &sm->sc[s][hd];
            if ((q & 1) == 0) run_done += sc->ends[3];                 // (both halves of a tile share its record)
            const uint32_t wp = sc->wp[(q & 1) * HT + srow];
            const float w = (__uint_as_float(wp << 16) + __uint_as_float(wp & 0xffff0000u)) *
                            tc::ex2_approx(run_total - run_done);
            const __nv_bfloat16 w_hi = __float2bfloat16_rn(w);
            const __nv_bfloat16 w_lo = __float2bfloat16_rn(w - __bfloat162float(w_hi));
            const __nv_bfloat162 w_hi2 = __halves2bfloat162(w_hi, w_hi), w_lo2 = __halves2bfloat162(w_lo, w_lo);
            uint8_t *s_x = smem + s * ST_STAGE_BYTES + (2 + hd) * HSLAB;
            uint4 xr[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) xr[c] = *reinterpret_cast<const uint4 *>(s_x + tc::sw128_offset(srow, 4 * shalf + c));
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t wv[4] = {xr[c].x, xr[c].y, xr[c].z, xr[c].w};
                uint32_t o[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const __nv_bfloat162 xv = *reinterpret_cast<const __nv_bfloat162 *>(&wv[e]);
                    const __nv_bfloat162 pr = __hfma2(w_hi2, xv, __hmul2(w_lo2, xv));
                    o[e] = *reinterpret_cast<const uint32_t *>(&pr);
                }
                *reinterpret_cast<uint4 *>(s_x + tc::sw128_offset(srow, 4 * shalf + c)) = make_uint4(o[0], o[1], o[2], o[3]);
            }
            tc::fence_proxy_async_smem();
            tc::mbar_arrive(&sm->scaled[s]);
        }
        // ---- the segment's end state (entry state zero) and its total decay
        float *dst = prm.h_out + ((((int64_t)seg_base + seg) * H + h) * SP) * SN;
        if (ntiles > 0) {
            tc::mbar_wait(&sm->done, 0, abort_flag, d_status);
            tc::tc_fence_after();
            const uint32_t tm = tmem + ((uint32_t)(wq * 32) << 16) + 64 * hd;
#pragma unroll
            for (int hh = 0; hh < 4; ++hh) {
                uint32_t dh[16];
                tc::tmem_ld16(tm + 16 * hh, dh);
                tc::tmem_ld_wait();
#pragma unroll
                for (int q = 0; q < 16; ++q) dst[(int64_t)(16 * hh + q) * SN + i] = __uint_as_float(dh[q]);
            }
        } else {
#pragma unroll 8
            for (int q = 0; q < SP; ++q) dst[(int64_t)q * SN + i] = 0.f;
        }
        if (i == 0) prm.seg_decay[((int64_t)seg_base + seg) * H + h] = tc::ex2_approx(run_total);
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 4 * NQ + 1) tc::tmem_dealloc(tmem, ST_TM_COLS);
}

static size_t ssd_state_smem_bytes() { return ST_SMALL + sizeof(StateSmall); }

// The state-only launch behind both the dense and the packed segment passes.
static int launch_state_pass(LaunchCtx &ctx, const void *x, const void *BC, int64_t rows, int nb, const SsdParams &p,
                             unsigned grid_x, int H, int G, unsigned grid_z)
{
    // tensor maps with boxes of half a tile (64 tokens) over x [nb, rows, H, P] and BC [nb, rows, S]
    CUtensorMap tm_bc, tm_x;
    {
        const int S = 2 * G * SN;
        const uint64_t dims3[3] = {(uint64_t)S, (uint64_t)rows, (uint64_t)nb};
        const uint64_t str3[2] = {(uint64_t)S * 2, (uint64_t)rows * S * 2};
        const uint32_t box3[3] = {64, (uint32_t)HT, 1};
        const uint64_t dims4[4] = {(uint64_t)SP, (uint64_t)H, (uint64_t)rows, (uint64_t)nb};
        const uint64_t str4[3] = {(uint64_t)SP * 2, (uint64_t)H * SP * 2, (uint64_t)rows * H * SP * 2};
        const uint32_t box4[4] = {SP, 1, (uint32_t)HT, 1};
        if (!encode_tmap_bf16_cached(ctx.tmaps, &tm_bc, BC, 3, dims3, str3, box3) ||
            !encode_tmap_bf16_cached(ctx.tmaps, &tm_x, x, 4, dims4, str4, box4))
            return SWIMBA_ERR_CUDA;
    }
    const size_t smem = ssd_state_smem_bytes();
    if (!ensure_dynamic_smem((const void *)ssd_state_kernel, smem)) return SWIMBA_ERR_CUDA;
    ctx.begin(STAGE_SSD_STATE);
    launch_kernel(ssd_state_kernel, dim3(grid_x, (unsigned)(G * quads_per_group(H, G)), grid_z), dim3(ST_THREADS), smem,
                  ctx.stream, true, tm_bc, tm_x, p);
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

bool ssd_tiles_supported(int dtype, int P, int N)
{
    return dtype == SWIMBA_DTYPE_BF16 && P == SP && N == SN;
}

static size_t ssd_smem_bytes() { return SM_SMALL + sizeof(SsdSmall); }

// Segment length (tokens, multiple of 128) so that the grid fills the SMs; L itself if one
// segment per sequence is enough.
int ssd_segment_len(int B, int L, int H, int G, int chunk, int sm_count)
{
    const int64_t ctas = (int64_t)B * G * pairs_per_group(H, G);
    const int tiles = ceil_div(L, ST);
    if (2 * ctas > sm_count || tiles <= 2) return tiles * ST;
    // segments per sequence: as many as keep the grid within two CTAs per SM (a few CTAs more
    // would cost a whole extra round)
    int want = (int)((2 * (int64_t)sm_count) / ctas);
    if (want < 1) want = 1;
    int q_tiles = chunk >= ST ? chunk / ST : 1;                       // segments are whole chunks
    int seg_tiles = ceil_div(tiles, want);
    seg_tiles = ceil_div(seg_tiles, q_tiles) * q_tiles;
    if (seg_tiles < 4) seg_tiles = 4 < tiles ? 4 : tiles;
    return seg_tiles * ST;
}

// Workspace: [log-decays B*H*Lpad float] [per-tile records B*H*(Lpad/128)] [segment states]
// [segment decays].
static size_t ssd_scalars_bytes(int B, int L, int H)
{
    const size_t Lpad = (size_t)ceil_div(L, ST) * ST;
    const size_t l2_bytes = ((size_t)B * H * Lpad * sizeof(float) + 255) / 256 * 256;
    const size_t rec_bytes = ((size_t)B * H * (Lpad / ST) * sizeof(TileScalars) + 255) / 256 * 256;
    return l2_bytes + rec_bytes;
}

size_t ssd_workspace_bytes(int B, int L, int H, int G, int chunk, int sm_count)
{
    const int seg_len = ssd_segment_len(B, L, H, G, chunk, sm_count);
    const int nseg = ceil_div(L, seg_len);
    size_t tot = ssd_scalars_bytes(B, L, H);
    if (nseg > 1)
        tot += (size_t)B * nseg * H * SP * SN * sizeof(float) + ((size_t)B * nseg * H * sizeof(float) + 255) / 256 * 256;
    return tot;
}

ScalarsArgs ssd_scalars_args(const float *dt, const float *A, const float *dt_bias, int B, int L, int H,
                             void *workspace)
{
    ScalarsArgs a;
    a.dt = dt; a.A = A; a.dt_bias = dt_bias; a.l2 = (float *)workspace;
    a.rec = (TileScalars *)((char *)workspace +
                            ((size_t)B * H * (ceil_div(L, ST) * ST) * sizeof(float) + 255) / 256 * 256);
    a.L = L; a.Lpad = ceil_div(L, ST) * ST; a.H = H; a.B = B;
    return a;
}

// Split of a one-segment launch (see ssd_tiles_kernel): 0 when one CTA per (sequence, head pair)
// already fills the GPU (or the segmented path applies), else the number of leading tiles a.  The
// CTAs that walk the whole sequence (started first, one per SM) cost (n - a) full tiles plus a
// state-only tiles at about 0.47 of a full one; the CTAs that produce y of the leading tiles run
// on the SMs left over, in ceil(ctas / spare) rounds of a tiles.  a minimises the later of the two.
static int ssd_split_tiles(int B, int L, int H, int G, int sm_count)
{
    const int64_t ctas = (int64_t)B * G * pairs_per_group(H, G);
    const int n = ceil_div(L, ST);
    if (2 * ctas <= sm_count || ctas >= sm_count || n < 4) return 0;
    const int64_t spare = sm_count - ctas, rounds = ceil_div64(ctas, spare);
    float best = (float)n;
    int best_a = 0;
    for (int a = 1; a < n; ++a) {
        const float whole = (float)n - 0.53f * a, lead = (float)(rounds * a);
        const float m = whole > lead ? whole : lead;
        if (m < best) { best = m; best_a = a; }
    }
    return best < 0.95f * n ? best_a : 0;
}

int launch_ssd_scalars(LaunchCtx &ctx, const ScalarsArgs &sa)
{
    if (scalars_units(sa) <= 0) return SWIMBA_OK;
    ctx.begin(STAGE_SSD_SCALARS);
    launch_kernel(ssd_scalars_kernel, dim3((unsigned)scalars_blocks(sa, 256)), dim3(256), 0, ctx.stream,
                  true, sa);
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

int launch_ssd_tiles(LaunchCtx &ctx, const void *x, const void *BC, const float *dt, const float *A,
                     const float *dt_bias, const float *D, const float *h0, int B, int L, int H, int G,
                     int chunk, int sm_count, void *y, float *h_final, void *workspace,
                     bool scalars_done)
{
    if (B <= 0 || L <= 0) return SWIMBA_OK;
    const int S = 2 * G * SN;
    CUtensorMap tm_bc, tm_x, tm_y;
    {
        const uint64_t dims[3] = {(uint64_t)S, (uint64_t)L, (uint64_t)B};
        const uint64_t str[2] = {(uint64_t)S * 2, (uint64_t)L * S * 2};
        const uint32_t box[3] = {64, ST, 1};
        if (!encode_tmap_bf16_cached(ctx.tmaps, &tm_bc, BC, 3, dims, str, box)) return SWIMBA_ERR_CUDA;
    }
    {
        const uint64_t dims[4] = {(uint64_t)SP, (uint64_t)H, (uint64_t)L, (uint64_t)B};
        const uint64_t str[3] = {(uint64_t)SP * 2, (uint64_t)H * SP * 2, (uint64_t)L * H * SP * 2};
        const uint32_t box[4] = {SP, 1, ST, 1};
        if (!encode_tmap_bf16_cached(ctx.tmaps, &tm_x, x, 4, dims, str, box)) return SWIMBA_ERR_CUDA;
        if (!encode_tmap_bf16_cached(ctx.tmaps, &tm_y, y, 4, dims, str, box)) return SWIMBA_ERR_CUDA;
    }
    const size_t smem = ssd_smem_bytes();
    if (!ensure_dynamic_smem((const void *)ssd_tiles_kernel<false>, smem) ||
        !ensure_dynamic_smem((const void *)ssd_tiles_kernel<true>, smem))
        return SWIMBA_ERR_CUDA;

    const int seg_len = ssd_segment_len(B, L, H, G, chunk, sm_count);
    const int nseg = ceil_div(L, seg_len);
    const int Lpad = ceil_div(L, ST) * ST;
    char *seg_ws = (char *)workspace + ssd_scalars_bytes(B, L, H);
    if (!scalars_done) {
        const int rc = launch_ssd_scalars(ctx, ssd_scalars_args(dt, A, dt_bias, B, L, H, workspace));
        if (rc != SWIMBA_OK) return rc;
    }
    SsdParams p;
    {
        const ScalarsArgs sa = ssd_scalars_args(nullptr, nullptr, nullptr, B, L, H, workspace);
        p.l2 = sa.l2;
        p.rec = sa.rec;
    }
    p.D = D;
    p.L = L; p.Lpad = Lpad; p.H = H; p.G = G; p.nseg = nseg; p.seg_len = seg_len;
    p.d_status = ctx.d_status;
    p.seqs = nullptr; p.items = nullptr; p.ntile_total = 0; p.seg_states = nseg > 1; p.y = y;
    dim3 grid((unsigned)nseg, (unsigned)(G * pairs_per_group(H, G)), (unsigned)B);
    p.split_tiles = 0;
    if (nseg == 1) {
        p.h_in = h0; p.h_out = h_final; p.seg_decay = nullptr; p.mode = MODE_FULL;
        p.split_tiles = ssd_split_tiles(B, L, H, G, sm_count);
        if (p.split_tiles > 0) grid = dim3((unsigned)B, (unsigned)(G * pairs_per_group(H, G)), 2u);
        ctx.begin(STAGE_SSD_TILES);
        if (p.split_tiles > 0)
            launch_kernel(ssd_tiles_kernel<true>, grid, dim3(SSD_THREADS), smem, ctx.stream, true, tm_bc, tm_x, tm_y, p);
        else
            launch_kernel(ssd_tiles_kernel<false>, grid, dim3(SSD_THREADS), smem, ctx.stream, true, tm_bc, tm_x, tm_y, p);
        ctx.end();
    } else {
        float *states = (float *)seg_ws;
        float *decay = states + (size_t)B * nseg * H * SP * SN;
        p.h_in = nullptr; p.h_out = states; p.seg_decay = decay; p.mode = MODE_STATE_ONLY;
        {
            // (the last segment's end state is nobody's entry state: the full pass produces it)
            const int rc = launch_state_pass(ctx, x, BC, L, B, p, (unsigned)(nseg - 1), H, G, (unsigned)B);
            if (rc != SWIMBA_OK) return rc;
        }
        const int PN4 = SP * SN / 4;
        ctx.begin(STAGE_SEGMENT_SCAN);
        segment_scan_kernel<<<dim3((unsigned)ceil_div(PN4, 256), (unsigned)H, (unsigned)B), 256, 0, ctx.stream>>>(
            states, decay, h0, nseg, H, PN4, nullptr, nullptr, nullptr);
        ctx.end();
        p.h_in = states; p.h_out = h_final; p.seg_decay = nullptr; p.mode = MODE_FULL;
        ctx.begin(STAGE_SSD_TILES);
        launch_kernel(ssd_tiles_kernel<false>, grid, dim3(SSD_THREADS), smem, ctx.stream, true, tm_bc, tm_x, tm_y, p);
        ctx.end();
    }
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// Packed batches: nseq sequences of different lengths back to back in [T, ...] arrays, sequence b
// holding tokens cu[b] .. cu[b+1]-1.  Tiles start at sequence starts.  A sequence longer than the
// segment length is cut into segments (state-only pass, segment scan, full pass, as in the dense
// case); the segment length is the per-SM share of the batch's tiles, so that one long sequence
// among short ones does not serialise the launch.
namespace {
struct PackedPlan {
    std::vector<SeqDesc> seqs;        // nseq + 1
    std::vector<int2> tiles;          // (first token, valid tokens) per tile
    std::vector<int2> items, pre;     // (sequence, segment): all of them / those whose end state the scan needs
    std::vector<int4> shorts;         // (first token, tokens, sequence, 0) of the sequences stepped token by token
    int total_tiles = 0, total_segs = 0, seg_len = 0;
    bool segmented = false;
};

PackedPlan packed_plan(const int32_t *cu, int nseq, int H, int G, int chunk, int sm_count)
{
    PackedPlan pl;
    // Sequences of a few tokens (decode tokens riding in a prefill batch) do not take a 128-token
    // tile and a CTA per head pair each: they are stepped token by token, one block per head.
    constexpr int SHORT_MAX = 4;
    auto is_short = [&](int b) { const int len = cu[b + 1] - cu[b]; return len >= 1 && len <= SHORT_MAX; };
    int64_t tiles = 0;
    for (int b = 0; b < nseq; ++b)
        if (!is_short(b)) tiles += ceil_div(cu[b + 1] - cu[b], ST);
    const int64_t pairs = (int64_t)G * pairs_per_group(H, G);
    const int q_tiles = chunk >= ST ? chunk / ST : 1;
    int64_t seg_tiles = ceil_div64(tiles * pairs, sm_count);
    if (seg_tiles < 4) seg_tiles = 4;
    seg_tiles = ceil_div64(seg_tiles, q_tiles) * q_tiles;
    if (seg_tiles > (1 << 22)) seg_tiles = 1 << 22;
    pl.seg_len = (int)seg_tiles * ST;
    pl.seqs.resize((size_t)nseq + 1);
    int tile0 = 0, seg0 = 0;
    for (int b = 0; b < nseq; ++b) {
        const int len = cu[b + 1] - cu[b];
        if (is_short(b)) {
            pl.seqs[b] = SeqDesc{cu[b], len, tile0, seg0};
            pl.shorts.push_back(make_int4(cu[b], len, b, 0));
            seg0 += 1;                                   // (keeps one segment slot, unused)
            continue;
        }
        const int nt = ceil_div(len, ST);
        const int ns = len > 0 ? ceil_div(len, pl.seg_len) : 1;
        pl.seqs[b] = SeqDesc{cu[b], len, tile0, seg0};
        for (int t = 0; t < nt; ++t)
            pl.tiles.push_back(make_int2(cu[b] + t * ST, len - t * ST < ST ? len - t * ST : ST));
        for (int sgi = 0; sgi < ns; ++sgi) {
            pl.items.push_back(make_int2(b, sgi));
            if (sgi + 1 < ns) pl.pre.push_back(make_int2(b, sgi));
        }
        if (ns > 1) pl.segmented = true;
        tile0 += nt;
        seg0 += ns;
    }
    pl.seqs[nseq] = SeqDesc{cu[nseq], 0, tile0, seg0};
    pl.total_tiles = tile0;
    pl.total_segs = seg0;
    return pl;
}

struct PackedLayout {
    size_t seqs, tiles, items, pre, shorts, l2, rec, states, decay, total;
};
PackedLayout packed_layout(const PackedPlan &pl, int nseq, int H)
{
    auto up = [](size_t v) { return (v + 255) / 256 * 256; };
    PackedLayout l;
    size_t off = 0;
    l.seqs = off;  off += up(((size_t)nseq + 1) * sizeof(SeqDesc));
    l.tiles = off; off += up((size_t)pl.total_tiles * sizeof(int2));
    l.items = off; off += up(pl.items.size() * sizeof(int2));
    l.pre = off;   off += up(pl.pre.size() * sizeof(int2));
    l.shorts = off; off += up(pl.shorts.size() * sizeof(int4));
    l.l2 = off;    off += up((size_t)H * pl.total_tiles * ST * sizeof(float));
    l.rec = off;   off += up((size_t)H * pl.total_tiles * sizeof(TileScalars));
    l.states = off;
    if (pl.segmented) off += up((size_t)pl.total_segs * H * SP * SN * sizeof(float));
    l.decay = off;
    if (pl.segmented) off += up((size_t)pl.total_segs * H * sizeof(float));
    l.total = off;
    return l;
}
}  // namespace

size_t ssd_packed_workspace_bytes(const int32_t *cu, int nseq, int H, int G, int chunk, int sm_count)
{
    const PackedPlan pl = packed_plan(cu, nseq, H, G, chunk, sm_count);
    return packed_layout(pl, nseq, H).total;
}

int ssd_packed_segments(const int32_t *cu, int nseq, int H, int G, int chunk, int sm_count)
{
    return packed_plan(cu, nseq, H, G, chunk, sm_count).total_segs;
}

int launch_ssd_tiles_packed(LaunchCtx &ctx, const void *x, const void *BC, const float *dt, const float *A,
                            const float *dt_bias, const float *D, const float *h0, const int32_t *cu, int nseq,
                            int H, int G, int chunk, int sm_count, void *y, float *h_final, void *workspace)
{
    const int64_t T = cu[nseq];
    if (nseq <= 0 || T <= 0) return SWIMBA_OK;
    const PackedPlan pl = packed_plan(cu, nseq, H, G, chunk, sm_count);
    const PackedLayout lay = packed_layout(pl, nseq, H);
    char *ws = (char *)workspace;
    // the tables go to the device in stream order (the copies read host memory before returning)
    if (cudaMemcpyAsync(ws + lay.seqs, pl.seqs.data(), pl.seqs.size() * sizeof(SeqDesc), cudaMemcpyHostToDevice, ctx.stream) != cudaSuccess ||
        cudaMemcpyAsync(ws + lay.tiles, pl.tiles.data(), pl.tiles.size() * sizeof(int2), cudaMemcpyHostToDevice, ctx.stream) != cudaSuccess ||
        cudaMemcpyAsync(ws + lay.items, pl.items.data(), pl.items.size() * sizeof(int2), cudaMemcpyHostToDevice, ctx.stream) != cudaSuccess ||
        (!pl.pre.empty() &&
         cudaMemcpyAsync(ws + lay.pre, pl.pre.data(), pl.pre.size() * sizeof(int2), cudaMemcpyHostToDevice, ctx.stream) != cudaSuccess) ||
        (!pl.shorts.empty() &&
         cudaMemcpyAsync(ws + lay.shorts, pl.shorts.data(), pl.shorts.size() * sizeof(int4), cudaMemcpyHostToDevice, ctx.stream) != cudaSuccess))
        return SWIMBA_ERR_CUDA;
    if (!pl.shorts.empty()) {
        const int rc = launch_ssd_sequential_listed(ctx, x, BC, dt, A, dt_bias, D, h0, (const int4 *)(ws + lay.shorts),
                                                    (int)pl.shorts.size(), H, SP, SN, G, y, h_final);
        if (rc != SWIMBA_OK) return rc;
    }
    if (pl.items.empty()) return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;

    const int S = 2 * G * SN;
    CUtensorMap tm_bc, tm_x, tm_y;
    {
        const uint64_t dims[3] = {(uint64_t)S, (uint64_t)T, 1};
        const uint64_t str[2] = {(uint64_t)S * 2, (uint64_t)T * S * 2};
        const uint32_t box[3] = {64, ST, 1};
        if (!encode_tmap_bf16_cached(ctx.tmaps, &tm_bc, BC, 3, dims, str, box)) return SWIMBA_ERR_CUDA;
    }
    {
        const uint64_t dims[4] = {(uint64_t)SP, (uint64_t)H, (uint64_t)T, 1};
        const uint64_t str[3] = {(uint64_t)SP * 2, (uint64_t)H * SP * 2, (uint64_t)T * H * SP * 2};
        const uint32_t box[4] = {SP, 1, ST, 1};
        if (!encode_tmap_bf16_cached(ctx.tmaps, &tm_x, x, 4, dims, str, box)) return SWIMBA_ERR_CUDA;
        if (!encode_tmap_bf16_cached(ctx.tmaps, &tm_y, y, 4, dims, str, box)) return SWIMBA_ERR_CUDA;
    }
    const size_t smem = ssd_smem_bytes();
    if (!ensure_dynamic_smem((const void *)ssd_tiles_kernel<false>, smem)) return SWIMBA_ERR_CUDA;

    ScalarsArgs sa;
    sa.dt = dt; sa.A = A; sa.dt_bias = dt_bias;
    sa.l2 = (float *)(ws + lay.l2);
    sa.rec = (TileScalars *)(ws + lay.rec);
    sa.L = (int)T; sa.Lpad = pl.total_tiles * ST; sa.H = H; sa.B = 1;
    sa.tile_tab = (const int2 *)(ws + lay.tiles);
    int rc = launch_ssd_scalars(ctx, sa);
    if (rc != SWIMBA_OK) return rc;

    SsdParams p;
    p.l2 = sa.l2; p.rec = sa.rec; p.D = D;
    p.L = 0; p.Lpad = sa.Lpad; p.H = H; p.G = G; p.nseg = 1; p.seg_len = pl.seg_len;
    p.split_tiles = 0;
    p.d_status = ctx.d_status;
    p.seqs = (const SeqDesc *)(ws + lay.seqs);
    p.ntile_total = pl.total_tiles;
    p.y = y;
    const unsigned pairs = (unsigned)(G * pairs_per_group(H, G));
    if (!pl.segmented) {
        p.items = (const int2 *)(ws + lay.items);
        p.h_in = h0; p.h_out = h_final; p.seg_decay = nullptr; p.mode = MODE_FULL; p.seg_states = 0;
        ctx.begin(STAGE_SSD_TILES);
        launch_kernel(ssd_tiles_kernel<false>, dim3((unsigned)pl.items.size(), pairs, 1), dim3(SSD_THREADS), smem,
                      ctx.stream, true, tm_bc, tm_x, tm_y, p);
        ctx.end();
    } else {
        float *states = (float *)(ws + lay.states);
        float *decay = (float *)(ws + lay.decay);
        p.items = (const int2 *)(ws + lay.pre);
        p.h_in = nullptr; p.h_out = states; p.seg_decay = decay; p.mode = MODE_STATE_ONLY; p.seg_states = 1;
        rc = launch_state_pass(ctx, x, BC, T, 1, p, (unsigned)pl.pre.size(), H, G, 1u);
        if (rc != SWIMBA_OK) return rc;
        const int PN4 = SP * SN / 4;
        ctx.begin(STAGE_SEGMENT_SCAN);
        segment_scan_kernel<<<dim3((unsigned)ceil_div(PN4, 256), (unsigned)H, (unsigned)nseq), 256, 0, ctx.stream>>>(
            states, decay, h0, 0, H, PN4, p.seqs, nullptr, nullptr);
        ctx.end();
        p.items = (const int2 *)(ws + lay.items);
        p.h_in = states; p.h_out = h_final; p.seg_decay = nullptr; p.mode = MODE_FULL;
        ctx.begin(STAGE_SSD_TILES);
        launch_kernel(ssd_tiles_kernel<false>, dim3((unsigned)pl.items.size(), pairs, 1), dim3(SSD_THREADS), smem,
                      ctx.stream, true, tm_bc, tm_x, tm_y, p);
        ctx.end();
    }
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// Sequence-sharded evaluation: every rank holds L consecutive tokens of each of the B sequences.
// First half (summary): state-only pass over the shard's segments and the local scan from a zero
// entry state; leaves the shard's end state and total decay for the exchange, and the zero-entry
// segment states in the workspace.  Second half (finish), after the ranks' summaries have been
// gathered: entry state from the ranks in front, segment states corrected, full pass.
namespace {
struct ShardLayout {
    size_t scal, states, decay, total;
    int seg_len, nseg;
};
ShardLayout shard_layout(int B, int L, int H, int G, int chunk, int sm_count)
{
    ShardLayout l;
    l.seg_len = ssd_segment_len(B, L, H, G, chunk, sm_count);
    l.nseg = ceil_div(L, l.seg_len);
    size_t off = 0;
    l.scal = off;   off += ssd_scalars_bytes(B, L, H);
    l.states = off; off += ((size_t)B * l.nseg * H * SP * SN * sizeof(float) + 255) / 256 * 256;
    l.decay = off;  off += ((size_t)B * l.nseg * H * sizeof(float) + 255) / 256 * 256;
    l.total = off;
    return l;
}

bool shard_maps(LaunchCtx &ctx, const void *x, const void *BC, const void *y, int B, int L, int H, int G,
                CUtensorMap *tm_bc, CUtensorMap *tm_x, CUtensorMap *tm_y)
{
    const int S = 2 * G * SN;
    const uint64_t dims3[3] = {(uint64_t)S, (uint64_t)L, (uint64_t)B};
    const uint64_t str3[2] = {(uint64_t)S * 2, (uint64_t)L * S * 2};
    const uint32_t box3[3] = {64, ST, 1};
    if (!encode_tmap_bf16_cached(ctx.tmaps, tm_bc, BC, 3, dims3, str3, box3)) return false;
    const uint64_t dims[4] = {(uint64_t)SP, (uint64_t)H, (uint64_t)L, (uint64_t)B};
    const uint64_t str[3] = {(uint64_t)SP * 2, (uint64_t)H * SP * 2, (uint64_t)L * H * SP * 2};
    const uint32_t box[4] = {SP, 1, ST, 1};
    if (!encode_tmap_bf16_cached(ctx.tmaps, tm_x, x, 4, dims, str, box)) return false;
    // (the state-only pass stores no y; its map is a copy of x's)
    if (!encode_tmap_bf16_cached(ctx.tmaps, tm_y, y ? y : x, 4, dims, str, box)) return false;
    return ensure_dynamic_smem((const void *)ssd_tiles_kernel<false>, ssd_smem_bytes());
}

SsdParams shard_params(LaunchCtx &ctx, const ShardLayout &lay, int B, int L, int H, int G, void *workspace)
{
    SsdParams p;
    const ScalarsArgs sa = ssd_scalars_args(nullptr, nullptr, nullptr, B, L, H, (char *)workspace + lay.scal);
    p.l2 = sa.l2; p.rec = sa.rec;
    p.D = nullptr;
    p.L = L; p.Lpad = ceil_div(L, ST) * ST; p.H = H; p.G = G; p.nseg = lay.nseg; p.seg_len = lay.seg_len;
    p.split_tiles = 0;
    p.d_status = ctx.d_status;
    p.seqs = nullptr; p.items = nullptr; p.ntile_total = 0; p.seg_states = 1; p.y = nullptr;
    return p;
}
}  // namespace

size_t ssd_shard_workspace_bytes(int B, int L, int H, int G, int chunk, int sm_count)
{
    return shard_layout(B, L, H, G, chunk, sm_count).total;
}

ScalarsArgs ssd_shard_scalars_args(const float *dt, const float *A, const float *dt_bias, int B, int L, int H,
                                   int G, int chunk, int sm_count, void *workspace)
{
    const ShardLayout lay = shard_layout(B, L, H, G, chunk, sm_count);
    return ssd_scalars_args(dt, A, dt_bias, B, L, H, (char *)workspace + lay.scal);
}

int launch_ssd_shard_summary(LaunchCtx &ctx, const void *x, const void *BC, const float *dt, const float *A,
                             const float *dt_bias, int B, int L, int H, int G, int chunk, int sm_count,
                             float *sum_state, float *sum_decay, void *workspace, bool scalars_done)
{
    if (B <= 0 || L <= 0) return SWIMBA_OK;
    const ShardLayout lay = shard_layout(B, L, H, G, chunk, sm_count);
    CUtensorMap tm_bc, tm_x, tm_y;
    if (!shard_maps(ctx, x, BC, nullptr, B, L, H, G, &tm_bc, &tm_x, &tm_y)) return SWIMBA_ERR_CUDA;
    if (!scalars_done) {
        const int rc = launch_ssd_scalars(ctx, ssd_scalars_args(dt, A, dt_bias, B, L, H, (char *)workspace + lay.scal));
        if (rc != SWIMBA_OK) return rc;
    }
    SsdParams p = shard_params(ctx, lay, B, L, H, G, workspace);
    float *states = (float *)((char *)workspace + lay.states);
    float *decay = (float *)((char *)workspace + lay.decay);
    p.h_in = nullptr; p.h_out = states; p.seg_decay = decay; p.mode = MODE_STATE_ONLY;
    {
        const int rc = launch_state_pass(ctx, x, BC, L, B, p, (unsigned)lay.nseg, H, G, (unsigned)B);
        if (rc != SWIMBA_OK) return rc;
    }
    const int PN4 = SP * SN / 4;
    ctx.begin(STAGE_SEGMENT_SCAN);
    segment_scan_kernel<<<dim3((unsigned)ceil_div(PN4, 256), (unsigned)H, (unsigned)B), 256, 0, ctx.stream>>>(
        states, decay, nullptr, lay.nseg, H, PN4, nullptr, sum_state, sum_decay);
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

int launch_ssd_shard_finish(LaunchCtx &ctx, const void *x, const void *BC, const float *D, const float *h0,
                            const float *all_state, const float *all_decay, int rank, int B, int L, int H, int G,
                            int chunk, int sm_count, void *y, float *h_end, void *workspace)
{
    if (B <= 0 || L <= 0) return SWIMBA_OK;
    const ShardLayout lay = shard_layout(B, L, H, G, chunk, sm_count);
    CUtensorMap tm_bc, tm_x, tm_y;
    if (!shard_maps(ctx, x, BC, y, B, L, H, G, &tm_bc, &tm_x, &tm_y)) return SWIMBA_ERR_CUDA;
    SsdParams p = shard_params(ctx, lay, B, L, H, G, workspace);
    float *states = (float *)((char *)workspace + lay.states);
    float *decay = (float *)((char *)workspace + lay.decay);
    const int PN4 = SP * SN / 4;
    ctx.begin(STAGE_SEGMENT_SCAN);
    shard_entry_kernel<<<dim3((unsigned)ceil_div(PN4, 256), (unsigned)H, (unsigned)B), 256, 0, ctx.stream>>>(
        states, decay, h0, all_state, all_decay, rank, B, lay.nseg, H, PN4);
    ctx.end();
    p.D = D; p.y = y;
    p.h_in = states; p.h_out = h_end; p.seg_decay = nullptr; p.mode = MODE_FULL;
    const dim3 grid((unsigned)lay.nseg, (unsigned)(G * pairs_per_group(H, G)), (unsigned)B);
    ctx.begin(STAGE_SSD_TILES);
    launch_kernel(ssd_tiles_kernel<false>, grid, dim3(SSD_THREADS), ssd_smem_bytes(), ctx.stream, true, tm_bc, tm_x,
                  tm_y, p);
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

}  // namespace swimba
