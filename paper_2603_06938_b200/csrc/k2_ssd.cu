// K2/K3: chunked SSD evaluation of the single selective SSM on tcgen05 tensor cores
// (Background, "Mamba-2 and SSD": matrix products inside chunks, a linear recurrence between
// chunks; the recurrence itself is Theorem 1's h_t = a_t h_{t-1} + Delta_t Btilde_t x_t^T,
// y_t = Ctilde_t^T h_t + D x_t).
//
// One CTA owns one (sequence, head, segment) and walks its segment in tiles of 128 tokens.  With
// l_i = sum_{r<=i} Delta_r A (inside the tile), for every tile:
//   G      = Ctilde Btilde^T                                  [128 x 128]   (MMA 1)
//   M[i,s] = G[i,s] exp(l_i - l_s) Delta_s  for s <= i, else 0               (CUDA cores -> TMEM)
//   Ydiag  = M X                                              [128 x 64]    (MMA 2, A from TMEM)
//   Yoff   = Ctilde H_prev^T                                  [128 x 64]    (MMA 3)
//   y_i    = Ydiag_i + exp(l_i) Yoff_i + D x_i
//   dH^T   = Btilde^T (w . X),  w_s = exp(l_last - l_s) Delta_s   [128 x 64] (MMA 4)
//   H      = exp(l_last) H_prev + dH                                         (fp32, registers)
// The carried state never leaves the SM inside a segment: the inter-chunk recurrence is fused.
// Long sequences with few (sequence, head) pairs are cut into segments: a first pass of this
// kernel computes every segment's local end state (MMA 4 only), segment_scan_kernel (K3) chains
// them, and a second pass evaluates each segment from its true incoming state.
#include "internal.h"
#include "tc05.cuh"

namespace swimba {

namespace {
constexpr int ST = 128;                 // tokens per tile
constexpr int SP = 64;                  // head dim this kernel is built for
constexpr int SN = 128;                 // state size this kernel is built for
constexpr int SSD_THREADS = 192;        // warps 0-3 compute, warp 4 TMA, warp 5 MMA
constexpr int SSD_STAGES = 2;
constexpr uint32_t SLAB = 16384;        // 128 rows x 128 bytes
constexpr uint32_t STAGE_BYTES = 5 * SLAB;   // C (2 slabs), B (2 slabs), X (1 slab)
constexpr float LOG2E = 1.4426950408889634f;

// TMEM columns
constexpr uint32_t TM_G = 0, TM_M = 128, TM_YD = 192, TM_YOFF = 256, TM_DH = 320, TM_COLS = 512;

enum { MODE_FULL = 0, MODE_STATE_ONLY = 1 };

struct SsdParams {
    const float *dt;        // [B,L,H] or null
    const float *A, *dt_bias, *D;
    const float *h_in;      // initial states: [B,H,P,N] (nseg == 1) or [B,nseg,H,P,N]; may be null
    __nv_bfloat16 *y;       // [B,L,H,P]
    float *h_out;           // MODE_FULL: h_final [B,H,P,N] (last segment writes) or null
                            // MODE_STATE_ONLY: local end states [B,nseg,H,P,N]
    float *seg_decay;       // MODE_STATE_ONLY: [B,nseg,H] product of a_t over the segment
    int L, H, G, nseg, seg_len, mode;
    int *d_status;
};

struct __align__(8) SsdBars {
    uint64_t load_full[SSD_STAGES], load_empty[SSD_STAGES];
    uint64_t g_full, m_full, yd_full, yoff_full, dh_full, h_ready;
};
}  // namespace

__global__ void __launch_bounds__(SSD_THREADS, 1)
ssd_tiles_kernel(const __grid_constant__ CUtensorMap tmap_bc, const __grid_constant__ CUtensorMap tmap_x,
                 const SsdParams prm)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *s_stage = smem;                                  // SSD_STAGES x (C0 C1 B0 B1 X)
    uint8_t *s_xp = smem + SSD_STAGES * STAGE_BYTES;          // w . X      (MN-major B operand)
    uint8_t *s_hb = s_xp + SLAB;                              // bf16 state (MN-major B operand)
    float *s_cs = (float *)(s_hb + SLAB);                     // [128] log2(Delta_s) - l2_s
    float *s_scan = s_cs + ST;                                // [8] warp totals
    SsdBars *bars = (SsdBars *)(s_scan + 8);
    uint32_t *tmem_slot = (uint32_t *)(bars + 1);
    int *abort_flag = (int *)(tmem_slot + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int seg = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int g = h / (prm.H / prm.G);
    const int L = prm.L, H = prm.H;
    const int t_begin = seg * prm.seg_len;
    const int t_end = min(L, t_begin + prm.seg_len);
    const int ntiles = (t_end - t_begin + ST - 1) / ST;
    const bool full = prm.mode == MODE_FULL;
    int *d_status = prm.d_status;

    if (tid == 0) {
        for (int s = 0; s < SSD_STAGES; ++s) {
            tc::mbar_init(&bars->load_full[s], 1);
            tc::mbar_init(&bars->load_empty[s], 1);
        }
        tc::mbar_init(&bars->g_full, 1);
        tc::mbar_init(&bars->m_full, 128);
        tc::mbar_init(&bars->yd_full, 1);
        tc::mbar_init(&bars->yoff_full, 1);
        tc::mbar_init(&bars->dh_full, 1);
        tc::mbar_init(&bars->h_ready, 128);
        *abort_flag = 0;
        tc::fence_mbar_init();
    }
    if (warp == 5) {
        tc::tmem_alloc(tmem_slot, TM_COLS);
        tc::tmem_relinquish();
    }
    if (warp == 4 && lane == 0) {
        tc::prefetch_tmap(&tmap_bc);
        tc::prefetch_tmap(&tmap_x);
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 4) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            for (int j = 0; j < ntiles; ++j) {
                const int st = j % SSD_STAGES;
                tc::mbar_wait(&bars->load_empty[st], ((j / SSD_STAGES) & 1) ^ 1, abort_flag, d_status);
                uint8_t *base = s_stage + st * STAGE_BYTES;
                const int t0 = t_begin + j * ST;
                tc::mbar_arrive_expect_tx(&bars->load_full[st], full ? STAGE_BYTES : 3 * SLAB);
                if (full) {
                    tc::tma_load_3d(base + 0 * SLAB, &tmap_bc, &bars->load_full[st], (prm.G + g) * SN, t0, b);
                    tc::tma_load_3d(base + 1 * SLAB, &tmap_bc, &bars->load_full[st], (prm.G + g) * SN + 64, t0, b);
                }
                tc::tma_load_3d(base + 2 * SLAB, &tmap_bc, &bars->load_full[st], g * SN, t0, b);
                tc::tma_load_3d(base + 3 * SLAB, &tmap_bc, &bars->load_full[st], g * SN + 64, t0, b);
                tc::tma_load_4d(base + 4 * SLAB, &tmap_x, &bars->load_full[st], 0, h, t0, b);
            }
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t id_g = tc::idesc_bf16(128, 128, 0, 0);     // C (K-major) x B (K-major)
            constexpr uint32_t id_y = tc::idesc_bf16(128, 64, 0, 1);      // K-major / TMEM A, MN-major B
            constexpr uint32_t id_h = tc::idesc_bf16(128, 64, 1, 1);      // MN-major A and B
            const uint32_t xp_addr = tc::smem_u32(s_xp), hb_addr = tc::smem_u32(s_hb);
            for (int j = 0; j < ntiles; ++j) {
                const int st = j % SSD_STAGES;
                const uint32_t base = tc::smem_u32(s_stage + st * STAGE_BYTES);
                const uint32_t c_addr = base, b_addr = base + 2 * SLAB, x_addr = base + 4 * SLAB;
                tc::mbar_wait(&bars->load_full[st], (j / SSD_STAGES) & 1, abort_flag, d_status);
                tc::tc_fence_after();
                if (full) {
                    // MMA 1: G = Ctilde Btilde^T  (K = state index)
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        const uint32_t off = (kk >> 2) * SLAB + (kk & 3) * 32;
                        tc::mma_ss(tmem + TM_G, tc::smem_desc_sw128(c_addr + off, 16, 1024),
                                   tc::smem_desc_sw128(b_addr + off, 16, 1024), id_g, kk > 0);
                    }
                    tc::mma_commit(&bars->g_full);
                    // MMA 3: Yoff = Ctilde Hprev^T  (K = state index; B = bf16 state, rows = n)
                    tc::mbar_wait(&bars->h_ready, j & 1, abort_flag, d_status);
                    tc::tc_fence_after();
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        const uint32_t off = (kk >> 2) * SLAB + (kk & 3) * 32;
                        tc::mma_ss(tmem + TM_YOFF, tc::smem_desc_sw128(c_addr + off, 16, 1024),
                                   tc::smem_desc_sw128(hb_addr + kk * 2048, SLAB, 1024), id_y, kk > 0);
                    }
                    tc::mma_commit(&bars->yoff_full);
                }
                tc::mbar_wait(&bars->m_full, j & 1, abort_flag, d_status);
                tc::tc_fence_after();
                if (full) {
                    // MMA 2: Ydiag = M X  (A = masked tile in TMEM, 8 columns per 16 tokens of K)
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)
                        tc::mma_ts(tmem + TM_YD, tmem + TM_M + kk * 8,
                                   tc::smem_desc_sw128(x_addr + kk * 2048, SLAB, 1024), id_y, kk > 0);
                    tc::mma_commit(&bars->yd_full);
                }
                // MMA 4: dH^T[n,p] = sum_s Btilde[s,n] (w_s x_s[p])   (K = token)
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    tc::mma_ss(tmem + TM_DH, tc::smem_desc_sw128(b_addr + kk * 2048, SLAB, 1024),
                               tc::smem_desc_sw128(xp_addr + kk * 2048, SLAB, 1024), id_h, kk > 0);
                tc::mma_commit(&bars->dh_full);
                tc::mma_commit(&bars->load_empty[st]);
            }
        }
    } else {
        // ------------------------------------------------------------------ compute warps
        const int i = tid;                                   // token row in the tile == state index n
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        const float Ah = prm.A[h] * LOG2E, bias = prm.dt_bias[h];
        const float Dh = prm.D ? prm.D[h] : 0.f;
        // fp32 master copy of the state: this thread holds H[n = i][p = 0..63]
        float Hst[SP];
        {
            const float *h_in = prm.h_in;
            if (h_in && full) {
                const int64_t base = prm.nseg > 1
                    ? ((((int64_t)b * prm.nseg + seg) * H + h) * SP) * SN
                    : (((int64_t)b * H + h) * SP) * SN;
#pragma unroll
                for (int p = 0; p < SP; ++p) Hst[p] = h_in[base + (int64_t)p * SN + i];
            } else {
#pragma unroll
                for (int p = 0; p < SP; ++p) Hst[p] = 0.f;
            }
            if (full) {
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) {
                    uint4 v = make_uint4(tc::pack_bf16x2(Hst[8 * ch + 0], Hst[8 * ch + 1]),
                                         tc::pack_bf16x2(Hst[8 * ch + 2], Hst[8 * ch + 3]),
                                         tc::pack_bf16x2(Hst[8 * ch + 4], Hst[8 * ch + 5]),
                                         tc::pack_bf16x2(Hst[8 * ch + 6], Hst[8 * ch + 7]));
                    *reinterpret_cast<uint4 *>(s_hb + tc::sw128_offset(i, ch)) = v;
                }
                tc::fence_proxy_async_smem();
                tc::mbar_arrive(&bars->h_ready);
            }
        }
        float seg_l2 = 0.f;      // log2 of the product of a_t over the tiles done so far

        for (int j = 0; j < ntiles; ++j) {
            const int st = j % SSD_STAGES;
            uint8_t *stage = s_stage + st * STAGE_BYTES;
            const int t = t_begin + j * ST + i;
            const bool valid = t < t_end;
            // ---- per-token scalars: Delta, cumulative log2 decay inside the tile
            float delta = 0.f;
            if (valid) {
                const float raw = prm.dt ? prm.dt[((int64_t)b * L + t) * H + h] : 0.f;
                delta = softplus_f(raw + bias);
            }
            float l2 = delta * Ah;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const float nb = __shfl_up_sync(0xffffffffu, l2, o);
                if (lane >= o) l2 += nb;
            }
            tc::named_bar_sync(1, 128);                       // previous tile's readers of s_cs/s_scan done
            if (lane == 31) s_scan[warp] = l2;
            tc::named_bar_sync(1, 128);
            float l2_last = 0.f;
#pragma unroll
            for (int w = 0; w < 4; ++w) {
                const float tot = s_scan[w];
                if (w < warp) l2 += tot;
                l2_last += tot;
            }
            s_cs[i] = (delta > 0.f ? tc::lg2_approx(delta) : -INFINITY) - l2;
            const float w_s = delta * tc::ex2_approx(l2_last - l2);
            tc::named_bar_sync(1, 128);

            // ---- w . X  (row i of the X slab -> row i of the X' slab), keep x_i for the epilogue
            tc::mbar_wait(&bars->load_full[st], (j / SSD_STAGES) & 1, abort_flag, d_status);
            uint4 xrow[8];
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) {
                const uint32_t off = tc::sw128_offset(i, ch);
                xrow[ch] = *reinterpret_cast<const uint4 *>(stage + 4 * SLAB + off);
                const uint32_t wv[4] = {xrow[ch].x, xrow[ch].y, xrow[ch].z, xrow[ch].w};
                uint32_t o[4];
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    o[q] = tc::pack_bf16x2(w_s * __uint_as_float(wv[q] << 16),
                                           w_s * __uint_as_float(wv[q] & 0xffff0000u));
                *reinterpret_cast<uint4 *>(s_xp + off) = make_uint4(o[0], o[1], o[2], o[3]);
            }

            if (full) {
                // ---- decay mask: G (fp32, TMEM) -> M (bf16, TMEM), this thread owns row i
                tc::mbar_wait(&bars->g_full, j & 1, abort_flag, d_status);
                tc::tc_fence_after();
#pragma unroll 1
                for (int c = 0; c < 4; ++c) {
                    uint32_t pk[16];
                    if (c <= warp) {
                        uint32_t gv[32];
                        tc::tmem_ld32(tmem + lane_base + TM_G + c * 32, gv);
                        tc::tmem_ld_wait();
                        const bool diag = (c == warp);
#pragma unroll
                        for (int q = 0; q < 16; ++q) {
                            const float2 cs = *reinterpret_cast<const float2 *>(&s_cs[c * 32 + 2 * q]);
                            float m0 = __uint_as_float(gv[2 * q]) * tc::ex2_approx(l2 + cs.x);
                            float m1 = __uint_as_float(gv[2 * q + 1]) * tc::ex2_approx(l2 + cs.y);
                            if (diag) {
                                if (2 * q > lane) m0 = 0.f;
                                if (2 * q + 1 > lane) m1 = 0.f;
                            }
                            pk[q] = tc::pack_bf16x2(m0, m1);
                        }
                    } else {
#pragma unroll
                        for (int q = 0; q < 16; ++q) pk[q] = 0u;
                    }
                    tc::tmem_st16(tmem + lane_base + TM_M + c * 16, pk);
                }
                tc::tmem_st_wait();
            }
            tc::fence_proxy_async_smem();
            tc::tc_fence_before();
            tc::mbar_arrive(&bars->m_full);

            if (full) {
                // ---- epilogue: y_i = Ydiag_i + exp(l_i) Yoff_i + D x_i
                tc::mbar_wait(&bars->yoff_full, j & 1, abort_flag, d_status);
                tc::mbar_wait(&bars->yd_full, j & 1, abort_flag, d_status);
                tc::tc_fence_after();
                const float e_i = tc::ex2_approx(l2);
                __nv_bfloat16 *yrow = prm.y + (((int64_t)b * L + t) * H + h) * SP;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    uint32_t yd[32], yo[32];
                    tc::tmem_ld32(tmem + lane_base + TM_YD + half * 32, yd);
                    tc::tmem_ld32(tmem + lane_base + TM_YOFF + half * 32, yo);
                    tc::tmem_ld_wait();
                    if (valid) {
#pragma unroll
                        for (int ch = 0; ch < 4; ++ch) {
                            const uint4 xr = xrow[half * 4 + ch];
                            const uint32_t xw[4] = {xr.x, xr.y, xr.z, xr.w};
                            uint32_t o[4];
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const int e0 = ch * 8 + 2 * q;
                                const float x0 = __uint_as_float(xw[q] << 16);
                                const float x1 = __uint_as_float(xw[q] & 0xffff0000u);
                                const float y0 = __uint_as_float(yd[e0]) + e_i * __uint_as_float(yo[e0]) + Dh * x0;
                                const float y1 = __uint_as_float(yd[e0 + 1]) + e_i * __uint_as_float(yo[e0 + 1]) + Dh * x1;
                                o[q] = tc::pack_bf16x2(y0, y1);
                            }
                            *reinterpret_cast<uint4 *>(yrow + half * 32 + ch * 8) = make_uint4(o[0], o[1], o[2], o[3]);
                        }
                    }
                }
            }

            // ---- state: H = exp(l_last) H + dH  (thread i owns state index n = i)
            tc::mbar_wait(&bars->dh_full, j & 1, abort_flag, d_status);
            tc::tc_fence_after();
            const float dec = tc::ex2_approx(l2_last);
            seg_l2 += l2_last;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t dh[32];
                tc::tmem_ld32(tmem + lane_base + TM_DH + half * 32, dh);
                tc::tmem_ld_wait();
#pragma unroll
                for (int q = 0; q < 32; ++q)
                    Hst[half * 32 + q] = fmaf(dec, Hst[half * 32 + q], __uint_as_float(dh[q]));
            }
            if (full) {
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) {
                    uint4 v = make_uint4(tc::pack_bf16x2(Hst[8 * ch + 0], Hst[8 * ch + 1]),
                                         tc::pack_bf16x2(Hst[8 * ch + 2], Hst[8 * ch + 3]),
                                         tc::pack_bf16x2(Hst[8 * ch + 4], Hst[8 * ch + 5]),
                                         tc::pack_bf16x2(Hst[8 * ch + 6], Hst[8 * ch + 7]));
                    *reinterpret_cast<uint4 *>(s_hb + tc::sw128_offset(i, ch)) = v;
                }
                tc::fence_proxy_async_smem();
                tc::tc_fence_before();
                tc::mbar_arrive(&bars->h_ready);
            } else {
                tc::tc_fence_before();
            }
        }

        // ---- final state of the segment
        if (full) {
            if (prm.h_out && seg == prm.nseg - 1) {
                float *dst = prm.h_out + (((int64_t)b * H + h) * SP) * SN;
#pragma unroll
                for (int p = 0; p < SP; ++p) dst[(int64_t)p * SN + i] = Hst[p];
            }
        } else {
            float *dst = prm.h_out + ((((int64_t)b * prm.nseg + seg) * H + h) * SP) * SN;
#pragma unroll
            for (int p = 0; p < SP; ++p) dst[(int64_t)p * SN + i] = Hst[p];
            if (i == 0) prm.seg_decay[((int64_t)b * prm.nseg + seg) * H + h] = tc::ex2_approx(seg_l2);
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 5) tc::tmem_dealloc(tmem, TM_COLS);
}

// K3: chain the segments.  states[b,s,h,:,:] holds segment s's local end state (computed from a
// zero initial state) on entry and the state ENTERING segment s on exit:
//   H_in(0) = h0,   H_in(s+1) = decay(s) H_in(s) + S(s).
// One thread per 4 consecutive state entries; segments are walked in order.
__global__ void __launch_bounds__(256)
segment_scan_kernel(float *__restrict__ states, const float *__restrict__ seg_decay,
                    const float *__restrict__ h0, int nseg, int H, int PN4)
{
    const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;   // float4 index inside [P*N/4]
    const int h = blockIdx.y, b = blockIdx.z;
    if (v >= PN4) return;
    float4 run = h0 ? reinterpret_cast<const float4 *>(h0)[((int64_t)b * H + h) * PN4 + v]
                    : make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < nseg; ++s) {
        float4 *p = reinterpret_cast<float4 *>(states) + (((int64_t)b * nseg + s) * H + h) * PN4 + v;
        const float4 loc = *p;
        const float d = seg_decay[((int64_t)b * nseg + s) * H + h];
        *p = run;
        run.x = fmaf(d, run.x, loc.x);
        run.y = fmaf(d, run.y, loc.y);
        run.z = fmaf(d, run.z, loc.z);
        run.w = fmaf(d, run.w, loc.w);
    }
}

bool ssd_tiles_supported(int dtype, int P, int N)
{
    return dtype == SWIMBA_DTYPE_BF16 && P == SP && N == SN;
}

static size_t ssd_smem_bytes()
{
    return 1024 + SSD_STAGES * STAGE_BYTES + 2 * SLAB + (ST + 8) * sizeof(float) + sizeof(SsdBars) + 64;
}

// Segment length (tokens, multiple of 128) so that the grid fills the SMs; L itself if one
// segment per sequence is enough.
int ssd_segment_len(int B, int L, int H, int chunk, int sm_count)
{
    const int64_t pairs = (int64_t)B * H;
    const int tiles = ceil_div(L, ST);
    if (pairs >= sm_count || tiles <= 2) return tiles * ST;
    int want = (int)ceil_div64(2 * (int64_t)sm_count, pairs);        // segments per sequence
    int q_tiles = chunk >= ST ? chunk / ST : 1;                       // segments are whole chunks
    int seg_tiles = ceil_div(tiles, want);
    seg_tiles = ceil_div(seg_tiles, q_tiles) * q_tiles;
    if (seg_tiles < 4) seg_tiles = 4 < tiles ? 4 : tiles;
    return seg_tiles * ST;
}

size_t ssd_workspace_bytes(int B, int L, int H, int chunk, int sm_count)
{
    const int seg_len = ssd_segment_len(B, L, H, chunk, sm_count);
    const int nseg = ceil_div(L, seg_len);
    if (nseg <= 1) return 0;
    return (size_t)B * nseg * H * SP * SN * sizeof(float) + ((size_t)B * nseg * H * sizeof(float) + 255) / 256 * 256;
}

int launch_ssd_tiles(LaunchCtx &ctx, const void *x, const void *BC, const float *dt, const float *A,
                     const float *dt_bias, const float *D, const float *h0, int B, int L, int H, int G,
                     int chunk, int sm_count, void *y, float *h_final, void *workspace)
{
    if (B <= 0 || L <= 0) return SWIMBA_OK;
    const int S = 2 * G * SN;
    CUtensorMap tm_bc, tm_x;
    {
        const uint64_t dims[3] = {(uint64_t)S, (uint64_t)L, (uint64_t)B};
        const uint64_t str[2] = {(uint64_t)S * 2, (uint64_t)L * S * 2};
        const uint32_t box[3] = {64, ST, 1};
        if (!encode_tmap_bf16(&tm_bc, BC, 3, dims, str, box)) return SWIMBA_ERR_CUDA;
    }
    {
        const uint64_t dims[4] = {(uint64_t)SP, (uint64_t)H, (uint64_t)L, (uint64_t)B};
        const uint64_t str[3] = {(uint64_t)SP * 2, (uint64_t)H * SP * 2, (uint64_t)L * H * SP * 2};
        const uint32_t box[4] = {SP, 1, ST, 1};
        if (!encode_tmap_bf16(&tm_x, x, 4, dims, str, box)) return SWIMBA_ERR_CUDA;
    }
    const size_t smem = ssd_smem_bytes();
    if (cudaFuncSetAttribute(ssd_tiles_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return SWIMBA_ERR_CUDA;

    const int seg_len = ssd_segment_len(B, L, H, chunk, sm_count);
    const int nseg = ceil_div(L, seg_len);
    SsdParams p;
    p.dt = dt; p.A = A; p.dt_bias = dt_bias; p.D = D;
    p.y = (__nv_bfloat16 *)y;
    p.L = L; p.H = H; p.G = G; p.nseg = nseg; p.seg_len = seg_len;
    p.d_status = ctx.d_status;
    dim3 grid((unsigned)nseg, (unsigned)H, (unsigned)B);
    if (nseg == 1) {
        p.h_in = h0; p.h_out = h_final; p.seg_decay = nullptr; p.mode = MODE_FULL;
        ctx.begin(STAGE_SSD_TILES);
        ssd_tiles_kernel<<<grid, SSD_THREADS, smem, ctx.stream>>>(tm_bc, tm_x, p);
        ctx.end();
    } else {
        float *states = (float *)workspace;
        float *decay = states + (size_t)B * nseg * H * SP * SN;
        p.h_in = nullptr; p.h_out = states; p.seg_decay = decay; p.mode = MODE_STATE_ONLY;
        ctx.begin(STAGE_SSD_TILES);
        ssd_tiles_kernel<<<grid, SSD_THREADS, smem, ctx.stream>>>(tm_bc, tm_x, p);
        ctx.end();
        const int PN4 = SP * SN / 4;
        ctx.begin(STAGE_SEGMENT_SCAN);
        segment_scan_kernel<<<dim3((unsigned)ceil_div(PN4, 256), (unsigned)H, (unsigned)B), 256, 0, ctx.stream>>>(
            states, decay, h0, nseg, H, PN4);
        ctx.end();
        p.h_in = states; p.h_out = h_final; p.seg_decay = nullptr; p.mode = MODE_FULL;
        ctx.begin(STAGE_SSD_TILES);
        ssd_tiles_kernel<<<grid, SSD_THREADS, smem, ctx.stream>>>(tm_bc, tm_x, p);
        ctx.end();
    }
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

}  // namespace swimba
