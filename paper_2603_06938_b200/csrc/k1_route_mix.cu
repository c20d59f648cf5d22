// K1 (SIMT part): router logits + softmax + top-k, and the plain projection/mix used by the
// fp32 path and by decode.  (Router softmax equation and top-k rule; Theorem 1, mixed streams.)
#include "internal.h"
#include "tc05.cuh"
#include <type_traits>

namespace swimba {

// Router: a block handles chunks of `chunk` consecutive tokens, one warp TPW tokens at a time;
// the router matrix is staged in shared memory once per block (when it fits) so that every token
// costs one pass over its own features.
//
// Logit summation order (fixed, so results are reproducible run to run): lane l accumulates
// features f = 256*c + 8*l + i (c ascending, i = 0..7) with fused multiply-adds; the 32 partial
// sums of each (token, expert) are then combined by a halving butterfly over lane distances
// 16, 8, 4, 2, 1 in which each step also halves the number of values a lane still carries, so
// that afterwards every lane owns the complete logit of one (token, expert) pair (or of V/32
// adjacent experts when V = TPW*EP exceeds 32).  bf16 products are exact in fp32, so the only
// rounding is in the additions.  Softmax and top-k then run across the lanes of a token's group.
//
// Grouping by expert is done here as well: entry (t, j) goes to its expert's list,
// perm[e * cap + pos] = t*k + j.  Positions are handed out per chunk: a shared-memory histogram
// gives every entry its rank inside the chunk, one global atomic per (chunk, expert) on counts[e]
// (zeroed by the caller) reserves the chunk's range.  The order inside a list is arbitrary; every
// output row is computed independently of its position, so results do not depend on it.
constexpr int ROUTER_MAX_CHUNK = 512;

template <typename T, int EP, int TPW>
__global__ void __launch_bounds__(256)
router_topk_kernel(const T *__restrict__ u, const T *__restrict__ W_r, int64_t Ttok, int F, int E,
                   int k, int32_t *__restrict__ idx, float *__restrict__ w, int *__restrict__ counts,
                   int *__restrict__ perm, int64_t cap, int stage_w, int chunk,
                   uint4 *__restrict__ zero_out, int zero_vec_per_token, int router_blocks)
{
    grid_dep_launch();      // the projection kernel may set itself up under this kernel's tail
    const int rblock = (int)blockIdx.x;
    constexpr int V = TPW * EP;                 // values per lane before the butterfly
    constexpr int R = V > 32 ? V / 32 : 1;      // values per lane after it (adjacent experts)
    constexpr int DUP = V >= 32 ? 1 : 32 / V;   // lanes holding the same value after it
    constexpr int GW = 32 / TPW;                // lanes per token group
    static_assert(V >= 2 && (V & (V - 1)) == 0 && R <= EP, "unsupported router shape");
    extern __shared__ __align__(16) unsigned char router_smem[];
    __shared__ int s_cnt[SWIMBA_MAX_EXPERTS], s_base[SWIMBA_MAX_EXPERTS];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
    int *s_ent = reinterpret_cast<int *>(router_smem);              // [chunk * k] expert | rank << 8
    const T *Wsrc = W_r;
    if (stage_w) {
        T *sW = reinterpret_cast<T *>(router_smem + (size_t)ROUTER_MAX_CHUNK * SWIMBA_MAX_TOPK * sizeof(int));
        const int nvec = (int)(((int64_t)E * F * sizeof(T)) >> 4);
        const uint4 *src = reinterpret_cast<const uint4 *>(W_r);
        uint4 *dst = reinterpret_cast<uint4 *>(sW);
        for (int i = threadIdx.x; i < nvec; i += blockDim.x) dst[i] = src[i];
        Wsrc = sW;
    }
    // after the butterfly this lane owns experts e0 .. e0+R-1 of token q_own of the pass
    const int q_own = lane / GW;
    const int e0 = ((lane % GW) / DUP) * R;
    const int64_t nchunks = ceil_div64(Ttok, chunk);
    for (int64_t c = rblock; c < nchunks; c += router_blocks) {
        const int64_t tbeg = c * chunk;
        const int64_t tend = (tbeg + chunk < Ttok) ? tbeg + chunk : Ttok;
        if (threadIdx.x < SWIMBA_MAX_EXPERTS) s_cnt[threadIdx.x] = 0;
        if (zero_out) {
            // the mixed-stream rows of this chunk start at zero: the projection adds its slots
            const int64_t nz = (tend - tbeg) * zero_vec_per_token;
            uint4 *z = zero_out + tbeg * zero_vec_per_token;
            for (int64_t i = threadIdx.x; i < nz; i += blockDim.x) z[i] = make_uint4(0u, 0u, 0u, 0u);
        }
        __syncthreads();
        // The feature loads run one step ahead of the arithmetic, across passes too: `raw` always
        // holds the next 8-feature slice of the next TPW tokens.
        typename Raw8<T>::type raw[TPW];
        auto prefetch = [&](int64_t tt0, int ff) {
#pragma unroll
            for (int q = 0; q < TPW; ++q) {
                const int64_t t = (tt0 + q < tend) ? tt0 + q : tt0;
                load_raw8(u + t * F + ff, raw[q]);
            }
        };
        if (tbeg + warp * TPW < tend && lane * 8 < F) prefetch(tbeg + warp * TPW, lane * 8);
        for (int64_t t0 = tbeg + warp * TPW; t0 < tend; t0 += nwarp * TPW) {
            float g[V];                                  // g[q * EP + e]
#pragma unroll
            for (int i = 0; i < V; ++i) g[i] = 0.f;
#pragma unroll 1
            for (int f = lane * 8; f < F; f += 256) {
                float uv[TPW][8];
#pragma unroll
                for (int q = 0; q < TPW; ++q) unpack8(raw[q], uv[q]);
                if (f + 256 < F) prefetch(t0, f + 256);
                else if (t0 + nwarp * TPW < tend) prefetch(t0 + nwarp * TPW, lane * 8);
#pragma unroll
                for (int e = 0; e < EP; ++e) {
                    if (e < E) {
                        float wv[8];
                        load8(Wsrc + (int64_t)e * F + f, wv);
#pragma unroll
                        for (int q = 0; q < TPW; ++q)
#pragma unroll
                            for (int i = 0; i < 8; ++i)
                                g[q * EP + e] = fmaf(wv[i], uv[q][i], g[q * EP + e]);
                    }
                }
            }
            // halving butterfly: V values on 32 lanes -> R values on this lane
            {
                int n = V;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    if (n > R) {
                        n >>= 1;
                        const bool up = (lane & o) != 0;
#pragma unroll
                        for (int i = 0; i < V / 2; ++i) {
                            if (i < n) {
                                const float send = up ? g[i] : g[i + n];
                                const float keep = up ? g[i + n] : g[i];
                                g[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
                            }
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < R; ++i) g[i] += __shfl_xor_sync(0xffffffffu, g[i], o);
                    }
                }
            }
            // softmax over ALL experts of the token (padding experts count as -inf)
            float gv[R], pv[R];
            float m = -INFINITY;
#pragma unroll
            for (int i = 0; i < R; ++i) {
                gv[i] = (e0 + i < E) ? g[i] : -INFINITY;
                m = fmaxf(m, gv[i]);
            }
#pragma unroll
            for (int o = GW / 2; o >= DUP; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            float z = 0.f;
#pragma unroll
            for (int i = 0; i < R; ++i) {
                pv[i] = expf(gv[i] - m);
                z += pv[i];
            }
#pragma unroll
            for (int o = GW / 2; o >= DUP; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
            // k rounds of "largest remaining logit, lowest index on ties"; weights are NOT
            // renormalised
            const int64_t t = t0 + q_own;
            for (int j = 0; j < k; ++j) {
                float bg = gv[0], bp = pv[0];
                int be = e0;
#pragma unroll
                for (int i = 1; i < R; ++i)
                    if (gv[i] > bg) { bg = gv[i]; bp = pv[i]; be = e0 + i; }
#pragma unroll
                for (int o = GW / 2; o >= DUP; o >>= 1) {
                    const float og = __shfl_xor_sync(0xffffffffu, bg, o);
                    const float op = __shfl_xor_sync(0xffffffffu, bp, o);
                    const int oe = __shfl_xor_sync(0xffffffffu, be, o);
                    if (og > bg || (og == bg && oe < be)) { bg = og; bp = op; be = oe; }
                }
#pragma unroll
                for (int i = 0; i < R; ++i) if (e0 + i == be) gv[i] = -INFINITY;
                if (lane % GW == 0 && t < tend) {
                    idx[t * k + j] = be;
                    w[t * k + j] = bp / z;
                    if (counts) {
                        const int rank = atomicAdd(&s_cnt[be], 1);
                        s_ent[(int)(t - tbeg) * k + j] = be | (rank << 8);
                    }
                }
            }
        }
        if (counts) {
            __syncthreads();
            if (threadIdx.x < E) s_base[threadIdx.x] = atomicAdd(&counts[threadIdx.x], s_cnt[threadIdx.x]);
            __syncthreads();
            const int n_ent = (int)(tend - tbeg) * k;
            for (int i = threadIdx.x; i < n_ent; i += blockDim.x) {
                const int ent = s_ent[i], e = ent & 255;
                perm[(int64_t)e * cap + s_base[e] + (ent >> 8)] = (int)(tbeg * k + i);
            }
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------
// Tensor-core router (bf16, F a multiple of 128).  The logits of 16 tokens and 8 experts are one
// m16n8k16 product chain; a block step covers 32 tokens with 8 warps: warp = (row group of 16
// tokens, quarter of the features).  The contraction runs over features in any order, so each lane
// reads 16 contiguous bytes of its two token rows (features 32 j + 8 c .. + 8 of the warp's
// quarter, c = lane % 4) and feeds them to two MMAs; the matching slice of the router matrix comes
// from shared memory (rows padded by 64 bytes against bank conflicts), rows past E are zero.
//
// Logit summation order (fixed, so results are reproducible run to run): inside a warp the MMAs
// run over j ascending, first the lower then the upper four features of a lane's eight; the four
// feature quarters are then added in ascending order by the thread that owns the logit.  bf16
// products are exact in fp32; the additions are those of the tensor core's fp32 accumulator.
// Softmax and top-k run on 8 lanes per token, lane s holding experts s, s + 8, ...
// ------------------------------------------------------------------------------------------
constexpr int RM_TOK = 32;        // tokens per block step
constexpr int RM_KSPLIT = 4;      // warps sharing the features of a row group
constexpr int RM_UNROLL = 3;      // 32-feature blocks whose loads are issued together

__device__ __forceinline__ void mma_bf16_16x8x16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                                 uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, "
        "{%8, %9}, {%0, %1, %2, %3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int NT>
__global__ void __launch_bounds__(256, NT <= 2 ? 4 : 2)
router_mma_kernel(const __nv_bfloat16 *__restrict__ u, const __nv_bfloat16 *__restrict__ W_r,
                  int64_t Ttok, int F, int E, int k, int32_t *__restrict__ idx, float *__restrict__ w,
                  int *__restrict__ counts, int *__restrict__ perm, int64_t cap, int stage_w,
                  int chunk, uint4 *__restrict__ zero_out, int zero_vec_per_token, int router_blocks,
                  int scalar_blocks, const ScalarsArgs scalars)
{
    grid_dep_launch();      // the projection kernel may set itself up under this kernel's tail
    if ((int)blockIdx.x < scalar_blocks) {
        // leading blocks: SSD step sizes and tile log-decays of the same call (they depend on dt
        // only); being short, they also stagger the start of the router blocks behind them
        ssd_scalars_block(scalars, blockIdx.x);
        return;
    }
    const int rblock = (int)blockIdx.x - scalar_blocks;       // index among the router blocks
    constexpr int EPAD = 8 * NT;
    extern __shared__ __align__(16) unsigned char router_smem[];
    __shared__ int s_cnt[SWIMBA_MAX_EXPERTS], s_base[SWIMBA_MAX_EXPERTS];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int *s_ent = reinterpret_cast<int *>(router_smem);              // [chunk * k] expert | rank << 8
    float *s_part = reinterpret_cast<float *>(router_smem + (((size_t)chunk * k * sizeof(int) + 15) & ~(size_t)15));
    unsigned char *sW = reinterpret_cast<unsigned char *>(s_part + RM_TOK * RM_KSPLIT * EPAD);
    const int w_stride = F * 2 + 64;                                 // bytes per staged row
    if (stage_w) {
        const int vec_per_row = F >> 3;
        const uint4 *src = reinterpret_cast<const uint4 *>(W_r);
        for (int i = tid; i < EPAD * vec_per_row; i += blockDim.x) {
            const int e = i / vec_per_row, v = i - e * vec_per_row;
            const uint4 val = e < E ? src[(int64_t)e * vec_per_row + v] : make_uint4(0u, 0u, 0u, 0u);
            *reinterpret_cast<uint4 *>(sW + e * w_stride + v * 16) = val;
        }
    }
    const int tg = warp >> 2, ks = warp & 3;          // row group, feature quarter
    const int g = lane >> 2, c = lane & 3;            // MMA row / column-pair of this lane
    const int fq = F / RM_KSPLIT, nblk = fq / 32;
    const int f_lane = ks * fq + 8 * c;               // first feature this lane reads
    const int tl = tid >> 3, sub = tid & 7;           // finalisation: token of the step, lane of 8
    const int64_t nchunks = ceil_div64(Ttok, chunk);
    for (int64_t cidx = rblock; cidx < nchunks; cidx += router_blocks) {
        const int64_t tbeg = cidx * chunk;
        const int64_t tend = (tbeg + chunk < Ttok) ? tbeg + chunk : Ttok;
        if (tid < SWIMBA_MAX_EXPERTS) s_cnt[tid] = 0;
        if (zero_out) {
            // the mixed-stream rows of this chunk start at zero: the projection adds its slots
            const int64_t nz = (tend - tbeg) * zero_vec_per_token;
            uint4 *z = zero_out + tbeg * zero_vec_per_token;
            for (int64_t i = tid; i < nz; i += blockDim.x) z[i] = make_uint4(0u, 0u, 0u, 0u);
        }
        __syncthreads();
        for (int64_t t0 = tbeg; t0 < tend; t0 += RM_TOK) {
            // rows past the chunk repeat its last token; their results are never written
            const int64_t r0 = t0 + tg * 16 + g, r1 = r0 + 8;
            const __nv_bfloat16 *p0 = u + (r0 < tend ? r0 : tend - 1) * F + f_lane;
            const __nv_bfloat16 *p1 = u + (r1 < tend ? r1 : tend - 1) * F + f_lane;
            float acc[NT][4];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[nt][i] = 0.f;
            for (int j0 = 0; j0 < nblk; j0 += RM_UNROLL) {
                uint4 xa[RM_UNROLL], xb[RM_UNROLL];
#pragma unroll
                for (int jj = 0; jj < RM_UNROLL; ++jj) {
                    if (j0 + jj < nblk) {
                        xa[jj] = *reinterpret_cast<const uint4 *>(p0 + (j0 + jj) * 32);
                        xb[jj] = *reinterpret_cast<const uint4 *>(p1 + (j0 + jj) * 32);
                    }
                }
#pragma unroll
                for (int jj = 0; jj < RM_UNROLL; ++jj) {
                    if (j0 + jj < nblk) {
                        const int f = f_lane + (j0 + jj) * 32;
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            const int e = nt * 8 + g;
                            uint4 wv;
                            if (stage_w) wv = *reinterpret_cast<const uint4 *>(sW + e * w_stride + f * 2);
                            else wv = e < E ? __ldg(reinterpret_cast<const uint4 *>(W_r + (int64_t)e * F + f))
                                            : make_uint4(0u, 0u, 0u, 0u);
                            mma_bf16_16x8x16(acc[nt], xa[jj].x, xb[jj].x, xa[jj].y, xb[jj].y, wv.x, wv.y);
                            mma_bf16_16x8x16(acc[nt], xa[jj].z, xb[jj].z, xa[jj].w, xb[jj].w, wv.z, wv.w);
                        }
                    }
                }
            }
            // partial logits of this warp's feature quarter: s_part[token][quarter][expert]
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                float *q0 = s_part + ((tg * 16 + g) * RM_KSPLIT + ks) * EPAD + nt * 8 + 2 * c;
                *reinterpret_cast<float2 *>(q0) = make_float2(acc[nt][0], acc[nt][1]);
                *reinterpret_cast<float2 *>(q0 + 8 * RM_KSPLIT * EPAD) = make_float2(acc[nt][2], acc[nt][3]);
            }
            __syncthreads();
            // softmax over ALL experts of the token (padding experts count as -inf)
            float gv[NT], pv[NT];
            float m = -INFINITY;
#pragma unroll
            for (int i = 0; i < NT; ++i) {
                const int e = sub + 8 * i;
                const float *q = s_part + tl * RM_KSPLIT * EPAD + e;
                float sum = q[0];
#pragma unroll
                for (int s = 1; s < RM_KSPLIT; ++s) sum += q[s * EPAD];
                gv[i] = e < E ? sum : -INFINITY;
                m = fmaxf(m, gv[i]);
            }
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
            float z = 0.f;
#pragma unroll
            for (int i = 0; i < NT; ++i) {
                pv[i] = expf(gv[i] - m);
                z += pv[i];
            }
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
            // k rounds of "largest remaining logit, lowest index on ties"; weights are NOT
            // renormalised
            const int64_t t = t0 + tl;
            for (int j = 0; j < k; ++j) {
                float bg = gv[0], bp = pv[0];
                int be = sub;
#pragma unroll
                for (int i = 1; i < NT; ++i)
                    if (gv[i] > bg) { bg = gv[i]; bp = pv[i]; be = sub + 8 * i; }
#pragma unroll
                for (int o = 4; o > 0; o >>= 1) {
                    const float og = __shfl_xor_sync(0xffffffffu, bg, o);
                    const float op = __shfl_xor_sync(0xffffffffu, bp, o);
                    const int oe = __shfl_xor_sync(0xffffffffu, be, o);
                    if (og > bg || (og == bg && oe < be)) { bg = og; bp = op; be = oe; }
                }
#pragma unroll
                for (int i = 0; i < NT; ++i) if (sub + 8 * i == be) gv[i] = -INFINITY;
                if (sub == 0 && t < tend) {
                    idx[t * k + j] = be;
                    w[t * k + j] = bp / z;
                    if (counts) {
                        const int rank = atomicAdd(&s_cnt[be], 1);
                        s_ent[(int)(t - tbeg) * k + j] = be | (rank << 8);
                    }
                }
            }
            __syncthreads();        // s_part is rewritten by the next step
        }
        if (counts) {
            if (tid < E) s_base[tid] = atomicAdd(&counts[tid], s_cnt[tid]);
            __syncthreads();
            const int n_ent = (int)(tend - tbeg) * k;
            for (int i = tid; i < n_ent; i += blockDim.x) {
                const int ent = s_ent[i], e = ent & 255;
                perm[(int64_t)e * cap + s_base[e] + (ent >> 8)] = (int)(tbeg * k + i);
            }
        }
        __syncthreads();
    }
}

// ------------------------------------------------------------------------------------------
// Streaming router (bf16): the token features are the only large operand, so the kernel is built
// around keeping HBM reads in flight and contiguous.  A CTA owns 64-token tiles (static round
// robin); warp w of its four holds tokens 16 w .. 16 w + 15 of a tile and runs its own pipeline: an
// elected lane issues TMA loads of [16 tokens x 64 features] boxes (128-byte rows, 128-byte swizzle;
// rows and features past the end are zero-filled), four to a stage (512 contiguous bytes of every
// row), into the warp's private ring of stages; the warp consumes a stage with m16n8k16 products
// against the router matrix, which sits in shared memory already arranged as B fragments (one
// 8-byte read per lane and product), and refills it at once with the stage that comes a ring later
// (of the next tile if need be).  No warp waits for another inside the feature loop, and the
// loads of the next tile proceed while a tile's softmax, top-k and list bookkeeping run.
//
// Logit summation order (fixed, so results are reproducible run to run): features ascending in
// blocks of 16, each block one tensor-core product accumulated in fp32 (with at most 16 experts,
// even and odd blocks in two accumulators that are added at the end).  bf16 products are exact
// in fp32; the additions are those of the tensor core's accumulator.  A token's logits end up on
// the four lanes of its row (lane c holds experts 8 n + 2 c, 8 n + 2 c + 1); softmax and top-k run
// across them.
// ------------------------------------------------------------------------------------------
constexpr int RS_TOK = 64;                       // tokens per tile
constexpr int RS_CW = RS_TOK / 16;               // warps
constexpr int RS_BOX = 64;                       // features per TMA box (128-byte rows)
constexpr int RS_NBOX = 4;                       // boxes per stage
constexpr int RS_BK = RS_BOX * RS_NBOX;          // features per stage
constexpr int RS_BOX_BYTES = 16 * 128;
constexpr int RS_STAGE_BYTES = RS_NBOX * RS_BOX_BYTES;
constexpr int RS_THREADS = 32 * RS_CW;
constexpr int RS_MAX_STAGES = 4;

struct RouterStreamSmall {
    uint64_t full[RS_CW][RS_MAX_STAGES];
    int cnt[SWIMBA_MAX_EXPERTS], base[SWIMBA_MAX_EXPERTS];
    int abort_flag;
};

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}

template <int NT>
__global__ void __launch_bounds__(RS_THREADS)
router_stream_kernel(const __grid_constant__ CUtensorMap tmap_u, const __nv_bfloat16 *__restrict__ W_r,
                     int64_t Ttok, int F, int E, int k, int32_t *__restrict__ idx, float *__restrict__ w,
                     int *__restrict__ counts, int *__restrict__ perm, int64_t cap,
                     uint4 *__restrict__ zero_out, int zero_vec_per_token, int router_ctas,
                     int nstages, int *d_status)
{
    grid_dep_launch();      // the projection kernel may set itself up under this kernel's tail
    const int cta = (int)blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31;
    const int cw = __shfl_sync(0xffffffffu, tid >> 5, 0);
    extern __shared__ __align__(16) unsigned char router_smem[];
    unsigned char *ring = reinterpret_cast<unsigned char *>(((uintptr_t)router_smem + 1023) & ~(uintptr_t)1023);
    const int KB = ceil_div(F, RS_BK);                               // stages per tile
    constexpr int KSTEPS = RS_BK / 16;                               // products per stage
    uint2 *sWp = reinterpret_cast<uint2 *>(ring + (size_t)RS_CW * nstages * RS_STAGE_BYTES);   // [KB*KSTEPS][NT][32]
    int *s_ent = reinterpret_cast<int *>(sWp + (size_t)KB * KSTEPS * NT * 32);                  // [RS_TOK * k]
    RouterStreamSmall *sm = reinterpret_cast<RouterStreamSmall *>(
        (reinterpret_cast<uintptr_t>(s_ent + RS_TOK * k) + 15) & ~(uintptr_t)15);
    int *abort_flag = &sm->abort_flag;

    if (tid == 0) {
        for (int q = 0; q < RS_CW; ++q)
            for (int s = 0; s < RS_MAX_STAGES; ++s) tc::mbar_init(&sm->full[q][s], 1);
        *abort_flag = 0;
        tc::fence_mbar_init();
    }
    if (tid == 32) tc::prefetch_tmap(&tmap_u);
    __syncthreads();
    // Loads are numbered across the CTA's tiles: load `n` is feature block n % KB of the CTA's tile
    // number n / KB and goes to stage n % nstages of the warp's ring.  The first ring-full is issued
    // before the router matrix is staged, so that both latencies overlap.
    const int64_t ntiles = ceil_div64(Ttok, RS_TOK);
    const uint32_t n_loads = cta < ntiles ? (uint32_t)((ntiles - cta + router_ctas - 1) / router_ctas) * KB : 0u;
    unsigned char *my_ring = ring + (size_t)cw * nstages * RS_STAGE_BYTES;
    uint64_t *my_full = sm->full[cw];
    const bool leader = tc::elect_one();
    auto issue_load = [&](uint32_t n) {
        const int s = n % nstages;
        const int64_t tile = cta + (int64_t)(n / KB) * router_ctas;
        tc::mbar_arrive_expect_tx(&my_full[s], RS_STAGE_BYTES);
#pragma unroll
        for (int bx = 0; bx < RS_NBOX; ++bx)
            tc::tma_load_2d(my_ring + s * RS_STAGE_BYTES + bx * RS_BOX_BYTES, &tmap_u, &my_full[s],
                            (int)(n % KB) * RS_BK + bx * RS_BOX, (int)(tile * RS_TOK) + cw * 16);
    };
    if (leader)
        for (uint32_t n = 0; n < n_loads && n < (uint32_t)nstages; ++n) issue_load(n);
    __syncwarp();
    // Router matrix as B fragments: entry ((kk * NT + nt) * 32 + lane) holds, for the 16-feature
    // block kk and expert e = 8 nt + lane / 4, the features 16 kk + 2 c, + 1 (low word) and
    // 16 kk + 8 + 2 c, + 1 (high word), c = lane % 4; zero past E or F.  Sixteen contiguous bytes
    // of an expert's row are the same word of four consecutive entries.
    {
        const int n_ent = KB * KSTEPS * NT * 32;
        if ((E & 7) != 0 || F % RS_BK != 0) {
            for (int i = tid; i < n_ent; i += RS_THREADS) sWp[i] = make_uint2(0u, 0u);
            __syncthreads();
        }
        const uint4 *W4 = reinterpret_cast<const uint4 *>(W_r);
        const int vec_per_row = F >> 3, n_vec = E * vec_per_row;
#pragma unroll 8
        for (int i = tid; i < n_vec; i += RS_THREADS) {
            const int e = i / vec_per_row, v = i - e * vec_per_row;
            const uint4 val = W4[i];
            uint32_t *dst = reinterpret_cast<uint32_t *>(&sWp[((v >> 1) * NT + (e >> 3)) * 32 + (e & 7) * 4]) + (v & 1);
            dst[0] = val.x;
            dst[2] = val.y;
            dst[4] = val.z;
            dst[6] = val.w;
        }
    }
    __syncthreads();

    const int g = lane >> 2, c = lane & 3;
    // ldmatrix: lane l addresses row (l % 8) + 8 * ((l / 8) % 2) of the warp's 16 rows and the
    // 16-byte chunk 2 kk + l / 16 of the 128-byte row
    const int lm_row = (lane & 7) + ((lane >> 3) & 1) * 8;
    const int lm_chunk = lane >> 4;
    const uint32_t ring_addr = tc::smem_u32(my_ring) + lm_row * 128;
    uint32_t n = 0;
    for (int64_t tile = cta; tile < ntiles; tile += router_ctas) {
        const int64_t tbeg = tile * RS_TOK;
        const int64_t tend = (tbeg + RS_TOK < Ttok) ? tbeg + RS_TOK : Ttok;
        if (tid < SWIMBA_MAX_EXPERTS) sm->cnt[tid] = 0;
        if (zero_out) {
            // the mixed-stream rows of this tile start at zero: the projection adds its slots
            const int64_t nz = (tend - tbeg) * zero_vec_per_token;
            uint4 *z = zero_out + tbeg * zero_vec_per_token;
            for (int64_t i = tid; i < nz; i += RS_THREADS) z[i] = make_uint4(0u, 0u, 0u, 0u);
        }
        // few expert tiles: even and odd feature blocks go to separate accumulators so that
        // consecutive products do not wait on each other
        constexpr int CH = NT <= 2 ? 2 : 1;
        float accs[CH][NT][4];
#pragma unroll
        for (int ch = 0; ch < CH; ++ch)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) accs[ch][nt][i] = 0.f;
        for (int kb = 0; kb < KB; ++kb, ++n) {
            const int s = n % nstages;
            tc::mbar_wait(&my_full[s], (n / nstages) & 1, abort_flag, d_status);
            const uint32_t st = ring_addr + s * RS_STAGE_BYTES;
#pragma unroll
            for (int kk = 0; kk < KSTEPS; ++kk) {
                uint32_t a[4];
                ldmatrix_x4(a, st + (kk >> 2) * RS_BOX_BYTES + ((((2 * kk) & 7) + lm_chunk) ^ (lm_row & 7)) * 16);
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const uint2 bv = sWp[((kb * KSTEPS + kk) * NT + nt) * 32 + lane];
                    mma_bf16_16x8x16(accs[kk % CH][nt], a[0], a[1], a[2], a[3], bv.x, bv.y);
                }
            }
            // the reads above must be ordered before the TMA write that refills the stage
            tc::fence_proxy_async_smem();
            __syncwarp();
            if (leader && n + nstages < n_loads) issue_load(n + nstages);
        }
        float acc[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[nt][i] = CH == 2 ? accs[0][nt][i] + accs[CH - 1][nt][i] : accs[0][nt][i];
        // the histogram is clear and the previous tile's lists have been written
        __syncthreads();
        // softmax over ALL experts of the token (padding experts count as -inf), top-k, for the
        // two token rows of this lane in turn
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int64_t t = tbeg + cw * 16 + g + 8 * half;
            float gv[2 * NT], pv[2 * NT];
            float m = -INFINITY;
#pragma unroll
            for (int i = 0; i < 2 * NT; ++i) {
                const int e = (i >> 1) * 8 + 2 * c + (i & 1);
                gv[i] = e < E ? acc[i >> 1][2 * half + (i & 1)] : -INFINITY;
                m = fmaxf(m, gv[i]);
            }
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
            m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
            float z = 0.f;
#pragma unroll
            for (int i = 0; i < 2 * NT; ++i) {
                pv[i] = expf(gv[i] - m);
                z += pv[i];
            }
            z += __shfl_xor_sync(0xffffffffu, z, 1);
            z += __shfl_xor_sync(0xffffffffu, z, 2);
            // k rounds of "largest remaining logit, lowest index on ties"; weights are NOT
            // renormalised
            for (int j = 0; j < k; ++j) {
                float bg = gv[0], bp = pv[0];
                int be = 2 * c;
#pragma unroll
                for (int i = 1; i < 2 * NT; ++i) {
                    const int e = (i >> 1) * 8 + 2 * c + (i & 1);
                    if (gv[i] > bg) { bg = gv[i]; bp = pv[i]; be = e; }
                }
#pragma unroll
                for (int o = 1; o <= 2; o <<= 1) {
                    const float og = __shfl_xor_sync(0xffffffffu, bg, o);
                    const float op = __shfl_xor_sync(0xffffffffu, bp, o);
                    const int oe = __shfl_xor_sync(0xffffffffu, be, o);
                    if (og > bg || (og == bg && oe < be)) { bg = og; bp = op; be = oe; }
                }
#pragma unroll
                for (int i = 0; i < 2 * NT; ++i)
                    if ((i >> 1) * 8 + 2 * c + (i & 1) == be) gv[i] = -INFINITY;
                if (c == 0 && t < tend) {
                    idx[t * k + j] = be;
                    w[t * k + j] = bp / z;
                    if (counts) {
                        const int rank = atomicAdd(&sm->cnt[be], 1);
                        s_ent[(int)(t - tbeg) * k + j] = be | (rank << 8);
                    }
                }
            }
        }
        if (counts) {
            // lists: a shared-memory histogram ranked the tile's entries, one global atomic per
            // expert reserves the tile's range
            __syncthreads();
            if (tid < E) sm->base[tid] = atomicAdd(&counts[tid], sm->cnt[tid]);
            __syncthreads();
            const int n_ent = (int)(tend - tbeg) * k;
            for (int i = tid; i < n_ent; i += RS_THREADS) {
                const int ent = s_ent[i], e = ent & 255;
                perm[(int64_t)e * cap + sm->base[e] + (ent >> 8)] = (int)(tbeg * k + i);
            }
        }
    }
    // When launched behind the SSD step-size kernel (beside which it runs): this grid must not
    // complete before that one has, so that every later kernel in the stream is ordered behind both.
    grid_dep_wait();
}

// One expert: the softmax is identically 1 and every token is routed to expert 0.
__global__ void __launch_bounds__(256)
router_single_expert_kernel(int64_t Ttok, int32_t *__restrict__ idx, float *__restrict__ w,
                            int *__restrict__ counts, int *__restrict__ perm)
{
    grid_dep_launch();
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < Ttok;
         t += (int64_t)gridDim.x * blockDim.x) {
        idx[t] = 0;
        w[t] = 1.f;
        if (counts) perm[t] = (int)t;
    }
    if (counts && blockIdx.x == 0 && threadIdx.x == 0) counts[0] = (int)Ttok;
}

static int router_chunk(int64_t Ttok, int sm_count)
{
    // enough chunks to give every SM four blocks, between 32 and ROUTER_MAX_CHUNK tokens
    int chunk = (int)(Ttok / (4 * (int64_t)sm_count));
    chunk = (chunk + 31) / 32 * 32;
    if (chunk < 32) chunk = 32;
    if (chunk > ROUTER_MAX_CHUNK) chunk = ROUTER_MAX_CHUNK;
    return chunk;
}

static size_t router_stream_smem(int F, int NT, int k, int nstages)
{
    const int KB = ceil_div(F, RS_BK);
    return 1024 + (size_t)RS_CW * nstages * RS_STAGE_BYTES +
           (size_t)KB * (RS_BK / 16) * NT * 32 * sizeof(uint2) + (size_t)RS_TOK * k * sizeof(int) + 16 +
           sizeof(RouterStreamSmall);
}

// The streaming kernel needs rows that TMA can address (16-byte aligned base and row pitch), the
// fragment-ordered router matrix in shared memory and enough tiles to occupy the GPU.
static bool router_stream_usable(const void *u, int64_t Ttok, int F, int E, int sm_count)
{
    const int NT = E <= 8 ? 1 : E <= 16 ? 2 : E <= 32 ? 4 : 8;
    return E <= 64 && F >= RS_BOX && F % 8 == 0 && ((uintptr_t)u & 15) == 0 &&
           (size_t)ceil_div(F, RS_BK) * (RS_BK / 16) * NT * 32 * sizeof(uint2) <= 64 * 1024 &&
           ceil_div64(Ttok, RS_TOK) >= 3 * (int64_t)sm_count;
}

static int launch_router_stream(LaunchCtx &ctx, const __nv_bfloat16 *u, const __nv_bfloat16 *W_r,
                                int64_t Ttok, int F, int E, int k, int32_t *idx, float *w, int *counts,
                                int *perm, int64_t cap, int sm_count, void *zero_out,
                                int zero_bytes_per_token, bool behind_scalars)
{
    const int NT = E <= 8 ? 1 : E <= 16 ? 2 : E <= 32 ? 4 : 8;
    // ring depth: the deepest (up to RS_MAX_STAGES) that still lets two CTAs share an SM, else
    // the deepest that fits one
    int nstages = RS_MAX_STAGES, per_sm = 1;
    for (int ns = RS_MAX_STAGES; ns >= 2; --ns)
        if (2 * (router_stream_smem(F, NT, k, ns) + 1024) <= 227 * 1024) { nstages = ns; per_sm = 2; break; }
    const size_t smem = router_stream_smem(F, NT, k, nstages);
    CUtensorMap tmap;
    const uint64_t dims[2] = {(uint64_t)F, (uint64_t)Ttok};
    const uint64_t strides[1] = {(uint64_t)F * 2};
    const uint32_t box[2] = {(uint32_t)RS_BOX, 16u};
    if (!encode_tmap_bf16_cached(ctx.tmaps, &tmap, u, 2, dims, strides, box)) return SWIMBA_ERR_CUDA;
    const int64_t ntiles = ceil_div64(Ttok, RS_TOK);
    int64_t ctas = (int64_t)sm_count * per_sm;
    if (ctas > ntiles) ctas = ntiles;
    ctx.begin(STAGE_ROUTER);
#define SWIMBA_ROUTER_STREAM_CASE(NTV)                                                          \
    do {                                                                                        \
        auto kern = router_stream_kernel<NTV>;                                                  \
        if (!ensure_dynamic_smem((const void *)kern,             \
                                 smem))                                     \
            return SWIMBA_ERR_CUDA;                                                             \
        launch_kernel(kern, dim3((unsigned)ctas), dim3(RS_THREADS), smem, ctx.stream, behind_scalars, tmap, \
                      W_r, Ttok, F, E, k, idx, w, counts, perm, cap, (uint4 *)zero_out,         \
                      zero_bytes_per_token / 16, (int)ctas, nstages, ctx.d_status);             \
    } while (0)
    if (NT == 1) SWIMBA_ROUTER_STREAM_CASE(1);
    else if (NT == 2) SWIMBA_ROUTER_STREAM_CASE(2);
    else if (NT == 4) SWIMBA_ROUTER_STREAM_CASE(4);
    else SWIMBA_ROUTER_STREAM_CASE(8);
#undef SWIMBA_ROUTER_STREAM_CASE
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

static int launch_router_mma(LaunchCtx &ctx, const __nv_bfloat16 *u, const __nv_bfloat16 *W_r,
                             int64_t Ttok, int F, int E, int k, int32_t *idx, float *w, int *counts,
                             int *perm, int64_t cap, int sm_count, void *zero_out,
                             int zero_bytes_per_token, const ScalarsArgs &scalars)
{
    const int NT = E <= 8 ? 1 : E <= 16 ? 2 : E <= 32 ? 4 : 8;
    const int chunk = router_chunk(Ttok, sm_count);
    const int64_t extra = scalars_blocks(scalars, 256);      // leading blocks for the SSD step sizes
    const size_t w_bytes = (size_t)NT * 8 * (F * 2 + 64);
    const int stage_w = w_bytes <= 64 * 1024 ? 1 : 0;
    const size_t smem = (((size_t)chunk * k * sizeof(int) + 15) & ~(size_t)15) +
                        (size_t)RM_TOK * RM_KSPLIT * NT * 8 * sizeof(float) + (stage_w ? w_bytes : 0);
    int64_t blocks = ceil_div64(Ttok, chunk);
    const int64_t cap_blocks = (int64_t)sm_count * (smem > 40 * 1024 ? 2 : 4);
    if (blocks > cap_blocks) blocks = cap_blocks;
    ctx.begin(STAGE_ROUTER);
#define SWIMBA_ROUTER_MMA_CASE(NTV)                                                             \
    do {                                                                                        \
        auto kern = router_mma_kernel<NTV>;                                                     \
        if (smem > 32 * 1024 &&  /* static shared memory counts toward the 48 KB default */     \
            !ensure_dynamic_smem((const void *)kern,             \
                                 smem))                                     \
            return SWIMBA_ERR_CUDA;                                                             \
        launch_kernel(kern, dim3((unsigned)(extra + blocks)), dim3(256), smem, ctx.stream, false, \
                      u, W_r, Ttok, F, E, k, idx, w, counts, perm, cap, stage_w, chunk,         \
                      (uint4 *)zero_out, zero_bytes_per_token / 16, (int)blocks, (int)extra,    \
                      scalars);                                                                 \
    } while (0)
    if (NT == 1) SWIMBA_ROUTER_MMA_CASE(1);
    else if (NT == 2) SWIMBA_ROUTER_MMA_CASE(2);
    else if (NT == 4) SWIMBA_ROUTER_MMA_CASE(4);
    else SWIMBA_ROUTER_MMA_CASE(8);
#undef SWIMBA_ROUTER_MMA_CASE
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

template <typename T>
static int launch_router_t(LaunchCtx &ctx, const T *u, const T *W_r, int64_t Ttok, int F, int E,
                           int k, int32_t *idx, float *w, int *counts, int *perm, int64_t cap,
                           int sm_count, void *zero_out, int zero_bytes_per_token,
                           const ScalarsArgs &scalars)
{
    const int warps = 8;
    // The SSD step sizes of the same call (scalars.l2 != NULL) depend on dt only and run beside the
    // router: as the leading blocks of the register-fed tensor-core kernel, else as a kernel of
    // their own in front of the router (the streaming router then starts while it runs).
    bool behind_scalars = false;
    if constexpr (std::is_same<T, __nv_bfloat16>::value) {
        if (E > 1 && !router_stream_usable(u, Ttok, F, E, sm_count) && F % (32 * RM_KSPLIT) == 0 && E <= 64)
            return launch_router_mma(ctx, u, W_r, Ttok, F, E, k, idx, w, counts, perm, cap, sm_count,
                                     zero_out, zero_bytes_per_token, scalars);
        behind_scalars = E > 1 && scalars.l2 && router_stream_usable(u, Ttok, F, E, sm_count);
    }
    if (scalars.l2) {
        const int rc = launch_ssd_scalars(ctx, scalars);
        if (rc != SWIMBA_OK) return rc;
    }
    if (E == 1) {
        int64_t blocks = ceil_div64(Ttok, 256);
        if (blocks > (int64_t)sm_count * 8) blocks = (int64_t)sm_count * 8;
        ctx.begin(STAGE_ROUTER);
        launch_kernel(router_single_expert_kernel, dim3((unsigned)blocks), dim3(256), 0, ctx.stream,
                      false, Ttok, idx, w, counts, perm);
        ctx.end();
        return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
    }
    if constexpr (std::is_same<T, __nv_bfloat16>::value) {
        if (router_stream_usable(u, Ttok, F, E, sm_count))
            return launch_router_stream(ctx, u, W_r, Ttok, F, E, k, idx, w, counts, perm, cap, sm_count,
                                        zero_out, zero_bytes_per_token, behind_scalars);
    }
    const size_t w_bytes = (size_t)E * F * sizeof(T);
    const int stage_w = (w_bytes <= 64 * 1024 && (w_bytes & 15) == 0) ? 1 : 0;
    const size_t smem = (size_t)ROUTER_MAX_CHUNK * SWIMBA_MAX_TOPK * sizeof(int) + (stage_w ? w_bytes : 0);
    const int chunk = router_chunk(Ttok, sm_count);
    ctx.begin(STAGE_ROUTER);
#define SWIMBA_ROUTER_CASE(EPV, TPWV)                                                          \
    do {                                                                                       \
        auto kern = router_topk_kernel<T, EPV, TPWV>;                                          \
        if (smem > 32 * 1024 &&  /* static shared memory counts toward the 48 KB default */    \
            !ensure_dynamic_smem((const void *)kern,            \
                                 smem))                                    \
            return SWIMBA_ERR_CUDA;                                                            \
        int64_t blocks = ceil_div64(Ttok, chunk);                                              \
        const int64_t cap_blocks = (int64_t)sm_count * (smem > 40 * 1024 ? 2 : 4);             \
        if (blocks > cap_blocks) blocks = cap_blocks;                                          \
        launch_kernel(kern, dim3((unsigned)blocks), dim3(warps * 32), smem, ctx.stream, false,   \
                      u, W_r, Ttok, F, E, k, idx, w, counts, perm, cap, stage_w, chunk,        \
                      (uint4 *)zero_out, zero_bytes_per_token / 16, (int)blocks);              \
    } while (0)
    if (E <= 2) SWIMBA_ROUTER_CASE(2, 8);
    else if (E <= 4) SWIMBA_ROUTER_CASE(4, 8);
    else if (E <= 8) SWIMBA_ROUTER_CASE(8, 4);
    else if (E <= 16) SWIMBA_ROUTER_CASE(16, 2);
    else if (E <= 32) SWIMBA_ROUTER_CASE(32, 1);
    else SWIMBA_ROUTER_CASE(64, 1);
#undef SWIMBA_ROUTER_CASE
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

int launch_router(LaunchCtx &ctx, int dtype, const void *u, const void *W_r, int64_t T, int F,
                  int E, int k, int32_t *idx, float *w, int *counts, int *perm, int64_t cap,
                  int sm_count, void *zero_out, int zero_bytes_per_token, const ScalarsArgs &scalars)
{
    if (T <= 0) return SWIMBA_OK;
    if (dtype == SWIMBA_DTYPE_FP32)
        return launch_router_t<float>(ctx, (const float *)u, (const float *)W_r, T, F, E, k, idx, w,
                                      counts, perm, cap, sm_count, zero_out, zero_bytes_per_token, scalars);
    return launch_router_t<__nv_bfloat16>(ctx, (const __nv_bfloat16 *)u,
                                          (const __nv_bfloat16 *)W_r, T, F, E, k, idx, w, counts,
                                          perm, cap, sm_count, zero_out, zero_bytes_per_token, scalars);
}

// One warp per (token, block of RW stream rows): BC[t, r] = sum_j w_j <W_e[e_j, r, :], u_t>.
// Only the k selected experts are touched.
template <typename T, typename TO, int RW>
__global__ void __launch_bounds__(256)
project_mix_simt_kernel(const T *__restrict__ u, const T *__restrict__ W_e,
                        const int32_t *__restrict__ idx, const float *__restrict__ w, int64_t Ttok,
                        int F, int S, int k, TO *__restrict__ BC, int E, int check, int *d_status,
                        int kst, int joff)
{
    // (kst, joff): the k experts of token t are entries t*kst + joff .. + k - 1 of idx / w and the
    // output row is t*(kst/k) + joff/k ... used with k = 1, joff = j to write unmixed slots
    const int lane = threadIdx.x & 31;
    const int nblk = ceil_div(S, RW);
    const int64_t wid = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (wid >= Ttok * nblk) return;
    const int64_t t = wid / nblk;
    const int r0 = (int)(wid % nblk) * RW;
    int ej[SWIMBA_MAX_TOPK];
    float wj[SWIMBA_MAX_TOPK];
#pragma unroll
    for (int j = 0; j < SWIMBA_MAX_TOPK; ++j) {
        ej[j] = (j < k) ? idx[t * kst + joff + j] : 0;
        wj[j] = (j < k) ? w[t * kst + joff + j] : 0.f;
        if (check && (ej[j] < 0 || ej[j] >= E)) {      // a bad expert index is skipped, not followed
            if (lane == 0) atomicCAS(d_status, 0, SWIMBA_ERR_DEVICE_BOUNDS);
            ej[j] = 0;
            wj[j] = 0.f;
        }
    }
    float acc[RW];
#pragma unroll
    for (int r = 0; r < RW; ++r) acc[r] = 0.f;
    const T *urow = u + t * F;
    for (int f = lane * 8; f < F; f += 256) {
        float uv[8];
        load8(urow + f, uv);
#pragma unroll
        for (int j = 0; j < SWIMBA_MAX_TOPK; ++j) {
            if (j < k) {
                float us[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) us[i] = wj[j] * uv[i];
                const T *wbase = W_e + ((int64_t)ej[j] * S + r0) * F + f;
#pragma unroll
                for (int r = 0; r < RW; ++r) {
                    if (r0 + r < S) {
                        float wv[8];
                        load8(wbase + (int64_t)r * F, wv);
#pragma unroll
                        for (int i = 0; i < 8; ++i) acc[r] = fmaf(wv[i], us[i], acc[r]);
                    }
                }
            }
        }
    }
    float mine = 0.f;
#pragma unroll
    for (int r = 0; r < RW; ++r) {
        const float s = warp_sum(acc[r]);
        if (lane == r) mine = s;
    }
    const int64_t orow = (kst == k) ? t : t * kst + joff;
    if (lane < RW && r0 + lane < S) BC[orow * S + r0 + lane] = from_f32<TO>(mine);
}

template <typename T, typename TO>
static int launch_pm(LaunchCtx &ctx, const void *u, const void *W_e, const int32_t *idx,
                     const float *w, int64_t T_, int F, int S, int E, int k, void *BC, int kst = -1,
                     int joff = 0)
{
    if (kst < 0) kst = k;
    constexpr int RW = 16;
    const int warps = 8;
    const int64_t nw = T_ * ceil_div(S, RW);
    dim3 grid((unsigned)ceil_div64(nw, warps)), block(warps * 32);
    ctx.begin(STAGE_PROJECT_SIMT);
    project_mix_simt_kernel<T, TO, RW><<<grid, block, 0, ctx.stream>>>(
        (const T *)u, (const T *)W_e, idx, w, T_, F, S, k, (TO *)BC, E, ctx.check_indices ? 1 : 0, ctx.d_status,
        kst, joff);
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

int launch_project_mix_simt(LaunchCtx &ctx, int dtype, const void *u, const void *W_e,
                            const int32_t *idx, const float *w, int64_t T, int F, int S, int E,
                            int k, void *BC, bool bc_fp32)
{
    if (T <= 0) return SWIMBA_OK;
    if (dtype == SWIMBA_DTYPE_FP32) return launch_pm<float, float>(ctx, u, W_e, idx, w, T, F, S, E, k, BC);
    if (bc_fp32) return launch_pm<__nv_bfloat16, float>(ctx, u, W_e, idx, w, T, F, S, E, k, BC);
    return launch_pm<__nv_bfloat16, __nv_bfloat16>(ctx, u, W_e, idx, w, T, F, S, E, k, BC);
}

int launch_project_slots_simt(LaunchCtx &ctx, int dtype, const void *u, const void *W_e,
                              const int32_t *idx, const float *w, int64_t T, int F, int S, int E,
                              int k, void *slots_out)
{
    if (T <= 0) return SWIMBA_OK;
    for (int j = 0; j < k; ++j) {
        const int rc = dtype == SWIMBA_DTYPE_FP32
            ? launch_pm<float, float>(ctx, u, W_e, idx, w, T, F, S, E, 1, slots_out, k, j)
            : launch_pm<__nv_bfloat16, __nv_bfloat16>(ctx, u, W_e, idx, w, T, F, S, E, 1, slots_out, k, j);
        if (rc != SWIMBA_OK) return rc;
    }
    return SWIMBA_OK;
}

// BCj[t, :] = [ slots[t*k + j, 0:half] | sum_j' slots[t*k + j', half:S] ]: slot j's own injection
// stream beside the readout stream mixed over all slots (the slots already carry their weights).
template <typename T>
__global__ void __launch_bounds__(256)
assemble_slot_streams_kernel(const T *__restrict__ slots, int64_t Ttok, int S, int k, int j, T *__restrict__ BCj)
{
    const int half = S >> 1;
    const int64_t n = Ttok * S;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t t = i / S;
        const int c = (int)(i % S);
        float v;
        if (c < half) {
            v = to_f32<T>(slots[(t * k + j) * S + c]);
        } else {
            v = 0.f;
            for (int q = 0; q < k; ++q) v += to_f32<T>(slots[(t * k + q) * S + c]);
        }
        BCj[i] = from_f32<T>(v);
    }
}

int launch_assemble_slot_streams(LaunchCtx &ctx, int dtype, const void *slots, int64_t T, int S, int k,
                                 int j, void *BCj)
{
    if (T <= 0) return SWIMBA_OK;
    int64_t blocks = ceil_div64(T * S, 256);
    if (blocks > 148 * 16) blocks = 148 * 16;
    ctx.begin(STAGE_SLOT_STREAMS);
    if (dtype == SWIMBA_DTYPE_FP32)
        assemble_slot_streams_kernel<float><<<(unsigned)blocks, 256, 0, ctx.stream>>>((const float *)slots, T, S, k, j, (float *)BCj);
    else
        assemble_slot_streams_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, ctx.stream>>>(
            (const __nv_bfloat16 *)slots, T, S, k, j, (__nv_bfloat16 *)BCj);
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

// y += y_add (sum in fp32, stored in T), h += h_add
template <typename T>
__global__ void __launch_bounds__(256)
accumulate_kernel(T *__restrict__ y, const T *__restrict__ y_add, int64_t ny, float *__restrict__ h,
                  const float *__restrict__ h_add, int64_t nh)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x, i0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (y && y_add)
        for (int64_t i = i0; i < ny; i += stride) y[i] = from_f32<T>(to_f32<T>(y[i]) + to_f32<T>(y_add[i]));
    if (h && h_add)
        for (int64_t i = i0; i < nh; i += stride) h[i] += h_add[i];
}

int launch_accumulate(LaunchCtx &ctx, int dtype, void *y, const void *y_add, int64_t ny, float *h,
                      const float *h_add, int64_t nh)
{
    const int64_t n = ny > nh ? ny : nh;
    if (n <= 0) return SWIMBA_OK;
    int64_t blocks = ceil_div64(n, 256);
    if (blocks > 148 * 16) blocks = 148 * 16;
    ctx.begin(STAGE_SLOT_SUM);
    if (dtype == SWIMBA_DTYPE_FP32)
        accumulate_kernel<float><<<(unsigned)blocks, 256, 0, ctx.stream>>>((float *)y, (const float *)y_add, ny, h, h_add, nh);
    else
        accumulate_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, ctx.stream>>>(
            (__nv_bfloat16 *)y, (const __nv_bfloat16 *)y_add, ny, h, h_add, nh);
    ctx.end();
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

}  // namespace swimba
