// K1 (tensor-core part): the expert stream projection as a grouped GEMM on tcgen05.
//
// Tokens are grouped by selected expert (only the k active experts of a token are ever
// projected, so the cost does not grow with E: Theorem 2).  For every (expert, 128-row tile)
// one CTA computes  D[128, BN] = U_rows[128, F] * W_e[e][n0:n0+BN, :]^T  with the gathered token
// rows as the K-major A operand and the expert's weight rows as the K-major B operand, scales
// row r by its router weight pi_{t,e} (Theorem 1's mixed streams) and writes it to slot (t, j).
// A last streaming kernel sums the k slots of each token.
#include "internal.h"
#include "tc05.cuh"

namespace swimba {

namespace {
constexpr int GM_BM = 128;     // rows (token, slot pairs) per tile
constexpr int GM_BK = 64;      // features per pipeline stage (128 bytes of bf16)
constexpr int GM_STAGES = 4;
constexpr int GM_LAG = 2;      // cp.async groups kept in flight per gather thread
constexpr int GM_THREADS = 192;
}  // namespace

// ------------------------------------------------------------------------------------------
// Grouped GEMM.  Warps 0-3: gather the A rows with cp.async, later the epilogue; warp 4: TMA
// loads of the weight tile; warp 5: TMEM allocation and MMA issue.
// ------------------------------------------------------------------------------------------
template <int BN>
__global__ void __launch_bounds__(GM_THREADS, 1)
expert_gemm_kernel(const __grid_constant__ CUtensorMap tmap_w, const __nv_bfloat16 *__restrict__ u,
                   const int *__restrict__ perm, int64_t cap, const float *__restrict__ w_slot,
                   const int *__restrict__ counts, int E, int F, int S, int k,
                   __nv_bfloat16 *__restrict__ out, int *d_status)
{
    // Tile -> (expert, rows): tiles are numbered expert by expert, ceil(counts[e] / 128) each.
    int e = 0, row0 = (int)blockIdx.x, cnt = 0;
    for (; e < E; ++e) {
        cnt = counts[e];
        const int nt = (cnt + GM_BM - 1) / GM_BM;
        if (row0 < nt) break;
        row0 -= nt;
    }
    if (e == E) return;
    row0 *= GM_BM;
    const int nrows = min(GM_BM, cnt - row0);
    perm += (int64_t)e * cap;
    const int n0 = blockIdx.y * BN;
    constexpr uint32_t A_BYTES = GM_BM * 128, B_BYTES = BN * 128;
    constexpr uint32_t TMEM_COLS = BN < 32 ? 32 : BN;

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *sA = smem;
    uint8_t *sB = smem + GM_STAGES * A_BYTES;
    uint64_t *full = (uint64_t *)(sB + GM_STAGES * B_BYTES);
    uint64_t *empty = full + GM_STAGES;
    uint64_t *acc_bar = empty + GM_STAGES;
    uint32_t *tmem_slot = (uint32_t *)(acc_bar + 1);
    int *abort_flag = (int *)(tmem_slot + 1);
    int *row_src = abort_flag + 1;            // [128] token index or -1
    int *row_dst = row_src + GM_BM;           // [128] output row
    float *row_w = (float *)(row_dst + GM_BM);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < GM_STAGES; ++s) {
            tc::mbar_init(&full[s], 128 + 1);
            tc::mbar_init(&empty[s], 1);
        }
        tc::mbar_init(acc_bar, 1);
        *abort_flag = 0;
        tc::fence_mbar_init();
    }
    if (tid < GM_BM) {
        if (tid < nrows) {
            const int entry = perm[row0 + tid];
            row_src[tid] = entry / k;
            row_dst[tid] = entry;
            row_w[tid] = w_slot[entry];
        } else {
            row_src[tid] = -1;
            row_dst[tid] = 0;
            row_w[tid] = 0.f;
        }
    }
    if (warp == 5) {
        tc::tmem_alloc(tmem_slot, TMEM_COLS);
        tc::tmem_relinquish();
    }
    if (warp == 4 && lane == 0) tc::prefetch_tmap(&tmap_w);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const int KB = ceil_div(F, GM_BK);

    if (warp < 4) {
        // ---- gather producers
        for (int kb = 0; kb < KB; ++kb) {
            const int s = kb % GM_STAGES;
            tc::mbar_wait(&empty[s], ((kb / GM_STAGES) & 1) ^ 1, abort_flag, d_status);
            const uint32_t a_base = tc::smem_u32(sA + s * A_BYTES);
            const int chunk = lane & 7;
            const int f = kb * GM_BK + chunk * 8;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int row = warp * 32 + i * 4 + (lane >> 3);
                const int t = row_src[row];
                const bool ok = (t >= 0) && (f < F);
                const __nv_bfloat16 *src = ok ? (u + (int64_t)t * F + f) : u;
                tc::cp_async16(a_base + tc::sw128_offset(row, chunk), src, ok ? 16u : 0u);
            }
            tc::cp_async_commit();
            if (kb >= GM_LAG) {
                tc::cp_async_wait<GM_LAG>();
                tc::fence_proxy_async_smem();
                tc::mbar_arrive(&full[(kb - GM_LAG) % GM_STAGES]);
            }
        }
        tc::cp_async_wait<0>();
        tc::fence_proxy_async_smem();
        for (int kb = (KB > GM_LAG ? KB - GM_LAG : 0); kb < KB; ++kb)
            tc::mbar_arrive(&full[kb % GM_STAGES]);

        // ---- epilogue: thread = output row
        tc::mbar_wait(acc_bar, 0, abort_flag, d_status);
        tc::tc_fence_after();
        const int row = warp * 32 + lane;
        const bool valid = row < nrows;
        const float wr = row_w[row];
        __nv_bfloat16 *orow = out + (int64_t)row_dst[row] * S + n0;
#pragma unroll 1
        for (int c = 0; c < BN / 32; ++c) {
            uint32_t v[32];
            tc::tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + c * 32, v);
            tc::tmem_ld_wait();
            if (valid) {
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    pk[i] = tc::pack_bf16x2(wr * __uint_as_float(v[2 * i]),
                                            wr * __uint_as_float(v[2 * i + 1]));
                uint4 *dst = reinterpret_cast<uint4 *>(orow + c * 32);
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    dst[i] = make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
            }
        }
    } else if (warp == 4) {
        if (lane == 0) {
            for (int kb = 0; kb < KB; ++kb) {
                const int s = kb % GM_STAGES;
                tc::mbar_wait(&empty[s], ((kb / GM_STAGES) & 1) ^ 1, abort_flag, d_status);
                tc::mbar_arrive_expect_tx(&full[s], B_BYTES);
                tc::tma_load_3d(sB + s * B_BYTES, &tmap_w, &full[s], kb * GM_BK, n0, e);
            }
        }
    } else {
        if (lane == 0) {
            constexpr uint32_t idesc = tc::idesc_bf16(GM_BM, BN, 0, 0);
            for (int kb = 0; kb < KB; ++kb) {
                const int s = kb % GM_STAGES;
                tc::mbar_wait(&full[s], (kb / GM_STAGES) & 1, abort_flag, d_status);
                tc::tc_fence_after();
                const uint32_t a_addr = tc::smem_u32(sA + s * A_BYTES);
                const uint32_t b_addr = tc::smem_u32(sB + s * B_BYTES);
#pragma unroll
                for (int kk = 0; kk < GM_BK / 16; ++kk) {
                    const uint64_t ad = tc::smem_desc_sw128(a_addr + kk * 32, 16, 1024);
                    const uint64_t bd = tc::smem_desc_sw128(b_addr + kk * 32, 16, 1024);
                    tc::mma_ss(tmem_base, ad, bd, idesc, (kb | kk) != 0);
                }
                tc::mma_commit(&empty[s]);
            }
            tc::mma_commit(acc_bar);
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 5) tc::tmem_dealloc(tmem_base, TMEM_COLS);
}

// BC[t, :] = sum_j P[t*k + j, :]   (slots already carry their router weight).
__global__ void __launch_bounds__(256)
mix_slots_kernel(const __nv_bfloat16 *__restrict__ P, int64_t T, int S, int k,
                 __nv_bfloat16 *__restrict__ BC)
{
    const int vec_per_row = S >> 3;
    const int64_t nvec = T * vec_per_row;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < nvec;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t t = i / vec_per_row;
        const int v = (int)(i % vec_per_row);
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int j = 0; j < k; ++j) {
            float pv[8];
            load8(P + ((t * k + j) * S) + v * 8, pv);
#pragma unroll
            for (int q = 0; q < 8; ++q) acc[q] += pv[q];
        }
        uint4 o = make_uint4(tc::pack_bf16x2(acc[0], acc[1]), tc::pack_bf16x2(acc[2], acc[3]),
                             tc::pack_bf16x2(acc[4], acc[5]), tc::pack_bf16x2(acc[6], acc[7]));
        *reinterpret_cast<uint4 *>(BC + t * S + v * 8) = o;
    }
}

static size_t gemm_smem_bytes(int BN)
{
    return 1024 + GM_STAGES * (GM_BM * 128 + BN * 128) + 8 * (2 * GM_STAGES + 1) + 16 +
           GM_BM * 12 + 64;
}

// Workspace: [counts: 64 ints] [perm: E lists of capacity T] [slot outputs T*k*S bf16 when k > 1].
static size_t gemm_ws_up(size_t v) { return (v + 255) / 256 * 256; }

size_t expert_gemm_workspace_bytes(int64_t T, int S, int E, int k)
{
    size_t tot = gemm_ws_up(SWIMBA_MAX_EXPERTS * sizeof(int));
    tot += gemm_ws_up((size_t)E * T * sizeof(int));
    if (k > 1) tot += gemm_ws_up((size_t)T * k * S * sizeof(__nv_bfloat16));
    return tot;
}

int *expert_gemm_counts(void *workspace) { return (int *)workspace; }
int *expert_gemm_perm(void *workspace)
{
    return (int *)((char *)workspace + gemm_ws_up(SWIMBA_MAX_EXPERTS * sizeof(int)));
}

bool expert_gemm_supported(int F, int S)
{
    return S % 32 == 0 && F >= 64;
}

int launch_expert_gemm(LaunchCtx &ctx, const void *u, const void *W_e, const float *w, int64_t T,
                       int F, int S, int E, int k, int sm_count, void *BC, void *workspace)
{
    if (T <= 0) return SWIMBA_OK;
    const int max_tiles = (int)ceil_div64(T * k, GM_BM) + E;
    int *counts = expert_gemm_counts(workspace);
    int *perm = expert_gemm_perm(workspace);
    __nv_bfloat16 *slots = (k > 1)
        ? (__nv_bfloat16 *)((char *)perm + gemm_ws_up((size_t)E * T * sizeof(int)))
        : (__nv_bfloat16 *)BC;

    // Widest column tile that divides S; narrower when there are too few row tiles to fill the
    // GPU (decode-sized calls), so that the weight rows are spread over more SMs.
    int BN = 32;
    for (int c : {256, 128, 64}) if (S % c == 0) { BN = c; break; }
    while (BN > 32 && (int64_t)max_tiles * (S / BN) < sm_count) BN >>= 1;

    CUtensorMap tmap;
    const uint64_t dims[3] = {(uint64_t)F, (uint64_t)S, (uint64_t)E};
    const uint64_t strides[2] = {(uint64_t)F * 2, (uint64_t)S * F * 2};
    const uint32_t box[3] = {(uint32_t)GM_BK, (uint32_t)BN, 1};
    if (!encode_tmap_bf16(&tmap, W_e, 3, dims, strides, box)) return SWIMBA_ERR_CUDA;

    const size_t smem = gemm_smem_bytes(BN);
    dim3 grid((unsigned)max_tiles, (unsigned)(S / BN));
#define SWIMBA_GEMM_CASE(BNV)                                                                   \
    do {                                                                                        \
        auto kern = expert_gemm_kernel<BNV>;                                                    \
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != \
            cudaSuccess)                                                                        \
            return SWIMBA_ERR_CUDA;                                                             \
        kern<<<grid, GM_THREADS, smem, ctx.stream>>>(tmap, (const __nv_bfloat16 *)u, perm, T, w,  \
                                                     counts, E, F, S, k, slots, ctx.d_status);  \
    } while (0)
    ctx.begin(STAGE_EXPERT_GEMM);
    if (BN == 256) SWIMBA_GEMM_CASE(256);
    else if (BN == 128) SWIMBA_GEMM_CASE(128);
    else if (BN == 64) SWIMBA_GEMM_CASE(64);
    else SWIMBA_GEMM_CASE(32);
#undef SWIMBA_GEMM_CASE
    ctx.end();
    if (k > 1) {
        const int64_t nvec = T * (S / 8);
        int64_t blocks = ceil_div64(nvec, 256);
        if (blocks > (int64_t)sm_count * 16) blocks = (int64_t)sm_count * 16;
        ctx.begin(STAGE_MIX_SLOTS);
        mix_slots_kernel<<<(unsigned)blocks, 256, 0, ctx.stream>>>(slots, T, S, k,
                                                                  (__nv_bfloat16 *)BC);
        ctx.end();
    }
    return cudaGetLastError() == cudaSuccess ? SWIMBA_OK : SWIMBA_ERR_CUDA;
}

}  // namespace swimba
