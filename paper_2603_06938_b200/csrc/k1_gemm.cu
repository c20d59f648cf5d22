// K1 (tensor-core part): the expert stream projection as a grouped GEMM on tcgen05.
//
// Tokens are grouped by selected expert (only the k active experts of a token are ever
// projected, so the cost does not grow with E: Theorem 2).  For every (expert, 256-row tile)
// one CTA computes  D[256, BN] = U_rows[256, F] * W_e[e][n0:n0+BN, :]^T  (two 128-row MMA halves)
// with the gathered token rows as the K-major A operand and the expert's weight rows as the
// K-major B operand, scales
// row r by its router weight pi_{t,e} (Theorem 1's mixed streams).  With two active experts per
// token the scaled row is added straight into the token's row of the mixed streams (zeroed by the
// router kernel): 0 + a + b in bf16 is the same whichever slot arrives first, so the result is
// reproducible and no slot buffer is needed.  With more experts the order of the additions would
// matter: the rows go to slots (t, j) and a last streaming kernel sums them in a fixed order.
#include "internal.h"
#include "tc05.cuh"

namespace swimba {

namespace {
constexpr int GM_BM = 256;     // rows (token, slot pairs) per tile: two 128-row MMA halves that
                               // share every weight tile
constexpr int GM_BK = 64;      // features per pipeline stage (128 bytes of bf16)
constexpr int GM_LAG = 2;      // cp.async groups kept in flight per gather thread
constexpr int GM_THREADS = 192;
__host__ __device__ constexpr int gm_stages(int BN) { return BN >= 256 ? 3 : 4; }
}  // namespace

// ------------------------------------------------------------------------------------------
// Grouped GEMM.  Warps 0-3: gather the A rows with cp.async, later the epilogue; warp 4: TMA
// loads of the weight tile; warp 5: TMEM allocation and MMA issue.
// ------------------------------------------------------------------------------------------
template <int BN>
__global__ void __launch_bounds__(GM_THREADS, 1)
expert_gemm_kernel(const __grid_constant__ CUtensorMap tmap_w, const __nv_bfloat16 *__restrict__ u,
                   const int *__restrict__ perm, int64_t cap, const float *__restrict__ w_slot,
                   const int *__restrict__ counts, int E, int F, int S, int k, int add_rows,
                   __nv_bfloat16 *__restrict__ out, int *d_status, int check)
{
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr int STAGES = gm_stages(BN);
    constexpr uint32_t A_BYTES = GM_BM * 128, B_BYTES = BN * 128;
    constexpr uint32_t TMEM_COLS = 2 * BN < 32 ? 32 : 2 * BN;

    extern __shared__ uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t *sA = smem;
    uint8_t *sB = smem + STAGES * A_BYTES;
    uint64_t *full = (uint64_t *)(sB + STAGES * B_BYTES);
    uint64_t *empty = full + STAGES;
    uint64_t *acc_bar = empty + STAGES;
    uint32_t *tmem_slot = (uint32_t *)(acc_bar + 1);
    int *abort_flag = (int *)(tmem_slot + 1);
    int *row_src = abort_flag + 1;            // [256] token index or -1
    int *row_dst = row_src + GM_BM;           // [256] output row

    const int uwarp = __shfl_sync(0xffffffffu, warp, 0);   // warp-uniform for the compiler

    // Set-up that needs nothing from the router kernel; it may run under that kernel's tail.
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            tc::mbar_init(&full[s], 128 + 1);
            tc::mbar_init(&empty[s], 1);
        }
        tc::mbar_init(acc_bar, 1);
        *abort_flag = 0;
        tc::fence_mbar_init();
    }
    if (uwarp == 5) {
        tc::tmem_alloc(tmem_slot, TMEM_COLS);
        tc::tmem_relinquish();
    }
    if (uwarp == 4 && lane == 0) tc::prefetch_tmap(&tmap_w);
    grid_dep_launch();
    grid_dep_wait();        // counts, lists and weights come from the router kernel

    // Tile -> (expert, rows): tiles are numbered expert by expert, ceil(counts[e] / GM_BM) each.
    // Every warp finds its tile with one load per lane and a shuffle scan.
    int e = -1, row0 = 0, cnt = 0;
    {
        int before = 0;
        for (int base = 0; base < E && e < 0; base += 32) {
            int c = (base + lane < E) ? counts[base + lane] : 0;
            if (check && (c < 0 || c > cap)) {          // a list cannot be longer than its capacity
                atomicCAS(d_status, 0, SWIMBA_ERR_DEVICE_BOUNDS);
                c = 0;
            }
            const int nt = (c + GM_BM - 1) / GM_BM;
            int incl = nt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int nb = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += nb;
            }
            const unsigned hit = __ballot_sync(0xffffffffu, before + incl > (int)blockIdx.x);
            if (hit) {
                const int src = __ffs(hit) - 1;
                e = base + src;
                cnt = __shfl_sync(0xffffffffu, c, src);
                const int excl = __shfl_sync(0xffffffffu, incl - nt, src);
                row0 = ((int)blockIdx.x - before - excl) * GM_BM;
            }
            before += __shfl_sync(0xffffffffu, incl, 31);
        }
    }
    const bool has_tile = e >= 0;                   // (the grid is sized for the worst case)
    const int nrows = has_tile ? min(GM_BM, cnt - row0) : 0;
    const int nhalf = nrows > 128 ? 2 : 1;          // 128-row halves that hold rows
    if (has_tile) perm += (int64_t)e * cap;
    const int n0 = blockIdx.y * BN;
    for (int r = tid; r < GM_BM; r += GM_THREADS) {
        if (r < nrows) {
            const int entry = perm[row0 + r];
            if (check && (entry < 0 || entry >= cap * k)) {  // entries are t * k + j with t < cap tokens
                atomicCAS(d_status, 0, SWIMBA_ERR_DEVICE_BOUNDS);
                row_src[r] = -1;
                row_dst[r] = 0;
                continue;
            }
            row_src[r] = entry / k;
            row_dst[r] = add_rows ? entry / k : entry;      // token row, or slot row
        } else {
            row_src[r] = -1;
            row_dst[r] = 0;
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    if (!has_tile) {
        if (uwarp == 5) tc::tmem_dealloc(tmem_base, TMEM_COLS);
        return;
    }
    const int KB = ceil_div(F, GM_BK);

    if (uwarp < 4) {
        // ---- gather producers: thread -> 16-byte chunk (lane & 7) of rows 4 i + (lane >> 3)
        // of its warp's 64-row quarter
        int tsrc[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) tsrc[i] = row_src[warp * 64 + i * 4 + (lane >> 3)];
        for (int kb = 0; kb < KB; ++kb) {
            const int s = kb % STAGES;
            tc::mbar_wait(&empty[s], ((kb / STAGES) & 1) ^ 1, abort_flag, d_status);
            const uint32_t a_base = tc::smem_u32(sA + s * A_BYTES);
            const int chunk = lane & 7;
            const int f = kb * GM_BK + chunk * 8;
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int row = warp * 64 + i * 4 + (lane >> 3);
                const int t = tsrc[i];
                const bool ok = (t >= 0) && (f < F);
                const __nv_bfloat16 *src = ok ? (u + (int64_t)t * F + f) : u;
                tc::cp_async16(a_base + tc::sw128_offset(row, chunk), src, ok ? 16u : 0u);
            }
            tc::cp_async_commit();
            if (kb >= GM_LAG) {
                tc::cp_async_wait<GM_LAG>();
                tc::fence_proxy_async_smem();
                tc::mbar_arrive(&full[(kb - GM_LAG) % STAGES]);
            }
        }
        tc::cp_async_wait<0>();
        tc::fence_proxy_async_smem();
        for (int kb = (KB > GM_LAG ? KB - GM_LAG : 0); kb < KB; ++kb)
            tc::mbar_arrive(&full[kb % STAGES]);
        // router weights of the two rows this thread scales in the epilogue: a dependent pair of
        // loads, fetched here, under the last products, instead of in front of the first gather
        float wr2[2];
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
            const int row = hf * 128 + warp * 32 + lane;
            wr2[hf] = (row < nrows && row_src[row] >= 0) ? w_slot[perm[row0 + row]] : 0.f;
        }

        // ---- epilogue: thread = output row of each half.  All MMAs have completed, so the
        // pipeline buffers are free: the scaled bf16 rows are staged there (row stride padded by
        // 16 bytes against bank conflicts).  Rows that are added in place leave as one bulk
        // reduce-add each, issued half by half so that the second half is converted while the
        // first is on its way; rows that are stored are sent by the warp that staged them with
        // BN / 8 lanes per row, 16 bytes per lane (whole lines per instruction).
        tc::mbar_wait(acc_bar, 0, abort_flag, d_status);
        tc::tc_fence_after();
        constexpr uint32_t ROW_STRIDE = BN * 2 + 16;
        for (int hf = 0; hf < nhalf; ++hf) {
            const int row = hf * 128 + warp * 32 + lane;
            const float wr = wr2[hf];
            uint8_t *srow = smem + (uint32_t)row * ROW_STRIDE;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t v[32];
                tc::tmem_ld32(tmem_base + ((uint32_t)(warp * 32) << 16) + hf * BN + c * 32, v);
                tc::tmem_ld_wait();
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    pk[i] = tc::pack_bf16x2(wr * __uint_as_float(v[2 * i]),
                                            wr * __uint_as_float(v[2 * i + 1]));
                uint4 *dst = reinterpret_cast<uint4 *>(srow + c * 64);
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    dst[i] = make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
            }
            if (add_rows) {
                tc::fence_proxy_async_smem();
                if (row < nrows && row_src[row] >= 0)
                    tc::bulk_reduce_add_bf16(out + (int64_t)row_dst[row] * S + n0, srow, BN * 2);
                tc::bulk_commit_group();
            }
        }
        if (add_rows) tc::bulk_wait_read_all();
        __syncwarp();
        constexpr int LPR = BN / 8, RPI = 32 / LPR;      // lanes per row, rows per instruction
        const int sub = lane / LPR, piece = lane % LPR;
        for (int hf = 0; hf < (add_rows ? 0 : nhalf); ++hf) {
#pragma unroll 4
            for (int r0 = 0; r0 < 32; r0 += RPI) {
                const int row = hf * 128 + warp * 32 + r0 + sub;
                if (row < nrows && row_src[row] >= 0) {
                    const uint4 v = *reinterpret_cast<const uint4 *>(smem + (uint32_t)row * ROW_STRIDE + piece * 16);
                    __nv_bfloat16 *dst = out + (int64_t)row_dst[row] * S + n0 + piece * 8;
                    *reinterpret_cast<uint4 *>(dst) = v;
                }
            }
        }
    } else if (uwarp == 4) {
        // ---- weight tiles by TMA (whole warp in the loop, one elected lane issues)
        const bool leader = tc::elect_one();
        for (int kb = 0; kb < KB; ++kb) {
            const int s = kb % STAGES;
            tc::mbar_wait(&empty[s], ((kb / STAGES) & 1) ^ 1, abort_flag, d_status);
            if (leader) {
                tc::mbar_arrive_expect_tx(&full[s], B_BYTES);
                tc::tma_load_3d(sB + s * B_BYTES, &tmap_w, &full[s], kb * GM_BK, n0, e);
            }
            __syncwarp();
        }
    } else {
        // ---- MMA issue (whole warp in the loop, one elected lane issues)
        const bool leader = tc::elect_one();
        constexpr uint32_t idesc = tc::idesc_bf16(128, BN, 0, 0);
        const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0);
        const uint64_t dA0 = tc::smem_desc_sw128(tc::smem_u32(sA), 16, 1024);
        const uint64_t dB0 = tc::smem_desc_sw128(tc::smem_u32(sB), 16, 1024);
        for (int kb = 0; kb < KB; ++kb) {
            const int s = kb % STAGES;
            tc::mbar_wait(&full[s], (kb / STAGES) & 1, abort_flag, d_status);
            tc::tc_fence_after();
            if (leader) {
                const uint64_t dA = tc::smem_desc_advance(dA0, s * A_BYTES);
                const uint64_t dB = tc::smem_desc_advance(dB0, s * B_BYTES);
#pragma unroll
                for (int kk = 0; kk < GM_BK / 16; ++kk) {
                    const uint64_t bd = tc::smem_desc_advance(dB, kk * 32);
                    tc::mma_ss(tmem_u, tc::smem_desc_advance(dA, kk * 32), bd, idesc, (kb | kk) != 0);
                    if (nhalf > 1)
                        tc::mma_ss(tmem_u + BN, tc::smem_desc_advance(dA, 128 * 128 + kk * 32), bd, idesc,
                                   (kb | kk) != 0);
                }
                tc::mma_commit(&empty[s]);
            }
            __syncwarp();
        }
        if (leader) tc::mma_commit(acc_bar);
        __syncwarp();
    }
    tc::tc_fence_before();
    __syncthreads();
    if (uwarp == 5) tc::tmem_dealloc(tmem_base, TMEM_COLS);
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
    const int stages = gm_stages(BN);
    return 1024 + (size_t)stages * (GM_BM * 128 + BN * 128) + 8 * (2 * stages + 1) + 16 +
           GM_BM * 12 + 64;
}

// Workspace: [counts: 64 ints] [perm: E lists of capacity T] [slot outputs T*k*S bf16 when k > 1].
static size_t gemm_ws_up(size_t v) { return (v + 255) / 256 * 256; }

size_t expert_gemm_workspace_bytes(int64_t T, int S, int E, int k)
{
    size_t tot = gemm_ws_up(SWIMBA_MAX_EXPERTS * sizeof(int));
    tot += gemm_ws_up((size_t)E * T * sizeof(int));
    if (k > 1 && !expert_gemm_adds_rows(k)) tot += gemm_ws_up((size_t)T * k * S * sizeof(__nv_bfloat16));
    return tot;
}

int *expert_gemm_counts(void *workspace) { return (int *)workspace; }
int *expert_gemm_perm(void *workspace)
{
    return (int *)((char *)workspace + gemm_ws_up(SWIMBA_MAX_EXPERTS * sizeof(int)));
}

// k == 2: the two slots of a token are added in place (BC must be zero when the GEMM starts).
bool expert_gemm_adds_rows(int k) { return k == 2; }

bool expert_gemm_supported(int F, int S)
{
    return S % 32 == 0 && F >= 64;
}

int launch_expert_gemm(LaunchCtx &ctx, const void *u, const void *W_e, const float *w, int64_t T,
                       int F, int S, int E, int k, int sm_count, void *BC, void *workspace,
                       void *slots_out)
{
    if (T <= 0) return SWIMBA_OK;
    const int max_tiles = (int)ceil_div64(T * k, GM_BM) + E;
    int *counts = expert_gemm_counts(workspace);
    int *perm = expert_gemm_perm(workspace);
    // slots_out given: every (token, slot) projection goes to its own row there and nothing is mixed
    const int add_rows = (!slots_out && expert_gemm_adds_rows(k)) ? 1 : 0;
    __nv_bfloat16 *slots = slots_out ? (__nv_bfloat16 *)slots_out
        : (k > 1 && !add_rows)
        ? (__nv_bfloat16 *)((char *)perm + gemm_ws_up((size_t)E * T * sizeof(int)))
        : (__nv_bfloat16 *)BC;

    // Widest column tile that divides S; narrower when there are too few row tiles to fill the
    // GPU (decode-sized calls), so that the weight rows are spread over more SMs.
    int BN = 32;
    for (int c : {256, 128, 64}) if (S % c == 0) { BN = c; break; }
    while (BN > 32 && 2 * (int64_t)max_tiles * (S / BN) <= sm_count) BN >>= 1;

    CUtensorMap tmap;
    const uint64_t dims[3] = {(uint64_t)F, (uint64_t)S, (uint64_t)E};
    const uint64_t strides[2] = {(uint64_t)F * 2, (uint64_t)S * F * 2};
    const uint32_t box[3] = {(uint32_t)GM_BK, (uint32_t)BN, 1};
    if (!encode_tmap_bf16_cached(ctx.tmaps, &tmap, W_e, 3, dims, strides, box)) return SWIMBA_ERR_CUDA;

    const size_t smem = gemm_smem_bytes(BN);
    dim3 grid((unsigned)max_tiles, (unsigned)(S / BN));
#define SWIMBA_GEMM_CASE(BNV)                                                                   \
    do {                                                                                        \
        auto kern = expert_gemm_kernel<BNV>;                                                    \
        if (!ensure_dynamic_smem((const void *)kern, smem)) return SWIMBA_ERR_CUDA;             \
        launch_kernel(kern, grid, dim3(GM_THREADS), smem, ctx.stream, true, tmap,               \
                      (const __nv_bfloat16 *)u, (const int *)perm, (int64_t)T, (const float *)w, \
                      (const int *)counts, E, F, S, k, add_rows, slots, ctx.d_status,           \
                      ctx.check_indices ? 1 : 0);                                               \
    } while (0)
    ctx.begin(STAGE_EXPERT_GEMM);
    if (BN == 256) SWIMBA_GEMM_CASE(256);
    else if (BN == 128) SWIMBA_GEMM_CASE(128);
    else if (BN == 64) SWIMBA_GEMM_CASE(64);
    else SWIMBA_GEMM_CASE(32);
#undef SWIMBA_GEMM_CASE
    ctx.end();
    if (k > 1 && !add_rows && !slots_out) {
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
