// Host side of the C ABI: handle, argument validation, workspace layout and kernel sequencing.
#include <cstdio>
#include <cstring>
#include <new>

#include "internal.h"
#include "tc05.cuh"

using namespace swimba;

struct swimba_handle {
    swimba_config cfg;
    int device;
    int sm_count;
    int *d_status;          // device status word
    cudaStream_t last_stream;
    int last_launches;
    Profiler prof;
    TmapCache tmaps;        // tensor maps encoded so far (same buffers call after call: encoded once)
    // host-buffer entry point: copy streams and events of its batch-slice pipeline
    cudaStream_t s_in, s_out;
    cudaEvent_t ev_start, ev_out, ev_in[32], ev_done[32];
    char err[256];
};

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }
inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t elt_size(int dtype) { return dtype == SWIMBA_DTYPE_FP32 ? 4 : 2; }

int fail(swimba_handle *h, int code, const char *msg)
{
    if (h) snprintf(h->err, sizeof(h->err), "%s", msg);
    return code;
}

// Workspace of the forward: [BC | idx | w], each 256-byte aligned.
struct FwdLayout {
    size_t bc, idx, w, gemm, ssd, total;
};
bool use_tensor_k1(const swimba_config &c)
{
    return c.dtype == SWIMBA_DTYPE_BF16 && expert_gemm_supported(c.d_model, 2 * c.n_groups * c.d_state);
}
FwdLayout fwd_layout(const swimba_config &c, int B, int L, int sm_count)
{
    FwdLayout l;
    const int64_t T = (int64_t)B * L;
    const size_t S = 2u * c.n_groups * c.d_state;
    size_t off = 0;
    l.bc = off;  off += align_up((size_t)T * S * elt_size(c.dtype));
    l.idx = off; off += align_up((size_t)T * c.top_k * sizeof(int32_t));
    l.w = off;   off += align_up((size_t)T * c.top_k * sizeof(float));
    l.gemm = off;
    if (use_tensor_k1(c)) off += align_up(expert_gemm_workspace_bytes(T, (int)S, c.n_experts, c.top_k));
    l.ssd = off;
    if (ssd_tiles_supported(c.dtype, c.head_dim, c.d_state))
        off += align_up(ssd_workspace_bytes(B, L, c.n_heads, c.n_groups, c.chunk, sm_count));
    l.total = off;
    return l;
}

// Workspace of a decode step: [BC (bf16 on the tensor-core path, else fp32) | idx | w | GEMM scratch].
struct DecLayout {
    size_t bc, idx, w, gemm, total;
};
DecLayout dec_layout(const swimba_config &c, int B)
{
    DecLayout l;
    const size_t S = 2u * c.n_groups * c.d_state;
    size_t off = 0;
    l.bc = off;  off += align_up((size_t)B * S * sizeof(float));
    l.idx = off; off += align_up((size_t)B * c.top_k * sizeof(int32_t));
    l.w = off;   off += align_up((size_t)B * c.top_k * sizeof(float));
    l.gemm = off;
    if (use_tensor_k1(c)) off += align_up(expert_gemm_workspace_bytes(B, (int)S, c.n_experts, c.top_k));
    l.total = off;
    return l;
}

// Host-variant staging: [u | x | dt | y | h_final | idx | w] in front of the forward workspace.
struct HostLayout {
    size_t u, x, dt, y, hf, hf2, idx, w, fwd, total;
};
constexpr int kHostSlices = 8;     // batch slices of the host-buffer pipeline when there are that many sequences
constexpr int kHostPieces = 16;    // slices aimed at when sequences have to be cut along time instead
// A slice is `seqs` whole sequences, or (seqs == 1) a run of `piece` tokens of one sequence (a
// multiple of 256 tokens; the state is carried from run to run).  Slices start at byte offsets
// that keep the 16-byte alignment; where a per-sequence size does not, the batch goes as one slice.
struct HostPlan {
    int seqs, piece, pieces;      // sequences per slice, tokens per piece, pieces per sequence
};
inline HostPlan host_plan(const swimba_config &c, int B, int L)
{
    const size_t es = elt_size(c.dtype);
    const size_t per_seq[5] = {(size_t)L * c.d_model * es, (size_t)L * c.n_heads * c.head_dim * es,
                               (size_t)L * c.n_heads * sizeof(float),
                               (size_t)L * c.top_k * sizeof(int32_t),
                               (size_t)c.n_heads * c.head_dim * c.d_state * sizeof(float)};
    for (size_t v : per_seq)
        if (v % 16 != 0) return HostPlan{B, L, 1};
    if (B >= kHostSlices) return HostPlan{(B + kHostSlices - 1) / kHostSlices, L, 1};
    int want = (kHostPieces + B - 1) / B;
    int piece = ((L + want - 1) / want + 255) / 256 * 256;
    if (piece >= L) return HostPlan{1, L, 1};
    return HostPlan{1, piece, (L + piece - 1) / piece};
}

HostLayout host_layout(const swimba_config &c, int B, int L, int sm_count)
{
    HostLayout l;
    const size_t T = (size_t)B * L, es = elt_size(c.dtype);
    const size_t HP = (size_t)c.n_heads * c.head_dim;
    size_t off = 0;
    l.u = off;   off += align_up(T * c.d_model * es);
    l.x = off;   off += align_up(T * HP * es);
    l.dt = off;  off += align_up(T * c.n_heads * sizeof(float));
    l.y = off;   off += align_up(T * HP * es);
    l.hf = off;  off += align_up((size_t)B * HP * c.d_state * sizeof(float));
    l.hf2 = off; off += align_up((size_t)B * HP * c.d_state * sizeof(float));   // (carried states alternate)
    l.idx = off; off += align_up(T * c.top_k * sizeof(int32_t));
    l.w = off;   off += align_up(T * c.top_k * sizeof(float));
    // the forward runs slice by slice on the same scratch
    const HostPlan hp = host_plan(c, B, L);
    l.fwd = off; off += fwd_layout(c, hp.seqs, hp.piece, sm_count).total;
    l.total = off;
    return l;
}

int check_weights(swimba_handle *h, const swimba_weights *w, bool need_experts)
{
    if (!w) return fail(h, SWIMBA_ERR_NULL_ARG, "weights struct is NULL");
    if (!w->A || !w->dt_bias) return fail(h, SWIMBA_ERR_NULL_ARG, "A or dt_bias is NULL");
    if (need_experts) {
        if (!w->W_expert) return fail(h, SWIMBA_ERR_NULL_ARG, "W_expert is NULL");
        if (!w->W_router && h->cfg.n_experts > 1)
            return fail(h, SWIMBA_ERR_NULL_ARG, "W_router is NULL with more than one expert");
        if (!aligned16(w->W_expert) || !aligned16(w->W_router))
            return fail(h, SWIMBA_ERR_MISALIGNED, "weights must be 16-byte aligned");
    }
    if (!aligned16(w->A) || !aligned16(w->dt_bias) || !aligned16(w->D))
        return fail(h, SWIMBA_ERR_MISALIGNED, "A/dt_bias/D must be 16-byte aligned");
    return SWIMBA_OK;
}

bool create_host_pipeline(swimba_handle *h)
{
    bool ok = cudaStreamCreateWithFlags(&h->s_in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&h->s_out, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&h->ev_start, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&h->ev_out, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; ok && i < 32; ++i)
        ok = cudaEventCreateWithFlags(&h->ev_in[i], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&h->ev_done[i], cudaEventDisableTiming) == cudaSuccess;
    return ok;
}

void destroy_host_pipeline(swimba_handle *h)
{
    if (h->s_in) cudaStreamDestroy(h->s_in);
    if (h->s_out) cudaStreamDestroy(h->s_out);
    if (h->ev_start) cudaEventDestroy(h->ev_start);
    if (h->ev_out) cudaEventDestroy(h->ev_out);
    for (int i = 0; i < 32; ++i) {
        if (h->ev_in[i]) cudaEventDestroy(h->ev_in[i]);
        if (h->ev_done[i]) cudaEventDestroy(h->ev_done[i]);
    }
}

int set_device(swimba_handle *h)
{
    int cur = -1;
    if (cudaGetDevice(&cur) != cudaSuccess) return fail(h, SWIMBA_ERR_CUDA, "cudaGetDevice failed");
    if (cur != h->device) return fail(h, SWIMBA_ERR_CUDA, "handle used on a different device than it was created on");
    return SWIMBA_OK;
}

// Router + projection + mix into BC (dtype, or fp32 when bc_fp32).  scalars != NULL: the SSD step
// sizes of the same call (they depend on dt only) are produced beside the router.
int run_route_mix(swimba_handle *h, LaunchCtx &ctx, const swimba_weights *w, const void *u,
                  int64_t T, void *BC, bool bc_fp32, int32_t *idx, float *wt, void *gemm_ws,
                  const ScalarsArgs *scalars = nullptr)
{
    const swimba_config &c = h->cfg;
    const int S = 2 * c.n_groups * c.d_state;
    // With one expert the softmax is identically 1; the router kernel handles it without W_router
    // being dereferenced only if it is given, so substitute the expert matrix as a dummy operand.
    const void *Wr = w->W_router ? w->W_router : w->W_expert;
    const bool tensor = gemm_ws && !bc_fp32 && use_tensor_k1(c);
    int *counts = nullptr, *perm = nullptr;
    if (tensor) {
        counts = expert_gemm_counts(gemm_ws);
        perm = expert_gemm_perm(gemm_ws);
        if (cudaMemsetAsync(counts, 0, sizeof(int) * SWIMBA_MAX_EXPERTS, ctx.stream) != cudaSuccess)
            return fail(h, SWIMBA_ERR_CUDA, "clearing the expert histogram failed");
    }
    const bool zero_bc = tensor && expert_gemm_adds_rows(c.top_k);
    int rc = launch_router(ctx, c.dtype, u, Wr, T, c.d_model, c.n_experts, c.top_k, idx, wt, counts,
                           perm, T, h->sm_count, zero_bc ? BC : nullptr, S * 2,
                           scalars ? *scalars : ScalarsArgs{});
    if (rc != SWIMBA_OK) return fail(h, rc, "router launch failed");
    if (tensor) {
        rc = launch_expert_gemm(ctx, u, w->W_expert, wt, T, c.d_model, S, c.n_experts, c.top_k,
                                h->sm_count, BC, gemm_ws);
        if (rc != SWIMBA_OK) return fail(h, rc, "expert GEMM launch failed");
        return SWIMBA_OK;
    }
    rc = launch_project_mix_simt(ctx, c.dtype, u, w->W_expert, idx, wt, T, c.d_model, S,
                                 c.n_experts, c.top_k, BC, bc_fp32);
    if (rc != SWIMBA_OK) return fail(h, rc, "projection launch failed");
    return SWIMBA_OK;
}

int run_ssd(swimba_handle *h, LaunchCtx &ctx, const swimba_weights *w, const void *x,
            const void *BC, const float *dt, const float *h0, int B, int L, void *y,
            float *h_final, void *ssd_ws, bool scalars_done = false)
{
    const swimba_config &c = h->cfg;
    if (ssd_ws && ssd_tiles_supported(c.dtype, c.head_dim, c.d_state)) {
        int rc = launch_ssd_tiles(ctx, x, BC, dt, w->A, w->dt_bias, w->D, h0, B, L, c.n_heads,
                                  c.n_groups, c.chunk, h->sm_count, y, h_final, ssd_ws, scalars_done);
        if (rc != SWIMBA_OK) return fail(h, rc, "SSD tile kernel launch failed");
        return SWIMBA_OK;
    }
    int rc = launch_ssd_sequential(ctx, c.dtype, x, BC, false, dt, w->A, w->dt_bias, w->D, h0, B, L,
                                   c.n_heads, c.head_dim, c.d_state, c.n_groups, y, h_final);
    if (rc != SWIMBA_OK) return fail(h, rc, "SSD launch failed");
    return SWIMBA_OK;
}

// The routing/projection stage with its scratch regions given one by one (idx_scratch / w_scratch
// are used when the caller does not ask for the routing outputs).
int route_mix_call(swimba_handle *h, const swimba_weights *w, const void *u, int64_t T, void *BC,
                   int32_t *topk_idx, float *topk_w, void *idx_scratch, void *w_scratch,
                   void *gemm_ws, void *cuda_stream)
{
    int rc = check_weights(h, w, true);
    if (rc != SWIMBA_OK) return rc;
    if (T == 0) { h->last_launches = 0; return SWIMBA_OK; }
    if (!u || !BC) return fail(h, SWIMBA_ERR_NULL_ARG, "u, BC or workspace is NULL");
    if (!aligned16(u) || !aligned16(BC) || !aligned16(idx_scratch) || !aligned16(w_scratch) ||
        !aligned16(gemm_ws) || !aligned16(topk_idx) || !aligned16(topk_w))
        return fail(h, SWIMBA_ERR_MISALIGNED, "tensors must be 16-byte aligned");
    if ((rc = set_device(h)) != SWIMBA_OK) return rc;
    LaunchCtx ctx{(cudaStream_t)cuda_stream, h->d_status, 0, &h->prof, (h->cfg.flags & SWIMBA_FLAG_CHECK_INDICES) != 0, &h->tmaps};
    h->prof.n = 0;
    int32_t *idx = topk_idx ? topk_idx : (int32_t *)idx_scratch;
    float *wt = topk_w ? topk_w : (float *)w_scratch;
    rc = run_route_mix(h, ctx, w, u, T, BC, false, idx, wt, gemm_ws);
    h->last_stream = ctx.stream;
    h->last_launches = ctx.launches;
    return rc;
}

}  // namespace

extern "C" {

int swimba_create(const swimba_config *cfg, swimba_handle **out)
{
    if (!cfg || !out) return SWIMBA_ERR_NULL_ARG;
    const swimba_config &c = *cfg;
    if (c.d_model <= 0 || c.n_heads <= 0 || c.head_dim <= 0 || c.d_state <= 0 || c.n_groups <= 0 ||
        c.n_experts <= 0 || c.top_k <= 0)
        return SWIMBA_ERR_BAD_CONFIG;
    if (c.n_heads % c.n_groups != 0) return SWIMBA_ERR_BAD_CONFIG;
    if (c.n_experts > SWIMBA_MAX_EXPERTS || c.top_k > c.n_experts || c.top_k > SWIMBA_MAX_TOPK)
        return SWIMBA_ERR_BAD_CONFIG;
    if (c.chunk != 64 && c.chunk != 128 && c.chunk != 256) return SWIMBA_ERR_BAD_CONFIG;
    if (c.dtype != SWIMBA_DTYPE_FP32 && c.dtype != SWIMBA_DTYPE_BF16) return SWIMBA_ERR_BAD_CONFIG;
    if ((c.flags & ~SWIMBA_FLAG_CHECK_INDICES) != 0) return SWIMBA_ERR_BAD_CONFIG;
    if (c.d_model % 8 != 0 || c.d_state % 16 != 0 || c.d_state > 256 || c.head_dim > 256)
        return SWIMBA_ERR_UNSUPPORTED_SHAPE;
    int ns = 1;
    while (ns * 16 < c.d_state) ns <<= 1;
    if (ns * c.head_dim > 1024) return SWIMBA_ERR_UNSUPPORTED_SHAPE;

    swimba_handle *h = new (std::nothrow) swimba_handle;
    if (!h) return SWIMBA_ERR_CUDA;
    memset(h, 0, sizeof(*h));
    h->cfg = c;
    if (cudaGetDevice(&h->device) != cudaSuccess ||
        cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device) != cudaSuccess ||
        cudaMalloc(&h->d_status, 64) != cudaSuccess || cudaMemset(h->d_status, 0, 64) != cudaSuccess ||
        !create_host_pipeline(h)) {
        destroy_host_pipeline(h);
        if (h->d_status) cudaFree(h->d_status);
        delete h;
        cudaGetLastError();
        return SWIMBA_ERR_CUDA;
    }
    *out = h;
    return SWIMBA_OK;
}

size_t swimba_workspace_bytes(const swimba_handle *h, int32_t B, int32_t L)
{
    if (!h || B <= 0 || L <= 0) return 0;
    return fwd_layout(h->cfg, B, L, h->sm_count).total;
}

int32_t swimba_ssd_segments(const swimba_handle *h, int32_t B, int32_t L)
{
    if (!h || B <= 0 || L <= 0) return 0;
    const swimba_config &c = h->cfg;
    if (!ssd_tiles_supported(c.dtype, c.head_dim, c.d_state)) return 1;
    const int seg_len = ssd_segment_len(B, L, c.n_heads, c.n_groups, c.chunk, h->sm_count);
    return (L + seg_len - 1) / seg_len;
}

size_t swimba_decode_workspace_bytes(const swimba_handle *h, int32_t B)
{
    if (!h || B <= 0) return 0;
    return dec_layout(h->cfg, B).total;
}

size_t swimba_host_workspace_bytes(const swimba_handle *h, int32_t B, int32_t L)
{
    if (!h || B <= 0 || L <= 0) return 0;
    return host_layout(h->cfg, B, L, h->sm_count).total;
}

int swimba_route_mix(swimba_handle *h, const swimba_weights *w, const void *u, int64_t T,
                     void *BC, int32_t *topk_idx, float *topk_w, void *workspace,
                     size_t workspace_bytes, void *cuda_stream)
{
    if (!h) return SWIMBA_ERR_NULL_ARG;
    h->err[0] = 0;
    // (token, slot) entries are indexed with 32-bit integers
    if (T < 0 || T * h->cfg.top_k >= (int64_t)1 << 31)
        return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "T out of range (T * top_k must stay below 2^31)");
    if (T > 0 && !workspace) return fail(h, SWIMBA_ERR_NULL_ARG, "u, BC or workspace is NULL");
    const FwdLayout l = fwd_layout(h->cfg, 1, (int)T, h->sm_count);
    if (T > 0 && workspace_bytes < l.ssd) return fail(h, SWIMBA_ERR_WORKSPACE_TOO_SMALL, "workspace too small");
    char *ws = (char *)workspace;
    return route_mix_call(h, w, u, T, BC, topk_idx, topk_w, ws + l.idx, ws + l.w, ws + l.gemm, cuda_stream);
}

int swimba_route_project_slots(swimba_handle *h, const swimba_weights *w, const void *u, int64_t T,
                               void *BC_slots, int32_t *topk_idx, float *topk_w, void *workspace,
                               size_t workspace_bytes, void *cuda_stream)
{
    if (!h) return SWIMBA_ERR_NULL_ARG;
    h->err[0] = 0;
    if (T < 0 || T * h->cfg.top_k >= (int64_t)1 << 31)
        return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "T out of range (T * top_k must stay below 2^31)");
    int rc = check_weights(h, w, true);
    if (rc != SWIMBA_OK) return rc;
    if (T == 0) { h->last_launches = 0; return SWIMBA_OK; }
    if (!u || !BC_slots || !workspace) return fail(h, SWIMBA_ERR_NULL_ARG, "u, BC_slots or workspace is NULL");
    if (!aligned16(u) || !aligned16(BC_slots) || !aligned16(workspace) || !aligned16(topk_idx) || !aligned16(topk_w))
        return fail(h, SWIMBA_ERR_MISALIGNED, "tensors must be 16-byte aligned");
    const swimba_config &c = h->cfg;
    const FwdLayout l = fwd_layout(c, 1, (int)T, h->sm_count);
    if (workspace_bytes < l.ssd) return fail(h, SWIMBA_ERR_WORKSPACE_TOO_SMALL, "workspace too small");
    if ((rc = set_device(h)) != SWIMBA_OK) return rc;
    char *ws = (char *)workspace;
    LaunchCtx ctx{(cudaStream_t)cuda_stream, h->d_status, 0, &h->prof, (c.flags & SWIMBA_FLAG_CHECK_INDICES) != 0, &h->tmaps};
    h->prof.n = 0;
    int32_t *idx = topk_idx ? topk_idx : (int32_t *)(ws + l.idx);
    float *wt = topk_w ? topk_w : (float *)(ws + l.w);
    const int S = 2 * c.n_groups * c.d_state;
    const void *Wr = w->W_router ? w->W_router : w->W_expert;
    const bool tensor = use_tensor_k1(c);
    int *counts = nullptr, *perm = nullptr;
    if (tensor) {
        counts = expert_gemm_counts(ws + l.gemm);
        perm = expert_gemm_perm(ws + l.gemm);
        if (cudaMemsetAsync(counts, 0, sizeof(int) * SWIMBA_MAX_EXPERTS, ctx.stream) != cudaSuccess)
            return fail(h, SWIMBA_ERR_CUDA, "clearing the expert histogram failed");
    }
    rc = launch_router(ctx, c.dtype, u, Wr, T, c.d_model, c.n_experts, c.top_k, idx, wt, counts, perm, T,
                       h->sm_count, nullptr, S * 2, ScalarsArgs{});
    if (rc != SWIMBA_OK) return fail(h, rc, "router launch failed");
    if (tensor)
        rc = launch_expert_gemm(ctx, u, w->W_expert, wt, T, c.d_model, S, c.n_experts, c.top_k, h->sm_count,
                                nullptr, ws + l.gemm, BC_slots);
    else
        rc = launch_project_slots_simt(ctx, c.dtype, u, w->W_expert, idx, wt, T, c.d_model, S, c.n_experts,
                                       c.top_k, BC_slots);
    if (rc != SWIMBA_OK) fail(h, rc, "projection launch failed");
    h->last_stream = ctx.stream;
    h->last_launches = ctx.launches;
    return rc;
}

size_t swimba_ssd_slots_workspace_bytes(const swimba_handle *h, int32_t B, int32_t L)
{
    if (!h || B <= 0 || L <= 0) return 0;
    const swimba_config &c = h->cfg;
    const size_t T = (size_t)B * L, es = elt_size(c.dtype);
    const size_t S = 2u * c.n_groups * c.d_state, HP = (size_t)c.n_heads * c.head_dim;
    // [forward workspace | BC of one slot | y of one slot | end state of one slot]
    return fwd_layout(c, B, L, h->sm_count).total + align_up(T * S * es) + align_up(T * HP * es) +
           align_up((size_t)B * HP * c.d_state * sizeof(float));
}

int swimba_ssd_slots(swimba_handle *h, const swimba_weights *w, const void *x_slots, const void *BC_slots,
                     const float *dt, const float *h0, int32_t B, int32_t L, void *y, float *h_final,
                     void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!h) return SWIMBA_ERR_NULL_ARG;
    h->err[0] = 0;
    if (B < 0 || L < 0) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "negative B or L");
    if (B > 65535) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "more than 65535 sequences per call");
    int rc = check_weights(h, w, false);
    if (rc != SWIMBA_OK) return rc;
    if (B == 0 || L == 0) { h->last_launches = 0; return SWIMBA_OK; }
    if (!x_slots || !BC_slots || !y || !workspace) return fail(h, SWIMBA_ERR_NULL_ARG, "x_slots, BC_slots, y or workspace is NULL");
    if (!aligned16(x_slots) || !aligned16(BC_slots) || !aligned16(y) || !aligned16(dt) || !aligned16(h0) ||
        !aligned16(h_final) || !aligned16(workspace))
        return fail(h, SWIMBA_ERR_MISALIGNED, "tensors must be 16-byte aligned");
    if (workspace_bytes < swimba_ssd_slots_workspace_bytes(h, B, L))
        return fail(h, SWIMBA_ERR_WORKSPACE_TOO_SMALL, "workspace too small");
    if ((rc = set_device(h)) != SWIMBA_OK) return rc;
    const swimba_config &c = h->cfg;
    const size_t T = (size_t)B * L, es = elt_size(c.dtype);
    const int S = 2 * c.n_groups * c.d_state, k = c.top_k;
    const size_t HP = (size_t)c.n_heads * c.head_dim;
    const FwdLayout l = fwd_layout(c, B, L, h->sm_count);
    char *ws = (char *)workspace;
    char *bcj = ws + l.total;
    char *ytmp = bcj + align_up(T * S * es);
    float *htmp = (float *)(ytmp + align_up(T * HP * es));
    LaunchCtx ctx{(cudaStream_t)cuda_stream, h->d_status, 0, &h->prof, (c.flags & SWIMBA_FLAG_CHECK_INDICES) != 0, &h->tmaps};
    h->prof.n = 0;
    // The injection is linear in (B^(e), X^(e)): the layer is the sum over the k slots of one
    // ordinary evaluation each, with slot j's own injection stream and input and the readout stream
    // mixed over all slots; the initial state enters through slot 0 only.  No skip term: the
    // paper's output equation has none, and with expert-specific inputs there is no single x.
    swimba_weights wj = *w;
    wj.D = nullptr;
    for (int j = 0; j < k && rc == SWIMBA_OK; ++j) {
        rc = launch_assemble_slot_streams(ctx, c.dtype, BC_slots, (int64_t)T, S, k, j, bcj);
        if (rc != SWIMBA_OK) { fail(h, rc, "slot stream launch failed"); break; }
        const char *xj = (const char *)x_slots + (size_t)j * T * HP * es;
        rc = run_ssd(h, ctx, &wj, xj, bcj, dt, j == 0 ? h0 : nullptr, B, L, j == 0 ? y : (void *)ytmp,
                     h_final ? (j == 0 ? h_final : htmp) : nullptr, ws + l.ssd);
        if (rc != SWIMBA_OK) break;
        if (j > 0) {
            rc = launch_accumulate(ctx, c.dtype, y, ytmp, (int64_t)(T * HP), h_final, h_final ? htmp : nullptr,
                                   (int64_t)B * HP * c.d_state);
            if (rc != SWIMBA_OK) fail(h, rc, "slot sum launch failed");
        }
    }
    h->last_stream = ctx.stream;
    h->last_launches = ctx.launches;
    return rc;
}

namespace {
// out[T,So] = in[T,Fi] W[So,Fi]^T as the grouped projection with a single expert (tensor cores
// where the shape allows, else the SIMT projection).  scratch: dense_scratch_bytes(T).
size_t dense_scratch_bytes(int64_t T)
{
    return align_up((size_t)T * sizeof(int32_t)) + align_up((size_t)T * sizeof(float)) +
           align_up(expert_gemm_workspace_bytes(T, 32, 1, 1));
}
int dense_linear(swimba_handle *h, LaunchCtx &ctx, const void *in, const void *W, int64_t T, int Fi, int So,
                 void *out, char *scratch)
{
    const int dtype = h->cfg.dtype;
    int32_t *idx = (int32_t *)scratch;
    float *wt = (float *)(scratch + align_up((size_t)T * sizeof(int32_t)));
    char *gws = (char *)wt + align_up((size_t)T * sizeof(float));
    const bool tensor = dtype == SWIMBA_DTYPE_BF16 && expert_gemm_supported(Fi, So);
    int *counts = nullptr, *perm = nullptr;
    if (tensor) {
        counts = expert_gemm_counts(gws);
        perm = expert_gemm_perm(gws);
        if (cudaMemsetAsync(counts, 0, sizeof(int) * SWIMBA_MAX_EXPERTS, ctx.stream) != cudaSuccess)
            return fail(h, SWIMBA_ERR_CUDA, "clearing the expert histogram failed");
    }
    // one expert: the router only writes idx = 0, w = 1 and the identity list (W stands in for the
    // router matrix, which is not read)
    int rc = launch_router(ctx, dtype, in, W, T, Fi, 1, 1, idx, wt, counts, perm, T, h->sm_count, nullptr, 0,
                           ScalarsArgs{});
    if (rc != SWIMBA_OK) return fail(h, rc, "list launch failed");
    rc = tensor ? launch_expert_gemm(ctx, in, W, wt, T, Fi, So, 1, 1, h->sm_count, out, gws)
                : launch_project_mix_simt(ctx, dtype, in, W, idx, wt, T, Fi, So, 1, 1, out, false);
    if (rc != SWIMBA_OK) return fail(h, rc, "linear map launch failed");
    return SWIMBA_OK;
}

struct BlockLayout {
    size_t zx, dtb, dt, bcp, x, bc, y, lin, fwd, total;
};
BlockLayout block_layout(const swimba_config &c, int B, int L, int sm_count)
{
    BlockLayout l;
    const size_t T = (size_t)B * L, es = elt_size(c.dtype);
    const size_t D = (size_t)c.n_heads * c.head_dim, S = 2u * c.n_groups * c.d_state;
    size_t off = 0;
    l.zx = off;  off += align_up(T * 2 * D * es);
    l.dtb = off; off += align_up(T * c.n_heads * es);
    l.dt = off;  off += align_up(T * c.n_heads * sizeof(float));
    l.bcp = off; off += align_up(T * S * es);
    l.x = off;   off += align_up(T * D * es);            // x, later the normalised gate output
    l.bc = off;  off += align_up(T * S * es);
    l.y = off;   off += align_up(T * D * es);
    l.lin = off; off += dense_scratch_bytes((int64_t)T);
    l.fwd = off; off += fwd_layout(c, B, L, sm_count).total;
    l.total = off;
    return l;
}
}  // namespace

size_t swimba_block_workspace_bytes(const swimba_handle *h, int32_t B, int32_t L)
{
    if (!h || B <= 0 || L <= 0) return 0;
    return block_layout(h->cfg, B, L, h->sm_count).total;
}

int swimba_block_forward(swimba_handle *h, const swimba_weights *w, const swimba_block_weights *bw,
                         const void *u, const void *conv_state_in, const float *h0, int32_t B, int32_t L,
                         void *out, void *conv_state_out, float *h_final, int32_t *topk_idx, float *topk_w,
                         void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!h) return SWIMBA_ERR_NULL_ARG;
    h->err[0] = 0;
    if (B < 0 || L < 0) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "negative B or L");
    if ((int64_t)B * L * h->cfg.top_k >= (int64_t)1 << 31)
        return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "too many tokens (B * L * top_k must stay below 2^31)");
    if (B > 65535) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "more than 65535 sequences per call");
    int rc = check_weights(h, w, true);
    if (rc != SWIMBA_OK) return rc;
    if (!bw || !bw->W_in || !bw->conv_w || !bw->norm_w || !bw->W_out)
        return fail(h, SWIMBA_ERR_NULL_ARG, "a block weight is NULL");
    if (bw->d_conv < 1 || bw->d_conv > 4) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "d_conv must lie in 1..4");
    const swimba_config &c = h->cfg;
    if (c.head_dim % 8 != 0) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "the block needs head_dim % 8 == 0");
    if (B == 0 || L == 0) { h->last_launches = 0; return SWIMBA_OK; }
    if (!u || !out || !workspace) return fail(h, SWIMBA_ERR_NULL_ARG, "u, out or workspace is NULL");
    if (!aligned16(u) || !aligned16(out) || !aligned16(conv_state_in) || !aligned16(conv_state_out) ||
        !aligned16(h0) || !aligned16(h_final) || !aligned16(topk_idx) || !aligned16(topk_w) ||
        !aligned16(workspace) || !aligned16(bw->W_in) || !aligned16(bw->W_out) || !aligned16(bw->conv_w) ||
        !aligned16(bw->conv_b) || !aligned16(bw->norm_w))
        return fail(h, SWIMBA_ERR_MISALIGNED, "tensors must be 16-byte aligned");
    const BlockLayout l = block_layout(c, B, L, h->sm_count);
    if (workspace_bytes < l.total) return fail(h, SWIMBA_ERR_WORKSPACE_TOO_SMALL, "workspace too small");
    if ((rc = set_device(h)) != SWIMBA_OK) return rc;
    const int64_t T = (int64_t)B * L;
    const size_t es = elt_size(c.dtype);
    const int D = c.n_heads * c.head_dim, S = 2 * c.n_groups * c.d_state, F = c.d_model, H = c.n_heads;
    char *ws = (char *)workspace;
    LaunchCtx ctx{(cudaStream_t)cuda_stream, h->d_status, 0, &h->prof, (c.flags & SWIMBA_FLAG_CHECK_INDICES) != 0, &h->tmaps};
    h->prof.n = 0;
    const FwdLayout fl = fwd_layout(c, B, L, h->sm_count);
    char *fws = ws + l.fwd;
    int32_t *idx = topk_idx ? topk_idx : (int32_t *)(fws + fl.idx);
    float *wt = topk_w ? topk_w : (float *)(fws + fl.w);
    // shared in-projection: [z | x'] (2 D columns) and the raw step sizes (H columns)
    rc = dense_linear(h, ctx, u, bw->W_in, T, F, 2 * D, ws + l.zx, ws + l.lin);
    if (rc == SWIMBA_OK)
        rc = dense_linear(h, ctx, u, (const char *)bw->W_in + (size_t)2 * D * F * es, T, F, H, ws + l.dtb, ws + l.lin);
    if (rc == SWIMBA_OK) rc = launch_dt_columns(ctx, c.dtype, ws + l.dtb, H, 0, T, H, (float *)(ws + l.dt));
    // routed mixture of the experts' B / C projections
    if (rc == SWIMBA_OK) rc = run_route_mix(h, ctx, w, u, T, ws + l.bcp, false, idx, wt, fws + fl.gemm);
    // convolution + SiLU over [x' | B' | C']
    if (rc == SWIMBA_OK)
        rc = launch_conv_silu(ctx, c.dtype, ws + l.zx + (size_t)D * es, 2 * (int64_t)D, ws + l.bcp, bw->conv_w,
                              bw->conv_b, conv_state_in, B, L, D, S, bw->d_conv, ws + l.x, ws + l.bc, conv_state_out);
    // the single recurrence
    if (rc == SWIMBA_OK)
        rc = run_ssd(h, ctx, w, ws + l.x, ws + l.bc, (const float *)(ws + l.dt), h0, B, L, ws + l.y, h_final,
                     fws + fl.ssd);
    // gate, norm, out-projection (the normalised rows reuse the x buffer)
    if (rc == SWIMBA_OK)
        rc = launch_gated_rmsnorm(ctx, c.dtype, ws + l.y, ws + l.zx, 2 * (int64_t)D, bw->norm_w, T, D, c.n_groups,
                                  bw->eps, ws + l.x);
    if (rc == SWIMBA_OK) rc = dense_linear(h, ctx, ws + l.x, bw->W_out, T, D, F, out, ws + l.lin);
    if (rc != SWIMBA_OK && !h->err[0]) fail(h, rc, "a block kernel launch failed");
    h->last_stream = ctx.stream;
    h->last_launches = ctx.launches;
    return rc;
}

int swimba_ssd(swimba_handle *h, const swimba_weights *w, const void *x, const void *BC,
               const float *dt, const float *h0, int32_t B, int32_t L, void *y, float *h_final,
               void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!h) return SWIMBA_ERR_NULL_ARG;
    h->err[0] = 0;
    if (B < 0 || L < 0) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "negative B or L");
    if (B > 65535) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "more than 65535 sequences per call");
    int rc = check_weights(h, w, false);
    if (rc != SWIMBA_OK) return rc;
    if (B == 0 || L == 0) { h->last_launches = 0; return SWIMBA_OK; }
    if (!x || !BC || !y) return fail(h, SWIMBA_ERR_NULL_ARG, "x, BC or y is NULL");
    if (!aligned16(x) || !aligned16(BC) || !aligned16(y) || !aligned16(dt) || !aligned16(h0) ||
        !aligned16(h_final) || !aligned16(workspace))
        return fail(h, SWIMBA_ERR_MISALIGNED, "tensors must be 16-byte aligned");
    const FwdLayout l = fwd_layout(h->cfg, B, L, h->sm_count);
    if (!workspace || workspace_bytes < l.total) return fail(h, SWIMBA_ERR_WORKSPACE_TOO_SMALL, "workspace too small");
    if ((rc = set_device(h)) != SWIMBA_OK) return rc;
    LaunchCtx ctx{(cudaStream_t)cuda_stream, h->d_status, 0, &h->prof, (h->cfg.flags & SWIMBA_FLAG_CHECK_INDICES) != 0, &h->tmaps};
    h->prof.n = 0;
    rc = run_ssd(h, ctx, w, x, BC, dt, h0, B, L, y, h_final, (char *)workspace + l.ssd);
    h->last_stream = ctx.stream;
    h->last_launches = ctx.launches;
    return rc;
}

int swimba_forward(swimba_handle *h, const swimba_weights *w, const void *u, const void *x,
                   const float *dt, const float *h0, int32_t B, int32_t L, void *y,
                   float *h_final, int32_t *topk_idx, float *topk_w, void *workspace,
                   size_t workspace_bytes, void *cuda_stream)
{
    if (!h) return SWIMBA_ERR_NULL_ARG;
    h->err[0] = 0;
    if (B < 0 || L < 0) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "negative B or L");
    if ((int64_t)B * L * h->cfg.top_k >= (int64_t)1 << 31)
        return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "too many tokens (B * L * top_k must stay below 2^31)");
    if (B > 65535) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "more than 65535 sequences per call");
    int rc = check_weights(h, w, true);
    if (rc != SWIMBA_OK) return rc;
    if (B == 0 || L == 0) { h->last_launches = 0; return SWIMBA_OK; }
    if (!u || !x || !y || !workspace) return fail(h, SWIMBA_ERR_NULL_ARG, "u, x, y or workspace is NULL");
    if (!aligned16(u) || !aligned16(x) || !aligned16(y) || !aligned16(dt) || !aligned16(h0) ||
        !aligned16(h_final) || !aligned16(topk_idx) || !aligned16(topk_w) || !aligned16(workspace))
        return fail(h, SWIMBA_ERR_MISALIGNED, "tensors must be 16-byte aligned");
    const int64_t T = (int64_t)B * L;
    const FwdLayout l = fwd_layout(h->cfg, B, L, h->sm_count);
    if (workspace_bytes < l.total) return fail(h, SWIMBA_ERR_WORKSPACE_TOO_SMALL, "workspace too small");
    if ((rc = set_device(h)) != SWIMBA_OK) return rc;
    char *ws = (char *)workspace;
    LaunchCtx ctx{(cudaStream_t)cuda_stream, h->d_status, 0, &h->prof, (h->cfg.flags & SWIMBA_FLAG_CHECK_INDICES) != 0, &h->tmaps};
    h->prof.n = 0;
    int32_t *idx = topk_idx ? topk_idx : (int32_t *)(ws + l.idx);
    float *wt = topk_w ? topk_w : (float *)(ws + l.w);
    void *BC = ws + l.bc;
    // The SSD step sizes depend on dt only: their kernel runs beside the router.
    const bool fuse = ssd_tiles_supported(h->cfg.dtype, h->cfg.head_dim, h->cfg.d_state);
    const ScalarsArgs sa = fuse ? ssd_scalars_args(dt, w->A, w->dt_bias, B, L, h->cfg.n_heads, ws + l.ssd)
                                : ScalarsArgs{};
    rc = run_route_mix(h, ctx, w, u, T, BC, false, idx, wt, ws + l.gemm, fuse ? &sa : nullptr);
    if (rc == SWIMBA_OK) rc = run_ssd(h, ctx, w, x, BC, dt, h0, B, L, y, h_final, ws + l.ssd, fuse);
    h->last_stream = ctx.stream;
    h->last_launches = ctx.launches;
    return rc;
}

namespace {
// Workspace of the packed forward: the forward's regions for T tokens, with the SSD region sized for
// the packed batch.
FwdLayout packed_fwd_layout(const swimba_config &c, const int32_t *cu, int nseq, int sm_count)
{
    const int64_t T = cu[nseq];
    FwdLayout l = fwd_layout(c, 1, (int)(T > 0 ? T : 1), sm_count);
    size_t off = l.ssd;
    if (ssd_tiles_supported(c.dtype, c.head_dim, c.d_state))
        off += align_up(ssd_packed_workspace_bytes(cu, nseq, c.n_heads, c.n_groups, c.chunk, sm_count));
    l.total = off;
    return l;
}
bool packed_offsets_ok(const int32_t *cu, int nseq)
{
    if (!cu || nseq < 0 || cu[0] != 0) return false;
    for (int b = 0; b < nseq; ++b)
        if (cu[b + 1] < cu[b]) return false;
    return true;
}
}  // namespace

size_t swimba_packed_workspace_bytes(const swimba_handle *h, const int32_t *cu_seqlens, int32_t nseq)
{
    if (!h || nseq <= 0 || !packed_offsets_ok(cu_seqlens, nseq) || cu_seqlens[nseq] <= 0) return 0;
    return packed_fwd_layout(h->cfg, cu_seqlens, nseq, h->sm_count).total;
}

int32_t swimba_packed_segments(const swimba_handle *h, const int32_t *cu_seqlens, int32_t nseq)
{
    if (!h || nseq <= 0 || !packed_offsets_ok(cu_seqlens, nseq)) return 0;
    const swimba_config &c = h->cfg;
    if (!ssd_tiles_supported(c.dtype, c.head_dim, c.d_state)) return nseq;
    return ssd_packed_segments(cu_seqlens, nseq, c.n_heads, c.n_groups, c.chunk, h->sm_count);
}

int swimba_forward_packed(swimba_handle *h, const swimba_weights *w, const void *u, const void *x,
                          const float *dt, const float *h0, const int32_t *cu_seqlens, int32_t nseq,
                          void *y, float *h_final, int32_t *topk_idx, float *topk_w, void *workspace,
                          size_t workspace_bytes, void *cuda_stream)
{
    if (!h) return SWIMBA_ERR_NULL_ARG;
    h->err[0] = 0;
    if (nseq < 0) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "negative number of sequences");
    if (nseq > 0 && !cu_seqlens) return fail(h, SWIMBA_ERR_NULL_ARG, "cu_seqlens is NULL");
    if (nseq > 0 && !packed_offsets_ok(cu_seqlens, nseq))
        return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "cu_seqlens must start at 0 and never decrease");
    const int64_t T = nseq > 0 ? cu_seqlens[nseq] : 0;
    if (T * h->cfg.top_k >= (int64_t)1 << 31)
        return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "too many tokens (T * top_k must stay below 2^31)");
    int rc = check_weights(h, w, true);
    if (rc != SWIMBA_OK) return rc;
    if (nseq == 0) { h->last_launches = 0; return SWIMBA_OK; }
    if (T > 0 && (!u || !x || !y || !workspace)) return fail(h, SWIMBA_ERR_NULL_ARG, "u, x, y or workspace is NULL");
    if (!aligned16(u) || !aligned16(x) || !aligned16(y) || !aligned16(dt) || !aligned16(h0) ||
        !aligned16(h_final) || !aligned16(topk_idx) || !aligned16(topk_w) || !aligned16(workspace))
        return fail(h, SWIMBA_ERR_MISALIGNED, "tensors must be 16-byte aligned");
    const swimba_config &c = h->cfg;
    const FwdLayout l = packed_fwd_layout(c, cu_seqlens, nseq, h->sm_count);
    if (T > 0 && workspace_bytes < l.total) return fail(h, SWIMBA_ERR_WORKSPACE_TOO_SMALL, "workspace too small");
    if ((rc = set_device(h)) != SWIMBA_OK) return rc;
    char *ws = (char *)workspace;
    LaunchCtx ctx{(cudaStream_t)cuda_stream, h->d_status, 0, &h->prof, (c.flags & SWIMBA_FLAG_CHECK_INDICES) != 0, &h->tmaps};
    h->prof.n = 0;
    const size_t PN = (size_t)c.n_heads * c.head_dim * c.d_state;
    if (T == 0) {
        // nothing but empty sequences: every state passes through
        if (h_final) {
            const cudaError_t e = h0 ? cudaMemcpyAsync(h_final, h0, (size_t)nseq * PN * sizeof(float), cudaMemcpyDeviceToDevice, ctx.stream)
                                     : cudaMemsetAsync(h_final, 0, (size_t)nseq * PN * sizeof(float), ctx.stream);
            if (e != cudaSuccess) return fail(h, SWIMBA_ERR_CUDA, "copying the states failed");
        }
        h->last_stream = ctx.stream;
        h->last_launches = 0;
        return SWIMBA_OK;
    }
    int32_t *idx = topk_idx ? topk_idx : (int32_t *)(ws + l.idx);
    float *wt = topk_w ? topk_w : (float *)(ws + l.w);
    void *BC = ws + l.bc;
    // routing, projection and mix are per token: the packed batch is one run of T tokens
    rc = run_route_mix(h, ctx, w, u, T, BC, false, idx, wt, ws + l.gemm);
    if (rc == SWIMBA_OK) {
        if (ssd_tiles_supported(c.dtype, c.head_dim, c.d_state)) {
            rc = launch_ssd_tiles_packed(ctx, x, BC, dt, w->A, w->dt_bias, w->D, h0, cu_seqlens, nseq, c.n_heads,
                                         c.n_groups, c.chunk, h->sm_count, y, h_final, ws + l.ssd);
            if (rc != SWIMBA_OK) rc = fail(h, rc, "SSD tile kernel launch failed");
        } else {
            // per-timestep evaluation, sequence by sequence
            const size_t es = elt_size(c.dtype);
            const size_t HP = (size_t)c.n_heads * c.head_dim, S = 2u * c.n_groups * c.d_state;
            for (int b = 0; b < nseq && rc == SWIMBA_OK; ++b) {
                const size_t t0 = (size_t)cu_seqlens[b];
                const int len = cu_seqlens[b + 1] - cu_seqlens[b];
                float *hf = h_final ? h_final + (size_t)b * PN : nullptr;
                const float *hin = h0 ? h0 + (size_t)b * PN : nullptr;
                if (len == 0) {
                    if (hf) {
                        const cudaError_t e = hin ? cudaMemcpyAsync(hf, hin, PN * sizeof(float), cudaMemcpyDeviceToDevice, ctx.stream)
                                                  : cudaMemsetAsync(hf, 0, PN * sizeof(float), ctx.stream);
                        if (e != cudaSuccess) rc = fail(h, SWIMBA_ERR_CUDA, "copying a state failed");
                    }
                    continue;
                }
                rc = launch_ssd_sequential(ctx, c.dtype, (const char *)x + t0 * HP * es, (const char *)BC + t0 * S * es,
                                           false, dt ? dt + t0 * c.n_heads : nullptr, w->A, w->dt_bias, w->D, hin, 1,
                                           len, c.n_heads, c.head_dim, c.d_state, c.n_groups,
                                           (char *)y + t0 * HP * es, hf);
                if (rc != SWIMBA_OK) rc = fail(h, rc, "SSD launch failed");
            }
        }
    }
    h->last_stream = ctx.stream;
    h->last_launches = ctx.launches;
    return rc;
}

namespace {
// Workspace of the sequence-sharded forward: the forward's token regions, then the shard's SSD region.
FwdLayout shard_fwd_layout(const swimba_config &c, int B, int L, int sm_count)
{
    FwdLayout l = fwd_layout(c, B, L, sm_count);
    l.total = l.ssd + align_up(ssd_shard_workspace_bytes(B, L, c.n_heads, c.n_groups, c.chunk, sm_count));
    return l;
}
}  // namespace

size_t swimba_shard_workspace_bytes(const swimba_handle *h, int32_t B, int32_t L)
{
    if (!h || B <= 0 || L <= 0) return 0;
    if (!ssd_tiles_supported(h->cfg.dtype, h->cfg.head_dim, h->cfg.d_state)) return 0;
    return shard_fwd_layout(h->cfg, B, L, h->sm_count).total;
}

int swimba_shard_summary(swimba_handle *h, const swimba_weights *w, const void *u, const void *x,
                         const float *dt, int32_t B, int32_t L, float *summary_state, float *summary_decay,
                         int32_t *topk_idx, float *topk_w, void *workspace, size_t workspace_bytes,
                         void *cuda_stream)
{
    if (!h) return SWIMBA_ERR_NULL_ARG;
    h->err[0] = 0;
    const swimba_config &c = h->cfg;
    if (B <= 0 || L <= 0) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "a shard needs B > 0 and L > 0");
    if ((int64_t)B * L * c.top_k >= (int64_t)1 << 31)
        return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "too many tokens (B * L * top_k must stay below 2^31)");
    if (B > 65535) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "more than 65535 sequences per call");
    if (!ssd_tiles_supported(c.dtype, c.head_dim, c.d_state))
        return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "the sequence-sharded forward needs bf16, head_dim 64, d_state 128");
    int rc = check_weights(h, w, true);
    if (rc != SWIMBA_OK) return rc;
    if (!u || !x || !summary_state || !summary_decay || !workspace)
        return fail(h, SWIMBA_ERR_NULL_ARG, "u, x, a summary output or the workspace is NULL");
    if (!aligned16(u) || !aligned16(x) || !aligned16(dt) || !aligned16(summary_state) || !aligned16(summary_decay) ||
        !aligned16(topk_idx) || !aligned16(topk_w) || !aligned16(workspace))
        return fail(h, SWIMBA_ERR_MISALIGNED, "tensors must be 16-byte aligned");
    const FwdLayout l = shard_fwd_layout(c, B, L, h->sm_count);
    if (workspace_bytes < l.total) return fail(h, SWIMBA_ERR_WORKSPACE_TOO_SMALL, "workspace too small");
    if ((rc = set_device(h)) != SWIMBA_OK) return rc;
    char *ws = (char *)workspace;
    LaunchCtx ctx{(cudaStream_t)cuda_stream, h->d_status, 0, &h->prof, (c.flags & SWIMBA_FLAG_CHECK_INDICES) != 0, &h->tmaps};
    h->prof.n = 0;
    int32_t *idx = topk_idx ? topk_idx : (int32_t *)(ws + l.idx);
    float *wt = topk_w ? topk_w : (float *)(ws + l.w);
    void *BC = ws + l.bc;
    const ScalarsArgs sa = ssd_shard_scalars_args(dt, w->A, w->dt_bias, B, L, c.n_heads, c.n_groups, c.chunk,
                                                  h->sm_count, ws + l.ssd);
    rc = run_route_mix(h, ctx, w, u, (int64_t)B * L, BC, false, idx, wt, ws + l.gemm, &sa);
    if (rc == SWIMBA_OK) {
        rc = launch_ssd_shard_summary(ctx, x, BC, dt, w->A, w->dt_bias, B, L, c.n_heads, c.n_groups, c.chunk,
                                      h->sm_count, summary_state, summary_decay, ws + l.ssd, true);
        if (rc != SWIMBA_OK) rc = fail(h, rc, "SSD state-only pass launch failed");
    }
    h->last_stream = ctx.stream;
    h->last_launches = ctx.launches;
    return rc;
}

int swimba_shard_finish(swimba_handle *h, const swimba_weights *w, const void *x, const float *h0,
                        const float *all_state, const float *all_decay, int32_t rank, int32_t n_ranks,
                        int32_t B, int32_t L, void *y, float *h_end, void *workspace, size_t workspace_bytes,
                        void *cuda_stream)
{
    if (!h) return SWIMBA_ERR_NULL_ARG;
    h->err[0] = 0;
    const swimba_config &c = h->cfg;
    if (B <= 0 || L <= 0) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "a shard needs B > 0 and L > 0");
    if (B > 65535) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "more than 65535 sequences per call");
    if (n_ranks <= 0 || rank < 0 || rank >= n_ranks) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "rank outside [0, n_ranks)");
    if (!ssd_tiles_supported(c.dtype, c.head_dim, c.d_state))
        return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "the sequence-sharded forward needs bf16, head_dim 64, d_state 128");
    int rc = check_weights(h, w, false);
    if (rc != SWIMBA_OK) return rc;
    if (!x || !y || !workspace || (rank > 0 && (!all_state || !all_decay)))
        return fail(h, SWIMBA_ERR_NULL_ARG, "x, y, the workspace or the gathered summaries are NULL");
    if (!aligned16(x) || !aligned16(y) || !aligned16(h0) || !aligned16(all_state) || !aligned16(all_decay) ||
        !aligned16(h_end) || !aligned16(workspace))
        return fail(h, SWIMBA_ERR_MISALIGNED, "tensors must be 16-byte aligned");
    const FwdLayout l = shard_fwd_layout(c, B, L, h->sm_count);
    if (workspace_bytes < l.total) return fail(h, SWIMBA_ERR_WORKSPACE_TOO_SMALL, "workspace too small");
    if ((rc = set_device(h)) != SWIMBA_OK) return rc;
    char *ws = (char *)workspace;
    LaunchCtx ctx{(cudaStream_t)cuda_stream, h->d_status, 0, &h->prof, (c.flags & SWIMBA_FLAG_CHECK_INDICES) != 0, &h->tmaps};
    h->prof.n = 0;
    rc = launch_ssd_shard_finish(ctx, x, ws + l.bc, w->D, h0, all_state, all_decay, rank, B, L, c.n_heads, c.n_groups,
                                 c.chunk, h->sm_count, y, h_end, ws + l.ssd);
    if (rc != SWIMBA_OK) rc = fail(h, rc, "SSD full pass launch failed");
    h->last_stream = ctx.stream;
    h->last_launches = ctx.launches;
    return rc;
}

namespace {
// Workspace of the backward: the forward's token regions, then [ones | slot projections | dBC | pi | dg].
struct BwdLayout {
    FwdLayout f;
    size_t ones, slots, dbc, pi, dg, adj, total;
};
BwdLayout bwd_layout(const swimba_config &c, int B, int L, int sm_count)
{
    BwdLayout l;
    l.f = fwd_layout(c, B, L, sm_count);
    const size_t T = (size_t)B * L, S = 2u * c.n_groups * c.d_state;
    size_t off = l.f.ssd;
    l.ones = off;  off += align_up(T * c.top_k * sizeof(float));
    l.slots = off; off += align_up(T * c.top_k * S * elt_size(c.dtype));
    l.dbc = off;   off += align_up(T * S * sizeof(float));
    l.pi = off;    off += align_up(T * c.n_experts * sizeof(float));
    l.dg = off;    off += align_up(T * c.n_experts * sizeof(float));
    l.adj = off;
    if (ssd_tiles_supported(c.dtype, c.head_dim, c.d_state))
        off += align_up(ssd_adjoint_tiles_workspace_bytes(B, L, c.n_heads, c.chunk, sm_count));
    l.total = off;
    return l;
}
}  // namespace

size_t swimba_backward_workspace_bytes(const swimba_handle *h, int32_t B, int32_t L)
{
    if (!h || B <= 0 || L <= 0) return 0;
    return bwd_layout(h->cfg, B, L, h->sm_count).total;
}

int swimba_backward_weights(swimba_handle *h, const swimba_weights *w, const void *u, const void *x,
                            const float *dt, const float *h0, const void *dy, int32_t B, int32_t L,
                            float *dW_router, float *dW_expert, int32_t *topk_idx, void *workspace,
                            size_t workspace_bytes, void *cuda_stream)
{
    if (!h) return SWIMBA_ERR_NULL_ARG;
    h->err[0] = 0;
    const swimba_config &c = h->cfg;
    if (B < 0 || L < 0) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "negative B or L");
    const int64_t T = (int64_t)B * L;
    if (T * c.top_k >= (int64_t)1 << 31)
        return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "too many tokens (B * L * top_k must stay below 2^31)");
    if (B > 65535) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "more than 65535 sequences per call");
    if (!ssd_adjoint_supported(c.head_dim, c.d_state) || (int64_t)c.n_experts * ((T + 2047) / 2048) > 65535 ||
        c.n_heads > 1024 ||
        (int64_t)B * c.n_heads >= (int64_t)1 << 31)
        return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "shape outside what the backward kernels take");
    int rc = check_weights(h, w, true);
    if (rc != SWIMBA_OK) return rc;
    if (!dW_expert || (!dW_router && c.n_experts > 1))
        return fail(h, SWIMBA_ERR_NULL_ARG, "a gradient output is NULL");
    if (!aligned16(u) || !aligned16(x) || !aligned16(dy) || !aligned16(dt) || !aligned16(h0) || !aligned16(dW_router) ||
        !aligned16(dW_expert) || !aligned16(topk_idx) || !aligned16(workspace))
        return fail(h, SWIMBA_ERR_MISALIGNED, "tensors must be 16-byte aligned");
    if ((rc = set_device(h)) != SWIMBA_OK) return rc;
    LaunchCtx ctx{(cudaStream_t)cuda_stream, h->d_status, 0, &h->prof, (c.flags & SWIMBA_FLAG_CHECK_INDICES) != 0, &h->tmaps};
    h->prof.n = 0;
    const size_t S = 2u * c.n_groups * c.d_state;
    // the gradients of an empty batch are zero
    if (cudaMemsetAsync(dW_expert, 0, (size_t)c.n_experts * S * c.d_model * sizeof(float), ctx.stream) != cudaSuccess ||
        (dW_router &&
         cudaMemsetAsync(dW_router, 0, (size_t)c.n_experts * c.d_model * sizeof(float), ctx.stream) != cudaSuccess))
        return fail(h, SWIMBA_ERR_CUDA, "clearing the gradients failed");
    h->last_stream = ctx.stream;
    if (T == 0) { h->last_launches = 0; return SWIMBA_OK; }
    if (!u || !x || !dy || !workspace) return fail(h, SWIMBA_ERR_NULL_ARG, "u, x, dy or workspace is NULL");
    const BwdLayout l = bwd_layout(c, B, L, h->sm_count);
    if (workspace_bytes < l.total) return fail(h, SWIMBA_ERR_WORKSPACE_TOO_SMALL, "workspace too small");
    char *ws = (char *)workspace;
    int32_t *idx = topk_idx ? topk_idx : (int32_t *)(ws + l.f.idx);
    float *wt = (float *)(ws + l.f.w);
    void *BC = ws + l.f.bc;
    float *ones = (float *)(ws + l.ones);
    void *slots = ws + l.slots;
    float *dBC = (float *)(ws + l.dbc);
    // forward quantities again: routing, mixed streams, and the unscaled projection of every kept slot
    rc = run_route_mix(h, ctx, w, u, T, BC, false, idx, wt, ws + l.f.gemm);
    if (rc == SWIMBA_OK) rc = launch_fill(ctx, ones, T * c.top_k, 1.f);
    if (rc == SWIMBA_OK) {
        if (use_tensor_k1(c))
            rc = launch_expert_gemm(ctx, u, w->W_expert, ones, T, c.d_model, (int)S, c.n_experts, c.top_k, h->sm_count,
                                    BC, ws + l.f.gemm, slots);
        else
            rc = launch_project_slots_simt(ctx, c.dtype, u, w->W_expert, idx, ones, T, c.d_model, (int)S, c.n_experts,
                                           c.top_k, slots);
        if (rc != SWIMBA_OK) rc = fail(h, rc, "slot projection launch failed");
    }
    if (rc == SWIMBA_OK && cudaMemsetAsync(dBC, 0, (size_t)T * S * sizeof(float), ctx.stream) != cudaSuccess)
        rc = fail(h, SWIMBA_ERR_CUDA, "clearing dBC failed");
    if (rc == SWIMBA_OK) {
        // shapes of the forward's tile kernel: the adjoint is two more evaluations of that kernel on
        // re-arranged operands; everything else: per-timestep passes
        if (ssd_tiles_supported(c.dtype, c.head_dim, c.d_state))
            rc = launch_ssd_adjoint_tiles(ctx, x, dy, BC, dt, w->A, w->dt_bias, h0, B, L, c.n_heads, c.n_groups,
                                          c.chunk, h->sm_count, dBC, ws + l.adj);
        else
            rc = launch_ssd_adjoint(ctx, c.dtype, x, dy, BC, dt, w->A, w->dt_bias, h0, B, L, c.n_heads, c.head_dim,
                                    c.d_state, c.n_groups, dBC);
        if (rc != SWIMBA_OK) rc = fail(h, rc, "adjoint recurrence launch failed");
    }
    if (rc == SWIMBA_OK) {
        const void *Wr = w->W_router ? w->W_router : w->W_expert;
        rc = launch_weight_grads(ctx, c.dtype, u, Wr, slots, idx, wt, dBC, T, c.d_model, (int)S, c.n_experts, c.top_k,
                                 (float *)(ws + l.pi), (float *)(ws + l.dg),
                                 dW_router, dW_expert);
        if (rc != SWIMBA_OK) rc = fail(h, rc, "weight gradient launch failed");
    }
    h->last_launches = ctx.launches;
    return rc;
}

int swimba_decode_step(swimba_handle *h, const swimba_weights *w, const void *u, const void *x,
                       const float *dt, float *state, int32_t B, void *y, int32_t *topk_idx,
                       float *topk_w, void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!h) return SWIMBA_ERR_NULL_ARG;
    h->err[0] = 0;
    if (B < 0) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "negative B");
    int rc = check_weights(h, w, true);
    if (rc != SWIMBA_OK) return rc;
    if (B == 0) { h->last_launches = 0; return SWIMBA_OK; }
    if (!u || !x || !y || !state || !workspace)
        return fail(h, SWIMBA_ERR_NULL_ARG, "u, x, y, state or workspace is NULL");
    if (!aligned16(u) || !aligned16(x) || !aligned16(y) || !aligned16(dt) || !aligned16(state) ||
        !aligned16(topk_idx) || !aligned16(topk_w) || !aligned16(workspace))
        return fail(h, SWIMBA_ERR_MISALIGNED, "tensors must be 16-byte aligned");
    const DecLayout l = dec_layout(h->cfg, B);
    if (workspace_bytes < l.total) return fail(h, SWIMBA_ERR_WORKSPACE_TOO_SMALL, "workspace too small");
    if ((rc = set_device(h)) != SWIMBA_OK) return rc;
    const swimba_config &c = h->cfg;
    char *ws = (char *)workspace;
    LaunchCtx ctx{(cudaStream_t)cuda_stream, h->d_status, 0, &h->prof, (h->cfg.flags & SWIMBA_FLAG_CHECK_INDICES) != 0, &h->tmaps};
    h->prof.n = 0;
    int32_t *idx = topk_idx ? topk_idx : (int32_t *)(ws + l.idx);
    float *wt = topk_w ? topk_w : (float *)(ws + l.w);
    void *BC = ws + l.bc;
    const int S = 2 * c.n_groups * c.d_state;
    // a handful of tokens: the two-kernel front end (fp32 streams); else bf16 streams from the
    // grouped GEMM, or fp32 from the SIMT projection
    const bool small = front_small_supported(c.dtype, B, c.d_model, S, c.n_experts, c.top_k);
    const bool tensor = !small && use_tensor_k1(c);
    if (small) {
        rc = launch_front_small(ctx, u, w->W_router ? w->W_router : w->W_expert, w->W_expert, B, c.d_model, S,
                                c.n_experts, c.top_k, idx, wt, (float *)BC);
        if (rc != SWIMBA_OK) fail(h, rc, "routing / projection launch failed");
    } else {
        rc = run_route_mix(h, ctx, w, u, B, BC, !tensor, idx, wt, tensor ? ws + l.gemm : nullptr);
    }
    if (rc == SWIMBA_OK) {
        rc = launch_decode_update(ctx, c.dtype, x, BC, !tensor, dt, w->A, w->dt_bias, w->D, state, B,
                                  c.n_heads, c.head_dim, c.d_state, c.n_groups, h->sm_count, y);
        if (rc != SWIMBA_OK) fail(h, rc, "decode launch failed");
    }
    h->last_stream = ctx.stream;
    h->last_launches = ctx.launches;
    return rc;
}

int swimba_forward_host(swimba_handle *h, const swimba_weights *w, const void *u_host,
                        const void *x_host, const float *dt_host, int32_t B, int32_t L,
                        void *y_host, float *h_final_host, int32_t *topk_idx_host,
                        float *topk_w_host, void *workspace, size_t workspace_bytes,
                        void *cuda_stream)
{
    if (!h) return SWIMBA_ERR_NULL_ARG;
    h->err[0] = 0;
    if (B < 0 || L < 0) return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "negative B or L");
    if (B == 0 || L == 0) { h->last_launches = 0; return SWIMBA_OK; }
    if (!u_host || !x_host || !y_host || !workspace)
        return fail(h, SWIMBA_ERR_NULL_ARG, "u_host, x_host, y_host or workspace is NULL");
    if (!aligned16(workspace)) return fail(h, SWIMBA_ERR_MISALIGNED, "workspace must be 16-byte aligned");
    const swimba_config &c = h->cfg;
    const HostLayout l = host_layout(c, B, L, h->sm_count);
    if (workspace_bytes < l.total) return fail(h, SWIMBA_ERR_WORKSPACE_TOO_SMALL, "workspace too small");
    int rc = check_weights(h, w, true);
    if (rc != SWIMBA_OK) return rc;
    if ((rc = set_device(h)) != SWIMBA_OK) return rc;
    // Batch slices flow through three streams: copies in (s_in), kernels (the caller's stream),
    // copies out (s_out), so that the host-to-device copy of slice i+1 and the device-to-host
    // copy of slice i-1 overlap the kernels of slice i.  Sequences are independent, so a slice is
    // a forward call of its own on the staged tensors.
    cudaStream_t st = (cudaStream_t)cuda_stream;
    char *ws = (char *)workspace;
    const size_t es = elt_size(c.dtype);
    const size_t HP = (size_t)c.n_heads * c.head_dim;
    const size_t tok_u = (size_t)c.d_model * es, tok_x = HP * es, tok_dt = c.n_heads * sizeof(float);
    const size_t seq_hf = HP * c.d_state * sizeof(float);
    const size_t tok_k = (size_t)c.top_k * sizeof(int32_t);
    const HostPlan plan = host_plan(c, B, L);
    bool ok = cudaEventRecord(h->ev_start, st) == cudaSuccess &&
              cudaStreamWaitEvent(h->s_in, h->ev_start, 0) == cudaSuccess &&
              cudaStreamWaitEvent(h->s_out, h->ev_start, 0) == cudaSuccess;
    int launches = 0, slice = 0;
    for (int b0 = 0; ok && rc == SWIMBA_OK && b0 < B; b0 += plan.seqs) {
        const int nb = (B - b0 < plan.seqs) ? B - b0 : plan.seqs;
        for (int pc = 0; ok && pc < plan.pieces; ++pc, ++slice) {
            const int l0 = pc * plan.piece;
            const int len = plan.pieces == 1 ? L : (L - l0 < plan.piece ? L - l0 : plan.piece);
            const size_t t0 = (size_t)b0 * L + l0, nt = (size_t)nb * len;
            ok = cudaMemcpyAsync(ws + l.u + t0 * tok_u, (const char *)u_host + t0 * tok_u, nt * tok_u,
                                 cudaMemcpyHostToDevice, h->s_in) == cudaSuccess &&
                 cudaMemcpyAsync(ws + l.x + t0 * tok_x, (const char *)x_host + t0 * tok_x, nt * tok_x,
                                 cudaMemcpyHostToDevice, h->s_in) == cudaSuccess;
            if (ok && dt_host)
                ok = cudaMemcpyAsync(ws + l.dt + t0 * tok_dt, (const char *)dt_host + t0 * tok_dt, nt * tok_dt,
                                     cudaMemcpyHostToDevice, h->s_in) == cudaSuccess;
            ok = ok && cudaEventRecord(h->ev_in[slice], h->s_in) == cudaSuccess &&
                 cudaStreamWaitEvent(st, h->ev_in[slice], 0) == cudaSuccess;
            if (!ok) break;
            // the state after a piece enters the next piece of the same sequence; the two buffers
            // alternate, since a call may still read its initial state while it writes its final one
            const size_t hf_cur = (pc & 1) ? l.hf2 : l.hf, hf_prev = (pc & 1) ? l.hf : l.hf2;
            const bool last_piece = pc == plan.pieces - 1;
            const bool want_state = !last_piece || h_final_host != nullptr;
            rc = swimba_forward(h, w, ws + l.u + t0 * tok_u, ws + l.x + t0 * tok_x,
                                dt_host ? (const float *)(ws + l.dt + t0 * tok_dt) : nullptr,
                                pc > 0 ? (const float *)(ws + hf_prev + (size_t)b0 * seq_hf) : nullptr, nb, len,
                                ws + l.y + t0 * tok_x,
                                want_state ? (float *)(ws + hf_cur + (size_t)b0 * seq_hf) : nullptr,
                                (int32_t *)(ws + l.idx + t0 * tok_k), (float *)(ws + l.w + t0 * tok_k),
                                ws + l.fwd, workspace_bytes - l.fwd, cuda_stream);
            if (rc != SWIMBA_OK) break;
            launches += h->last_launches;
            ok = cudaEventRecord(h->ev_done[slice], st) == cudaSuccess &&
                 cudaStreamWaitEvent(h->s_out, h->ev_done[slice], 0) == cudaSuccess &&
                 cudaMemcpyAsync((char *)y_host + t0 * tok_x, ws + l.y + t0 * tok_x, nt * tok_x,
                                 cudaMemcpyDeviceToHost, h->s_out) == cudaSuccess;
            if (ok && h_final_host && last_piece)
                ok = cudaMemcpyAsync((char *)h_final_host + (size_t)b0 * seq_hf, ws + hf_cur + (size_t)b0 * seq_hf,
                                     (size_t)nb * seq_hf, cudaMemcpyDeviceToHost, h->s_out) == cudaSuccess;
            if (ok && topk_idx_host)
                ok = cudaMemcpyAsync((char *)topk_idx_host + t0 * tok_k, ws + l.idx + t0 * tok_k, nt * tok_k,
                                     cudaMemcpyDeviceToHost, h->s_out) == cudaSuccess;
            if (ok && topk_w_host)
                ok = cudaMemcpyAsync((char *)topk_w_host + t0 * tok_k, ws + l.w + t0 * tok_k, nt * tok_k,
                                     cudaMemcpyDeviceToHost, h->s_out) == cudaSuccess;
        }
    }
    // The caller's stream ends after the last copy in and the last copy out, on the error paths
    // too (copies of earlier slices may still be in flight): synchronising it is enough before the
    // host buffers are read, reused or freed.
    const bool joined = cudaEventRecord(h->ev_out, h->s_out) == cudaSuccess &&
                        cudaStreamWaitEvent(st, h->ev_out, 0) == cudaSuccess &&
                        cudaEventRecord(h->ev_start, h->s_in) == cudaSuccess &&
                        cudaStreamWaitEvent(st, h->ev_start, 0) == cudaSuccess;
    h->last_launches = launches;
    if (rc != SWIMBA_OK) return rc;             // (message set by the failing forward)
    if (!ok || !joined) { cudaGetLastError(); return fail(h, SWIMBA_ERR_CUDA, "a copy or an event of the host pipeline failed"); }
    return SWIMBA_OK;
}

int swimba_profile(swimba_handle *h, int enable)
{
    if (!h) return SWIMBA_ERR_NULL_ARG;
    if (enable && !h->prof.ev[0]) {
        for (int i = 0; i < 2 * PROF_MAX; ++i)
            if (cudaEventCreate(&h->prof.ev[i]) != cudaSuccess) return fail(h, SWIMBA_ERR_CUDA, "event creation failed");
    }
    h->prof.on = enable != 0;
    h->prof.n = 0;
    return SWIMBA_OK;
}

int swimba_profile_read(swimba_handle *h, int32_t *kernel_ids, float *ms, int32_t max_entries)
{
    if (!h || !kernel_ids || !ms) return SWIMBA_ERR_NULL_ARG;
    if (!h->prof.on) return 0;
    if (cudaStreamSynchronize(h->last_stream) != cudaSuccess) return fail(h, SWIMBA_ERR_CUDA, "stream synchronisation failed");
    int n = h->prof.n < max_entries ? h->prof.n : max_entries;
    for (int i = 0; i < n; ++i) {
        kernel_ids[i] = h->prof.stage[i];
        if (cudaEventElapsedTime(&ms[i], h->prof.ev[2 * i], h->prof.ev[2 * i + 1]) != cudaSuccess)
            return fail(h, SWIMBA_ERR_CUDA, "cudaEventElapsedTime failed");
    }
    return n;
}

int swimba_selftest_wait(swimba_handle *h, int64_t limit_cycles, int64_t *result_host, void *cuda_stream)
{
    if (!h) return SWIMBA_ERR_NULL_ARG;
    h->err[0] = 0;
    if (limit_cycles < 1000 || limit_cycles > 100000000)
        return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "limit_cycles must lie in [1e3, 1e8]");
    int rc = set_device(h);
    if (rc != SWIMBA_OK) return rc;
    // the three result words live behind the status word in the handle's 64-byte device block
    long long *out_dev = (long long *)(h->d_status + 4);
    LaunchCtx ctx{(cudaStream_t)cuda_stream, h->d_status, 0, nullptr};
    rc = launch_wait_selftest(ctx, (long long)limit_cycles, out_dev);
    h->last_stream = ctx.stream;
    h->last_launches = ctx.launches;
    if (rc != SWIMBA_OK) return fail(h, rc, "self-test launch failed");
    if (result_host) {
        long long tmp[3];
        if (cudaStreamSynchronize(ctx.stream) != cudaSuccess ||
            cudaMemcpy(tmp, out_dev, sizeof(tmp), cudaMemcpyDeviceToHost) != cudaSuccess)
            return fail(h, SWIMBA_ERR_CUDA, "reading the self-test result failed");
        for (int i = 0; i < 3; ++i) result_host[i] = (int64_t)tmp[i];
    }
    return SWIMBA_OK;
}

int swimba_last_launch_count(const swimba_handle *h) { return h ? h->last_launches : 0; }

int swimba_status(swimba_handle *h)
{
    if (!h) return SWIMBA_ERR_NULL_ARG;
    if (cudaStreamSynchronize(h->last_stream) != cudaSuccess) {
        snprintf(h->err, sizeof(h->err), "stream synchronisation failed: %s",
                 cudaGetErrorString(cudaGetLastError()));
        return SWIMBA_ERR_CUDA;
    }
    int word[4] = {0, 0, 0, 0};
    if (cudaMemcpy(word, h->d_status, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess)
        return fail(h, SWIMBA_ERR_CUDA, "reading the device status word failed");
    const int code = word[0];
    if (code != 0) {
        cudaMemset(h->d_status, 0, 64);
        if (code == SWIMBA_ERR_DEVICE_TIMEOUT)
            snprintf(h->err, sizeof(h->err),
                     "device reported error %d (a wait ran out: barrier at shared address 0x%x, parity %d, block %d, thread %d)",
                     code, (unsigned)word[1], word[2], word[3] >> 12, word[3] & 0xfff);
        else
            snprintf(h->err, sizeof(h->err), "device reported error %d", code);
    }
    return code;
}

const char *swimba_last_error(const swimba_handle *h) { return h ? h->err : ""; }

void swimba_destroy(swimba_handle *h)
{
    if (!h) return;
    if (h->d_status) cudaFree(h->d_status);
    destroy_host_pipeline(h);
    if (h->prof.ev[0])
        for (int i = 0; i < 2 * PROF_MAX; ++i) if (h->prof.ev[i]) cudaEventDestroy(h->prof.ev[i]);
    delete h;
}

}  // extern "C"

// ------------------------------------------------------------------------------------------
// Allocation-free variant of swimba_route_mix.
//
// Some callers cannot obtain device memory at the point where they call the library: code that
// runs inside a memory-budgeted serving process whose pool is already handed out, plug-ins that
// receive only their input and output buffers from a host framework, or set-up paths that run
// before an allocator exists.  For them the scratch that the routing/projection stage needs (the
// expert histogram, the tile table, the row permutation and the per-slot projections) lives in a
// fixed array that is part of the library image.  Every GPU that loads the library holds these
// SWIMBA_STATIC_SCRATCH_BYTES until the process exits.
// ------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_scratch[SWIMBA_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void *g_static_scratch_ptr[kMaxDevices];   // device address of g_static_scratch, per device
}  // namespace

extern "C" int swimba_route_mix_static(swimba_handle *h, const swimba_weights *w, const void *u,
                                       int64_t T, void *BC, int32_t *topk_idx, float *topk_w,
                                       void *cuda_stream)
{
    if (!h) return SWIMBA_ERR_NULL_ARG;
    h->err[0] = 0;
    // (token, slot) entries are indexed with 32-bit integers
    if (T < 0 || T * h->cfg.top_k >= (int64_t)1 << 31)
        return fail(h, SWIMBA_ERR_UNSUPPORTED_SHAPE, "T out of range (T * top_k must stay below 2^31)");
    if (T == 0) { h->last_launches = 0; return SWIMBA_OK; }
    int rc = set_device(h);
    if (rc != SWIMBA_OK) return rc;
    if (h->device < 0 || h->device >= kMaxDevices)
        return fail(h, SWIMBA_ERR_CUDA, "device ordinal beyond the static-scratch table");
    // In host code the array's name is only a stand-in; the kernels need its device address.
    // Looked up once per device, with that device current (set_device checked it above).
    if (!g_static_scratch_ptr[h->device]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return fail(h, SWIMBA_ERR_CUDA, "cudaGetSymbolAddress on the static scratch failed");
        }
        g_static_scratch_ptr[h->device] = p;
    }
    // Regions the stage really uses: routing outputs the caller did not ask for, then the grouped
    // GEMM's scratch (histogram, per-expert lists, slot buffer when k > 2).  BC is the caller's.
    const swimba_config &c = h->cfg;
    const size_t off_idx = 0;
    const size_t off_w = off_idx + align_up((size_t)T * c.top_k * sizeof(int32_t));
    const size_t off_gemm = off_w + align_up((size_t)T * c.top_k * sizeof(float));
    const size_t need = off_gemm +
        (use_tensor_k1(c) ? align_up(expert_gemm_workspace_bytes(T, 2 * c.n_groups * c.d_state, c.n_experts, c.top_k)) : 0);
    if (need > (size_t)SWIMBA_STATIC_SCRATCH_BYTES) {
        snprintf(h->err, sizeof(h->err),
                 "T = %lld tokens needs %zu bytes of scratch, the static scratch holds %d",
                 (long long)T, need, (int)SWIMBA_STATIC_SCRATCH_BYTES);
        return SWIMBA_ERR_WORKSPACE_TOO_SMALL;
    }
    char *ws = (char *)g_static_scratch_ptr[h->device];
    return route_mix_call(h, w, u, T, BC, topk_idx, topk_w, ws + off_idx, ws + off_w, ws + off_gemm,
                          cuda_stream);
}
