/*
 * swimba.h -- C ABI of the Swimba (Switch Mamba) token-mixer forward for NVIDIA B200.
 *
 * The layer (paper, Section "MoE-parameterized SSM" and Theorem 1):
 *   router    g_t = W_r u_t, pi_t = softmax(g_t) over all E experts; the k largest entries
 *             are kept with their softmax values, NOT renormalised (Background, "Mixture of
 *             Experts and Switching Dynamics", router softmax equation and the text after it);
 *   streams   every active expert maps the same token features to candidate streams
 *             [B_t^(e) ; C_t^(e)] = W_e[e] u_t (Section "MoE-parameterized SSM");
 *   mix       Btilde_t = sum_{e in K_t} pi_{t,e} B_t^(e), Ctilde_t likewise (Theorem 1);
 *   SSM       ONE recurrence with the transition shared by all experts (shared-A equation):
 *             Delta = softplus(dt + dt_bias), a = exp(Delta * A_h),
 *             h_t = a h_{t-1} + Delta Btilde_t x_t^T,   y_t = Ctilde_t^T h_t + D_h x_t
 *             (selective-SSM equation, channelwise convention), evaluated chunk-wise in the
 *             SSD form (Background, "Mamba-2 and SSD").
 *
 * Conventions
 *   - Every tensor pointer is a DEVICE pointer unless its name ends in _host.  All tensors are
 *     row-major with the last index contiguous and must be 16-byte aligned.
 *   - The caller owns every tensor and the workspace; the library owns only the handle (a few
 *     bytes of device memory for a status word).  Nothing is allocated or freed after create.
 *   - Calls enqueue work on the given CUDA stream and return without synchronising.
 *   - Return value: SWIMBA_OK or a negative SWIMBA_ERR_* code.  When an error is detected on
 *     the host nothing is enqueued and no output is touched.  Nothing throws or aborts.
 *   - "dtype" below means: float for SWIMBA_DTYPE_FP32, bfloat16 for SWIMBA_DTYPE_BF16.
 *     A, dt, dt_bias, D, the SSM state and the router weights returned are always float.
 *   - Notation: T = B*L tokens, F = d_model, H heads, P head_dim, N d_state, G groups,
 *     S = 2*G*N (mixed stream width: G*N entries of Btilde then G*N of Ctilde), E experts,
 *     k = top_k.  Head h reads group h / (H/G).
 */
#ifndef SWIMBA_H_
#define SWIMBA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SWIMBA_OK 0
#define SWIMBA_ERR_NULL_ARG (-1)           /* a required pointer is NULL                      */
#define SWIMBA_ERR_BAD_CONFIG (-2)         /* a configuration field is out of range           */
#define SWIMBA_ERR_UNSUPPORTED_SHAPE (-3)  /* B, L or a size combination the kernels lack     */
#define SWIMBA_ERR_MISALIGNED (-4)         /* a tensor or the workspace is not 16-B aligned   */
#define SWIMBA_ERR_WORKSPACE_TOO_SMALL (-5)
#define SWIMBA_ERR_CUDA (-6)               /* a CUDA runtime/driver call failed               */
#define SWIMBA_ERR_DEVICE_TIMEOUT (-7)     /* a bounded device-side wait ran out              */
#define SWIMBA_ERR_DEVICE_BOUNDS (-8)      /* a device-side index check failed                */

#define SWIMBA_DTYPE_FP32 0
#define SWIMBA_DTYPE_BF16 1

/* Debug aid (no counterpart in the paper): kernels validate every index they read back from
 * device memory (expert indices, per-expert token lists and their lengths) before using it as an
 * address.  A bad value is skipped -- nothing is read or written through it -- and
 * SWIMBA_ERR_DEVICE_BOUNDS is recorded for swimba_status.  Costs one comparison per row. */
#define SWIMBA_FLAG_CHECK_INDICES 1

#define SWIMBA_MAX_EXPERTS 64
#define SWIMBA_MAX_TOPK 8

typedef struct swimba_handle swimba_handle; /* opaque, library-owned */

typedef struct {
    int32_t d_model;   /* F: width of the token features the router and experts read          */
    int32_t n_heads;   /* H                                                                    */
    int32_t head_dim;  /* P                                                                    */
    int32_t d_state;   /* N                                                                    */
    int32_t n_groups;  /* G, H % G == 0                                                        */
    int32_t n_experts; /* E, 1..SWIMBA_MAX_EXPERTS                                             */
    int32_t top_k;     /* k, 1..min(E, SWIMBA_MAX_TOPK); k == E is dense routing               */
    int32_t chunk;     /* Q in {64,128,256}: SSD chunk length (results do not depend on it)    */
    int32_t dtype;     /* SWIMBA_DTYPE_*                                                       */
    int32_t flags;     /* 0 or SWIMBA_FLAG_CHECK_INDICES; other bits are reserved              */
} swimba_config;

typedef struct {
    const void *W_router;  /* [E, F]        dtype; may be NULL when E == 1                     */
    const void *W_expert;  /* [E, S, F]     dtype; rows [0,GN) give B, rows [GN,2GN) give C    */
    const float *A;        /* [H]  negative reals                                              */
    const float *dt_bias;  /* [H]                                                              */
    const float *D;        /* [H]  skip weight, may be NULL (no skip term)                     */
} swimba_weights;

/* Create a layer handle.  Validates the configuration (Section "MoE-parameterized SSM":
 * E experts, k active, one shared transition) against what the kernels support:
 * F % 8 == 0, N % 16 == 0 and N <= 256, P <= 256, (N/16 rounded up to a power of two) * P <= 1024.
 * Uses the current CUDA device.  *out is set only on success.
 * Which kernels serve a configuration: with SWIMBA_DTYPE_BF16, P == 64 and N == 128 the SSD runs
 * on the tensor cores in 128-token tiles; every other shape, and SWIMBA_DTYPE_FP32, evaluates the
 * recurrence token by token with one block per (sequence, head), which is exact in fp32 but
 * serial over L (orders of magnitude slower on long sequences).  The expert projection uses the
 * tensor cores for SWIMBA_DTYPE_BF16 with F >= 64 and S % 32 == 0. */
int swimba_create(const swimba_config *cfg, swimba_handle **out);

/* Bytes of device workspace swimba_forward / swimba_route_mix / swimba_ssd need for B
 * sequences of L tokens (0 if B or L is not positive). */
size_t swimba_workspace_bytes(const swimba_handle *h, int32_t B, int32_t L);

/* Whole token-mixer forward: router -> top-k -> expert projection -> parameter-space mix ->
 * one chunked SSD evaluation (Section "MoE-parameterized SSM", state and output equations;
 * Theorem 1).
 *   u        [B,L,F]   dtype  token features read by the router and the experts
 *   x        [B,L,H,P] dtype  SSM input stream (shared by all experts)
 *   dt       [B,L,H]   float  raw (pre-softplus) step sizes, or NULL meaning dt == 0
 *   h0       [B,H,P,N] float  initial state, or NULL meaning zeros
 *   y        [B,L,H,P] dtype  out
 *   h_final  [B,H,P,N] float  out, may be NULL
 *   topk_idx [B,L,k]   int32  out, may be NULL: active experts, largest weight first, ties
 *                             to the lower expert index
 *   topk_w   [B,L,k]   float  out, may be NULL: their softmax values
 * L need not be a multiple of the chunk length.  B == 0 or L == 0 is a no-op returning OK.
 * Limits: B <= 65535 and B*L*k < 2^31 (SWIMBA_ERR_UNSUPPORTED_SHAPE beyond them). */
int swimba_forward(swimba_handle *h, const swimba_weights *w, const void *u, const void *x,
                   const float *dt, const float *h0, int32_t B, int32_t L, void *y,
                   float *h_final, int32_t *topk_idx, float *topk_w, void *workspace,
                   size_t workspace_bytes, void *cuda_stream);

/* First half of the forward only (router softmax equation, top-k rule, Theorem 1's mixed
 * streams): u[T,F] -> BC[T,S] dtype (Btilde then Ctilde), topk_idx[T,k], topk_w[T,k]
 * (either may be NULL).  A workspace sized by swimba_workspace_bytes(h, B, L) for any B*L == T
 * is large enough. */
int swimba_route_mix(swimba_handle *h, const swimba_weights *w, const void *u, int64_t T,
                     void *BC, int32_t *topk_idx, float *topk_w, void *workspace,
                     size_t workspace_bytes, void *cuda_stream);

/* Second half only: the single selective-SSM evaluation (selective-SSM equation; Background,
 * "Mamba-2 and SSD") on given mixed streams BC[B,L,S] dtype.  Other arguments as in
 * swimba_forward; w->W_router and w->W_expert are not read. */
int swimba_ssd(swimba_handle *h, const swimba_weights *w, const void *x, const void *BC,
               const float *dt, const float *h0, int32_t B, int32_t L, void *y, float *h_final,
               void *workspace, size_t workspace_bytes, void *cuda_stream);

/* How many segments the SSD evaluation cuts every sequence of a B x L call into (Background,
 * "Mamba-2 and SSD": a linear recurrence between blocks of tokens).  1: each sequence is walked
 * once with the carried state kept on chip.  More than 1 (long sequences, few of them): a first
 * pass computes every segment's end state, a scan chains them, a second pass produces y; the
 * workspace then holds segments * B*H*P*N floats of segment states.  0 if B or L is not
 * positive.  The result does not depend on the segmentation beyond rounding. */
int32_t swimba_ssd_segments(const swimba_handle *h, int32_t B, int32_t L);

/* The layer forward over a PACKED batch of sequences of different lengths (serving-shaped
 * batches: Section "Efficiency" measures prefill and decoding over mixes of batch size and input
 * length).  Sequence b of nseq holds tokens cu_seqlens[b] .. cu_seqlens[b+1]-1 of the packed arrays
 *   u [T, F] dtype, x [T, H, P] dtype, dt [T, H] fp32 or NULL, y [T, H, P] dtype out,
 *   topk_idx / topk_w [T, k] out (may be NULL),   T = cu_seqlens[nseq];
 * every sequence runs its own recurrence (Theorem 1) from h0[b] (h0 [nseq, H, P, N] fp32 or NULL =>
 * zeros) and leaves its end state in h_final[b] (may be NULL); a sequence of length 0 passes its
 * state through.  Routing, projection and mix are per token and see the batch as one run of T
 * tokens.  cu_seqlens is a HOST array of nseq + 1 non-decreasing offsets starting at 0; it is read
 * (and small tables derived from it are copied to the device, in stream order) before the call
 * returns, and may be freed then.  Everything else: device pointers, caller-owned, 16-byte aligned,
 * enqueued on cuda_stream.  The workspace must hold swimba_packed_workspace_bytes(h, cu_seqlens,
 * nseq) bytes (0 for invalid offsets or T == 0).  A sequence much longer than the batch's per-SM
 * share of tokens is cut into segments as in swimba_ssd_segments; swimba_packed_segments returns
 * the number of segments over the whole batch (nseq when nothing is cut).
 * Errors: as swimba_forward; SWIMBA_ERR_UNSUPPORTED_SHAPE for offsets that do not start at 0 or
 * decrease.  Rows of y outside every sequence do not exist; no byte outside y[0 .. T) is written. */
size_t swimba_packed_workspace_bytes(const swimba_handle *h, const int32_t *cu_seqlens, int32_t nseq);
int32_t swimba_packed_segments(const swimba_handle *h, const int32_t *cu_seqlens, int32_t nseq);
int swimba_forward_packed(swimba_handle *h, const swimba_weights *w, const void *u, const void *x,
                          const float *dt, const float *h0, const int32_t *cu_seqlens, int32_t nseq,
                          void *y, float *h_final, int32_t *topk_idx, float *topk_w, void *workspace,
                          size_t workspace_bytes, void *cuda_stream);

/* The layer forward with the SEQUENCE dimension sharded over n_ranks devices (one process per
 * device): rank r holds tokens [r L, (r+1) L) of each of the B sequences, in u [B,L,F], x [B,L,H,P],
 * dt [B,L,H].  The recurrence of Theorem 1 is linear in the state, so a shard is summarised by its
 * end state from a ZERO entry state and the product of a_t over the shard (Background, "Mamba-2 and
 * SSD": a linear recurrence between blocks of tokens; here the blocks are the ranks' shards).
 *   1. swimba_shard_summary: routing, projection, mix and a state-only pass over the local shard;
 *      writes summary_state [B,H,P,N] fp32 and summary_decay [B,H] fp32 (and the routing outputs,
 *      [B,L,k], may be NULL).  The mixed streams and intermediate states stay in the workspace.
 *   2. The caller gathers all ranks' summaries in rank order (one all-gather; the library holds no
 *      communicator): all_state [n_ranks,B,H,P,N], all_decay [n_ranks,B,H].  Rank 0 may pass NULL.
 *   3. swimba_shard_finish, with the SAME workspace, untouched in between, and the same x, B, L:
 *      chains h0 [B,H,P,N] (the state in front of rank 0's tokens; NULL => zeros; every rank passes
 *      the same) through the summaries of the ranks in front, produces y [B,L,H,P] of the local
 *      shard and h_end [B,H,P,N] (may be NULL), the state after the shard's last token (on the last
 *      rank: the sequence's final state).
 * bf16, head_dim 64, d_state 128 only (SWIMBA_ERR_UNSUPPORTED_SHAPE otherwise; the workspace query
 * then returns 0).  Device pointers, caller-owned, 16-byte aligned; everything is enqueued on
 * cuda_stream; errors as swimba_forward. */
size_t swimba_shard_workspace_bytes(const swimba_handle *h, int32_t B, int32_t L);
int swimba_shard_summary(swimba_handle *h, const swimba_weights *w, const void *u, const void *x,
                         const float *dt, int32_t B, int32_t L, float *summary_state, float *summary_decay,
                         int32_t *topk_idx, float *topk_w, void *workspace, size_t workspace_bytes,
                         void *cuda_stream);
int swimba_shard_finish(swimba_handle *h, const swimba_weights *w, const void *x, const float *h0,
                        const float *all_state, const float *all_decay, int32_t rank, int32_t n_ranks,
                        int32_t B, int32_t L, void *y, float *h_end, void *workspace, size_t workspace_bytes,
                        void *cuda_stream);

/* Backward pass for the weights the paper trains (Section "Training": the router and the expert
 * parameters; everything else in the layer is frozen): given dy [B,L,H,P] dtype, the gradient of a
 * scalar loss with respect to y, writes
 *   dW_router [E, F] fp32   and   dW_expert [E, 2*G*N, F] fp32
 * (overwritten; dW_router may be NULL when E == 1).  The forward's routing and mixed streams are
 * recomputed from u; the active sets K_t are constants of the differentiation and the kept weights
 * are differentiated as softmax values over all E (router equation, no renormalisation).  The
 * recurrence's adjoint (Theorem 1's state equation run backwards) gives dBtilde, dCtilde; the
 * mix, the softmax and the logits follow.  The final state does not enter the loss.  topk_idx
 * [B,L,k] (may be NULL) receives the active sets the gradients were taken with.  u, x, dt, h0 as
 * in swimba_forward; device pointers, caller-owned, 16-byte aligned; workspace of
 * swimba_backward_workspace_bytes(h, B, L) bytes.  Sums over tokens are accumulated with fp32
 * atomics: results are reproducible to rounding, not bit for bit.  Errors as swimba_forward;
 * SWIMBA_ERR_UNSUPPORTED_SHAPE when d_state * ceil(head_dim / 16) exceeds 1024 threads. */
size_t swimba_backward_workspace_bytes(const swimba_handle *h, int32_t B, int32_t L);
int swimba_backward_weights(swimba_handle *h, const swimba_weights *w, const void *u, const void *x,
                            const float *dt, const float *h0, const void *dy, int32_t B, int32_t L,
                            float *dW_router, float *dW_expert, int32_t *topk_idx, void *workspace,
                            size_t workspace_bytes, void *cuda_stream);

/* The general form of the layer, with expert-specific SSM inputs (the state equation of Section
 * "MoE-parameterized SSM" as printed: h_t = A h_{t-1} + sum_{e in K_t} pi_{t,e} B_t^(e) X_t^(e)^T,
 * Y_t = (sum_{e in K_t} pi_{t,e} C_t^(e))^T h_t).  The caller's experts produce X^(e) themselves (in
 * the paper they are in-projection layers), so the work is cut in two calls around that step:
 *
 * swimba_route_project_slots: router + projection WITHOUT the mix.
 *   u [T,F] dtype -> BC_slots [T,k,S] dtype: row (t, j) = pi_{t,e} [B_t^(e) ; C_t^(e)] for the j-th
 *   active expert e = topk_idx[t,j] (weight already applied), topk_idx [T,k], topk_w [T,k] (may be
 *   NULL).  Workspace as for swimba_route_mix.
 *
 * swimba_ssd_slots: the single recurrence on those streams.
 *   x_slots  [k,B,L,H,P] dtype  slot j holds, for every token, X^(e) of its j-th active expert
 *   BC_slots [B*L,k,S]   dtype  as produced above
 *   dt, h0, y, h_final as in swimba_forward; there is no skip term (w->D is not read).
 * The injection is linear in (B^(e), X^(e)), so the call evaluates k ordinary chunked recurrences
 * (one per slot, each with its own injection stream and the readout stream mixed over all slots)
 * and adds them; cost is k times swimba_ssd plus two streaming passes per extra slot, and the state
 * stays [B,H,P,N] whatever E is (Theorem 1).  Workspace: swimba_ssd_slots_workspace_bytes. */
int swimba_route_project_slots(swimba_handle *h, const swimba_weights *w, const void *u, int64_t T,
                               void *BC_slots, int32_t *topk_idx, float *topk_w, void *workspace,
                               size_t workspace_bytes, void *cuda_stream);
size_t swimba_ssd_slots_workspace_bytes(const swimba_handle *h, int32_t B, int32_t L);
int swimba_ssd_slots(swimba_handle *h, const swimba_weights *w, const void *x_slots,
                     const void *BC_slots, const float *dt, const float *h0, int32_t B, int32_t L,
                     void *y, float *h_final, void *workspace, size_t workspace_bytes,
                     void *cuda_stream);

/* The whole block around the mixer (Section "Swimba layer": the in-projection of a Mamba-2 block
 * becomes a mixture of expert projections, "the rest of the Mamba-2 layer is kept unchanged"; that
 * rest is the public Mamba-2 block):
 *   [z | x' | dt] = W_in u               shared in-projection: D = H*P gate columns, D input columns,
 *                                        H raw step sizes
 *   [B' | C']     = router, top-k, expert projections, parameter-space mix of u (as swimba_route_mix)
 *   [x | B | C]   = silu(causal depthwise conv of width d_conv over [x' | B' | C'])
 *   y             = the single selective-SSM recurrence on (x, B, C, dt), skip term included
 *   out           = W_out ( rmsnorm over each of the G channel groups of y * silu(z), times norm_w )
 * Weights (device pointers): W_in [2D + H, F] dtype; conv_w [D + S, d_conv] float, tap d_conv - 1
 * multiplies the current token; conv_b [D + S] float or NULL; norm_w [D] float; W_out [F, D] dtype.
 *   u [B,L,F] -> out [B,L,F] dtype.  conv_state_in / conv_state_out [B, d_conv - 1, D + S] dtype: the
 * d_conv - 1 pre-convolution rows before / at the end of the call (NULL: zeros / not wanted); with
 * h0 / h_final they carry a sequence across calls (chunked prefill).  d_conv in 1..4, P % 8 == 0.
 * Linear maps whose width is not a multiple of 32 run on the CUDA cores. */
typedef struct {
    const void *W_in;
    const float *conv_w;
    const float *conv_b;
    const float *norm_w;
    const void *W_out;
    int32_t d_conv;
    float eps;
} swimba_block_weights;
size_t swimba_block_workspace_bytes(const swimba_handle *h, int32_t B, int32_t L);
int swimba_block_forward(swimba_handle *h, const swimba_weights *w, const swimba_block_weights *bw,
                         const void *u, const void *conv_state_in, const float *h0, int32_t B,
                         int32_t L, void *out, void *conv_state_out, float *h_final,
                         int32_t *topk_idx, float *topk_w, void *workspace, size_t workspace_bytes,
                         void *cuda_stream);

/* Bytes of device workspace swimba_decode_step needs for B sequences. */
size_t swimba_decode_workspace_bytes(const swimba_handle *h, int32_t B);

/* One autoregressive step (the recurrence of Theorem 1 advanced by one token per sequence,
 * the O(T) inference mode of Background "Mamba-2 and SSD"): routes and mixes the B tokens,
 * then state <- a*state + Delta x Btilde^T in place and y = state Ctilde + D x.
 *   u [B,F] dtype, x [B,H,P] dtype, dt [B,H] float or NULL, state [B,H,P,N] float in/out,
 *   y [B,H,P] dtype out, topk_idx [B,k] / topk_w [B,k] out or NULL. */
int swimba_decode_step(swimba_handle *h, const swimba_weights *w, const void *u, const void *x,
                       const float *dt, float *state, int32_t B, void *y, int32_t *topk_idx,
                       float *topk_w, void *workspace, size_t workspace_bytes, void *cuda_stream);

/* End-to-end variant of swimba_forward for callers whose activations live in HOST memory
 * (pinned memory makes the copies asynchronous): copies u_host, x_host, dt_host (may be NULL)
 * to device staging, runs the forward of Theorem 1, copies y (and h_final / topk outputs when
 * given) back; the batch goes through in slices so that the copies in, the kernels and the copies
 * out of successive slices overlap (two copy streams owned by the handle, the kernels on the given
 * stream): up to eight slices of whole sequences, or, with fewer than eight sequences, runs of
 * consecutive tokens (multiples of 256) of one sequence at a time, the state carried from run to
 * run (Theorem 1: the recurrence needs nothing else from the past), about sixteen slices in all.  The given stream ends after the last copy out: the
 * caller synchronises it before reading.
 * Weights stay device pointers.  The workspace holds the staging buffers as well and is sized
 * by swimba_host_workspace_bytes. */
size_t swimba_host_workspace_bytes(const swimba_handle *h, int32_t B, int32_t L);
int swimba_forward_host(swimba_handle *h, const swimba_weights *w, const void *u_host,
                        const void *x_host, const float *dt_host, int32_t B, int32_t L,
                        void *y_host, float *h_final_host, int32_t *topk_idx_host,
                        float *topk_w_host, void *workspace, size_t workspace_bytes,
                        void *cuda_stream);

/* Allocation-free variant of swimba_route_mix (the paper has no counterpart: this is a
 * packaging convenience).  For callers that cannot allocate device memory where they call the
 * library -- a plug-in that is handed only its input and output buffers, a serving process whose
 * memory pool is fully handed out, set-up code that runs before any allocator exists -- the
 * scratch of the routing/projection stage lives in a fixed array inside the library image instead
 * of a caller-provided workspace.  Same arguments and results as swimba_route_mix, minus the
 * workspace.
 *   - The array is SWIMBA_STATIC_SCRATCH_BYTES large and is held by every GPU that loads the
 *     library until the process exits.  Token counts whose scratch need exceeds it are rejected
 *     with SWIMBA_ERR_WORKSPACE_TOO_SMALL and a message naming both sizes (the need is 8 k bytes per
 *     token for the routing outputs plus, on the bf16 tensor-core path, 4 E bytes per token of
 *     per-expert lists and, for k > 2, 2 k S bytes of per-slot projections: about 170000 tokens
 *     per call with E = 8, k = 2; about 5000 with S = 256, k = 3).
 *   - The first call on each device looks up the array's device address; make that first call
 *     outside any stream capture.  No call allocates or frees device memory.
 *   - All calls on a device share the one array, and it keeps the previous call's contents (the
 *     entry point clears the part that must start at zero).  Two calls that overlap on the GPU,
 *     e.g. on different streams, race on it: serialise them. */
#define SWIMBA_STATIC_SCRATCH_BYTES (8 * 1024 * 1024)
int swimba_route_mix_static(swimba_handle *h, const swimba_weights *w, const void *u, int64_t T,
                            void *BC, int32_t *topk_idx, float *topk_w, void *cuda_stream);

/* Optional per-kernel timing (no counterpart in the paper; measurement aid).  While enabled,
 * every kernel a call enqueues is bracketed by CUDA events on the call's stream.
 * swimba_profile_read synchronises that stream and returns how many kernels the most recent call
 * (for swimba_forward_host: its last batch slice) launched (at most max_entries), with kernel_ids[i] in 1..24 (1 router + grouping by
 * expert (for fewer than about 28000 tokens the launch also computes the SSD step sizes), 4 expert GEMM, 5 slot mix, 6 SIMT projection, 7 per-timestep SSM, 8 decode update, 9 SSD
 * tile kernel, 10 segment scan, 11 SSD step sizes and decays, 12 slot stream assembly, 13 slot sum, 14 small-batch projection, 15 convolution + SiLU, 16 gated norm, 17 step-size columns, 18 adjoint recurrence pass, 19 router softmax over all experts, 20 weight / logit adjoints, 21 router-matrix gradient, 22 expert-matrix gradient, 23 operand re-arrangement / head sum of the tile-kernel adjoint, 24 state-only SSD pass; 2 and 3 are not in use) and ms[i] its duration in milliseconds.
 * Both arrays are HOST arrays. */
int swimba_profile(swimba_handle *h, int enable);
int swimba_profile_read(swimba_handle *h, int32_t *kernel_ids, float *ms, int32_t max_entries);

/* Self-test of the failure path (no counterpart in the paper).  Every device-side wait in the
 * tensor-core kernels is bounded: when it runs out, the kernel records
 * SWIMBA_ERR_DEVICE_TIMEOUT, makes its later waits return at once and runs to its normal exit.
 * This call exercises exactly that code on a barrier that nothing signals: one warp waits for
 * limit_cycles SM cycles (1e3 .. 1e8), gives up, and waits once more.  Afterwards swimba_status
 * returns SWIMBA_ERR_DEVICE_TIMEOUT (and clears it), and the handle stays usable.
 *   result_host  HOST array of 3, may be NULL; when given the call synchronises the stream and
 *                returns {first wait gave up (1/0), second wait gave up (1/0), cycles the second
 *                wait took}. */
int swimba_selftest_wait(swimba_handle *h, int64_t limit_cycles, int64_t *result_host,
                         void *cuda_stream);

/* Number of kernels the most recent forward/route_mix/ssd/decode call on this handle enqueued. */
int swimba_last_launch_count(const swimba_handle *h);

/* Synchronises the stream of the most recent call, then returns SWIMBA_OK or the error code the
 * device recorded (bounded waits that ran out, failed index checks) and clears it. */
int swimba_status(swimba_handle *h);

/* Human-readable description of the most recent error on this handle ("" if none). */
const char *swimba_last_error(const swimba_handle *h);

/* Frees the handle and its device status word.  NULL is allowed. */
void swimba_destroy(swimba_handle *h);

#ifdef __cplusplus
}
#endif
#endif /* SWIMBA_H_ */
