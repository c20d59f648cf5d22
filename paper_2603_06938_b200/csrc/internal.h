// Launchers shared between the API translation unit and the kernel files.
#pragma once
#include "common.cuh"
#include "ssd_scalars.cuh"

namespace swimba {

// K1a: router logits, softmax over all E, top-k (indices + un-renormalised weights).
// When counts is given (zeroed beforehand) the (token, slot) pairs are also grouped by expert:
// perm[e * cap + i], i < counts[e], lists the entries t*k + j routed to expert e.
// zero_out (may be NULL): a [T, zero_bytes_per_token] buffer the kernel clears on the way (the
// mixed streams, when the projection adds its slots in place).  scalars.l2 != NULL: the call also
// produces the SSD step sizes and tile log-decays of the same forward (they depend on dt only and
// run beside the router, inside its launch or as a kernel in front of it).
int launch_router(LaunchCtx &ctx, int dtype, const void *u, const void *W_r, int64_t T, int F,
                  int E, int k, int32_t *idx, float *w, int *counts, int *perm, int64_t cap,
                  int sm_count, void *zero_out, int zero_bytes_per_token, const ScalarsArgs &scalars);

// K1b (tensor cores): grouped GEMM over the per-expert lists + slot sum.  `workspace` is sized
// by expert_gemm_workspace_bytes and holds the histogram (zeroed by the caller before the
// router runs), the per-expert lists (capacity T each) and the per-slot projections.
size_t expert_gemm_workspace_bytes(int64_t T, int S, int E, int k);
bool expert_gemm_supported(int F, int S);
bool expert_gemm_adds_rows(int k);   // true: BC must be zero before launch_expert_gemm runs
int *expert_gemm_counts(void *workspace);
int *expert_gemm_perm(void *workspace);
// slots_out (may be NULL): [T*k, S] bf16; when given, the projection of (token t, slot j), scaled by
// its router weight, is stored in row t*k + j and nothing is mixed (BC is not touched).
int launch_expert_gemm(LaunchCtx &ctx, const void *u, const void *W_e, const float *w, int64_t T,
                       int F, int S, int E, int k, int sm_count, void *BC, void *workspace,
                       void *slots_out = nullptr);

// K1b (SIMT): project the k selected experts and mix.  BC is written in `dtype`, or as float
// per slot-sum when bc_fp32 is set.
int launch_project_mix_simt(LaunchCtx &ctx, int dtype, const void *u, const void *W_e,
                            const int32_t *idx, const float *w, int64_t T, int F, int S, int E,
                            int k, void *BC, bool bc_fp32);
// The same without the mix: row t*k + j of slots_out (dtype) = w[t,j] * W_e[idx[t,j]] u_t.
int launch_project_slots_simt(LaunchCtx &ctx, int dtype, const void *u, const void *W_e,
                              const int32_t *idx, const float *w, int64_t T, int F, int S, int E,
                              int k, void *slots_out);

// General injection (expert-specific SSM inputs) helpers, all dtype-generic streaming kernels:
//   assemble: BCj[t, :] = [ slots[t*k + j, 0:GN] | sum_j' slots[t*k + j', GN:2GN] ]
//   accumulate: y += y_add (dtype, fp32 sum), h += h_add (float); either pair may be NULL
int launch_assemble_slot_streams(LaunchCtx &ctx, int dtype, const void *slots, int64_t T, int S, int k,
                                 int j, void *BCj);
int launch_accumulate(LaunchCtx &ctx, int dtype, void *y, const void *y_add, int64_t ny, float *h,
                      const float *h_add, int64_t nh);

// K1 for at most a few hundred tokens (decode): two short kernels, no lists in global memory.
// idx [T,k], w [T,k] and the fp32 mixed streams BC [T,S] are written.
bool front_small_supported(int dtype, int64_t T, int F, int S, int E, int k);
int launch_front_small(LaunchCtx &ctx, const void *u, const void *W_r, const void *W_e, int64_t T, int F,
                       int S, int E, int k, int32_t *idx, float *w, float *BC);

// K2/K3 (tensor cores): tiled SSD with the carried state kept on chip; bf16, P == 64, N == 128.
bool ssd_tiles_supported(int dtype, int P, int N);
size_t ssd_workspace_bytes(int B, int L, int H, int G, int chunk, int sm_count);
// Tokens per segment the tile path cuts a sequence into (a multiple of 128; >= L: one segment).
int ssd_segment_len(int B, int L, int H, int G, int chunk, int sm_count);
// scalars_done: the step sizes and tile log-decays (ssd_scalars_args over the same workspace) have
// already been produced earlier in the stream (launch_router with scalars, or launch_ssd_scalars).
ScalarsArgs ssd_scalars_args(const float *dt, const float *A, const float *dt_bias, int B, int L, int H,
                             void *workspace);
int launch_ssd_scalars(LaunchCtx &ctx, const ScalarsArgs &args);
int launch_ssd_tiles(LaunchCtx &ctx, const void *x, const void *BC, const float *dt, const float *A,
                     const float *dt_bias, const float *D, const float *h0, int B, int L, int H, int G,
                     int chunk, int sm_count, void *y, float *h_final, void *workspace,
                     bool scalars_done);

// The same over a packed batch: nseq sequences back to back in [T, ...] arrays, sequence b holding
// tokens cu[b] .. cu[b+1]-1 (cu is a HOST array of nseq + 1 entries, read before the call returns).
// h0 / h_final are [nseq, H, P, N].  The step sizes are produced inside the call.
size_t ssd_packed_workspace_bytes(const int32_t *cu, int nseq, int H, int G, int chunk, int sm_count);
int ssd_packed_segments(const int32_t *cu, int nseq, int H, int G, int chunk, int sm_count);
int launch_ssd_tiles_packed(LaunchCtx &ctx, const void *x, const void *BC, const float *dt, const float *A,
                            const float *dt_bias, const float *D, const float *h0, const int32_t *cu, int nseq,
                            int H, int G, int chunk, int sm_count, void *y, float *h_final, void *workspace);

// Sequence-sharded evaluation (every rank holds L consecutive tokens of each of B sequences), in two
// halves around the exchange of the ranks' summaries.  summary: state-only pass + local scan from a
// zero entry state; sum_state [B,H,P,N] and sum_decay [B,H] receive the shard's end state and the
// product of a_t over the shard; the workspace keeps the step sizes and the zero-entry segment
// states for the second half.  finish: all_state [R,B,H,P,N] / all_decay [R,B,H] are the gathered
// summaries in rank order; the state entering this rank's shard is chained from h0 through the
// ranks in front, y [B,L,H,P] is produced and h_end [B,H,P,N] (may be NULL) is the state after the
// shard's last token.
size_t ssd_shard_workspace_bytes(int B, int L, int H, int G, int chunk, int sm_count);
ScalarsArgs ssd_shard_scalars_args(const float *dt, const float *A, const float *dt_bias, int B, int L, int H,
                                   int G, int chunk, int sm_count, void *workspace);
int launch_ssd_shard_summary(LaunchCtx &ctx, const void *x, const void *BC, const float *dt, const float *A,
                             const float *dt_bias, int B, int L, int H, int G, int chunk, int sm_count,
                             float *sum_state, float *sum_decay, void *workspace, bool scalars_done);
int launch_ssd_shard_finish(LaunchCtx &ctx, const void *x, const void *BC, const float *D, const float *h0,
                            const float *all_state, const float *all_decay, int rank, int B, int L, int H, int G,
                            int chunk, int sm_count, void *y, float *h_end, void *workspace);

// Backward for the trained weights (router and expert matrices), plain CUDA-core kernels.
// adjoint: both passes of the recurrence's adjoint; dBC [T,S] fp32 (zeroed by the caller) receives
// dBtilde | dCtilde.  weight_grads: softmax over all E (pi [T,E] scratch), dpi / dg (dg [T,E]
// scratch) from the unscaled slot projections slots [T*k,S] (dtype), then dW_r [E,F] and dW_e
// [E,S,F] (fp32, zeroed by the caller, accumulated with atomics).
bool ssd_adjoint_supported(int P, int N);
int launch_fill(LaunchCtx &ctx, float *p, int64_t n, float v);
int launch_ssd_adjoint(LaunchCtx &ctx, int dtype, const void *x, const void *dy, const void *BC, const float *dt,
                       const float *A, const float *dt_bias, const float *h0, int B, int L, int H, int P, int N,
                       int G, float *dBC);
// The same adjoint through the forward's tile kernel (bf16, P = 64, N = 128): both passes are
// evaluations of a virtual layer of 2H heads in H groups; dBC is overwritten, not accumulated.
size_t ssd_adjoint_tiles_workspace_bytes(int B, int L, int H, int chunk, int sm_count);
int launch_ssd_adjoint_tiles(LaunchCtx &ctx, const void *x, const void *dy, const void *BC, const float *dt,
                             const float *A, const float *dt_bias, const float *h0, int B, int L, int H, int G,
                             int chunk, int sm_count, float *dBC, void *workspace);
int launch_weight_grads(LaunchCtx &ctx, int dtype, const void *u, const void *W_r, const void *slots,
                        const int32_t *idx, const float *w, const float *dBC, int64_t Tn, int F, int S, int E,
                        int k, float *pi, float *dg, float *dW_r, float *dW_e);

// One warp waiting on a barrier nobody signals, with the given limit (see swimba_selftest_wait).
// out_dev: three 64-bit words on the device.
int launch_wait_selftest(LaunchCtx &ctx, long long limit_cycles, long long *out_dev);

// The rest of the block: causal depthwise convolution + SiLU over the channels [x' (D columns of a
// matrix with row stride ldx) | B'C' (S)], gated RMS norm, step-size columns to fp32.
int launch_conv_silu(LaunchCtx &ctx, int dtype, const void *xp, int64_t ldx, const void *bcp, const float *cw,
                     const float *cb, const void *state_in, int B, int L, int D, int S, int K, void *x,
                     void *bc, void *state_out);
int launch_gated_rmsnorm(LaunchCtx &ctx, int dtype, const void *y, const void *z, int64_t ldz, const float *wt,
                         int64_t T, int D, int ngroups, float eps, void *out);
int launch_dt_columns(LaunchCtx &ctx, int dtype, const void *zxdt, int64_t ld, int off, int64_t T, int H, float *dt);

// Per-timestep SIMT evaluation of the recurrence (fp32 state in registers).
int launch_ssd_sequential(LaunchCtx &ctx, int dtype, const void *x, const void *BC, bool bc_fp32,
                          const float *dt, const float *A, const float *dt_bias, const float *D,
                          const float *h0, int B, int L, int H, int P, int N, int G, void *y,
                          float *h_final);

// The per-timestep evaluation over n listed sequences of a packed batch (bf16 streams): seq_tab[i] =
// (first token, tokens, sequence index, 0), a device array; x, BC, dt, y are the packed arrays, h0 /
// h_final are indexed by the sequence.
int launch_ssd_sequential_listed(LaunchCtx &ctx, const void *x, const void *BC, const float *dt, const float *A,
                                 const float *dt_bias, const float *D, const float *h0, const int4 *seq_tab, int n,
                                 int H, int P, int N, int G, void *y, float *h_final);

// K4: one-token state update, state[B,H,P,N] in place.
// BC [B,S] is fp32 when bc_fp32, else bf16.
int launch_decode_update(LaunchCtx &ctx, int dtype, const void *x, const void *BC, bool bc_fp32,
                         const float *dt, const float *A, const float *dt_bias, const float *D,
                         float *state, int B, int H, int P, int N, int G, int sm_count, void *y);

}  // namespace swimba
