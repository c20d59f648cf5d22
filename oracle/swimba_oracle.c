/*
 * Swimba token-mixer oracle: plain, slow, double-precision CPU code.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing on the product path may call into this
 * file; it exists so that the CUDA library can be compared against an
 * independent statement of what the method computes.  It shares no code,
 * header, table or helper with the CUDA sources.
 *
 * Every function takes HOST pointers to row-major arrays of double (int for
 * indices) and follows the paper's steps in the paper's order:
 *
 *   router      : g_t = W_r u_t,  pi_t = softmax(g_t) over all E experts
 *                 (Background, "Mixture of Experts", router softmax equation);
 *                 top-k keeps the softmax values of the k largest entries and
 *                 does not renormalise (same paragraph).
 *   streams     : B_t^(e), C_t^(e) are expert-specific linear maps of the same
 *                 token features (Section "MoE-parameterized SSM").
 *   mix         : Btilde_t = sum_{e in K_t} pi_{t,e} B_t^(e), Ctilde_t likewise
 *                 (Theorem 1, definition of the mixed streams).
 *   recurrence  : h_t = a_t h_{t-1} + Delta_t Btilde_t x_t^T,
 *                 y_t = Ctilde_t^T h_t + D x_t, channel by channel
 *                 (selective-SSM equation, Mamba-2 channelwise convention;
 *                 Theorem 1).  The transition is shared by all experts
 *                 (shared-A equation) and is the scalar a_{t,h} =
 *                 exp(Delta_{t,h} A_h) per head, Delta = softplus(dt+dt_bias).
 *   separated   : h_t^(e) = a_t h_{t-1}^(e) + Delta_t B_t^(e) x_t^(e)T,
 *                 y_t = sum_{e in K_t} pi_{t,e} C_t^(e)T h_t^(e)
 *                 (Section "Alternative: MoE of separated SSMs").
 *
 * Layouts (last index contiguous):
 *   u[T,F]  W_r[E,F]  W_e[E,S,F] with S = 2*G*N, rows [0,GN) -> B, [GN,2GN) -> C
 *   BC[T,S] = [Btilde (G*N) | Ctilde (G*N)]      x,y[B,L,H,P]     dt[B,L,H]
 *   state h[B,H,P,N]      head h reads group h / (H/G).
 *
 * Return value: 0 on success, a negative number for an invalid argument.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_BAD_ARG (-1)
#define ORACLE_NO_MEM (-2)

static double softplus(double v) {
    /* log(1 + e^v), written so that neither branch overflows */
    return (v > 0.0 ? v : 0.0) + log1p(exp(-fabs(v)));
}

/* ---------------------------------------------------------------------------
 * Router (router softmax equation; top-k rule of the same paragraph).
 *   idx[T,k]    experts kept, ordered by decreasing logit, ties -> lower index
 *   w[T,k]      their softmax values (softmax over ALL E, no renormalisation)
 *   pi[T,E]     optional: full softmax
 *   margin[T]   optional: smallest gap between consecutive logits among the
 *               k+1 largest (k largest when k == E): how far the selection and
 *               its order are from changing
 *   absdot[T]   optional: max_e sum_f |W_r[e,f] u[t,f]|, the scale against
 *               which a lower-precision logit error is bounded
 * ------------------------------------------------------------------------- */
int oracle_router(const double *u, const double *W_r, long T, int F, int E, int k,
                  int *idx, double *w, double *pi, double *margin, double *absdot)
{
    if (!u || !W_r || !idx || !w || T < 0 || F <= 0 || E <= 0 || k <= 0 || k > E)
        return ORACLE_BAD_ARG;
    int fail = 0;
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t) {
        double *g = (double *)malloc(sizeof(double) * (size_t)E * 2);
        int *taken = (int *)calloc((size_t)E, sizeof(int));
        if (!g || !taken) { fail = 1; free(g); free(taken); continue; }
        double *p = g + E;
        double amax = 0.0;
        for (int e = 0; e < E; ++e) {
            double s = 0.0, sa = 0.0;
            for (int f = 0; f < F; ++f) {
                double term = W_r[(long)e * F + f] * u[t * F + f];
                s += term;
                sa += fabs(term);
            }
            g[e] = s;
            if (sa > amax) amax = sa;
        }
        double m = g[0];
        for (int e = 1; e < E; ++e) if (g[e] > m) m = g[e];
        double z = 0.0;
        for (int e = 0; e < E; ++e) { p[e] = exp(g[e] - m); z += p[e]; }
        for (int e = 0; e < E; ++e) p[e] /= z;
        if (pi) for (int e = 0; e < E; ++e) pi[t * E + e] = p[e];
        /* k (+1) rounds of "largest remaining logit, lowest index on ties" */
        double gap = INFINITY, prev = 0.0;
        int rounds = (k < E) ? k + 1 : k;
        for (int j = 0; j < rounds; ++j) {
            int best = -1;
            for (int e = 0; e < E; ++e)
                if (!taken[e] && (best < 0 || g[e] > g[best])) best = e;
            taken[best] = 1;
            if (j > 0 && prev - g[best] < gap) gap = prev - g[best];
            prev = g[best];
            if (j < k) { idx[t * k + j] = best; w[t * k + j] = p[best]; }
        }
        if (margin) margin[t] = gap;
        if (absdot) absdot[t] = amax;
        free(g); free(taken);
    }
    return fail ? ORACLE_NO_MEM : ORACLE_OK;
}

/* ---------------------------------------------------------------------------
 * Expert streams for EVERY expert (Section "MoE-parameterized SSM"):
 *   BCe[t,e,:] = W_e[e] u_t.   Small cases only (dense over E).
 * ------------------------------------------------------------------------- */
int oracle_expert_streams(const double *u, const double *W_e, long T, int F, int S, int E,
                          double *BCe)
{
    if (!u || !W_e || !BCe || T < 0 || F <= 0 || S <= 0 || E <= 0) return ORACLE_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t)
        for (int e = 0; e < E; ++e)
            for (int s = 0; s < S; ++s) {
                double acc = 0.0;
                const double *wrow = W_e + ((long)e * S + s) * F;
                for (int f = 0; f < F; ++f) acc += wrow[f] * u[t * F + f];
                BCe[(t * E + e) * S + s] = acc;
            }
    return ORACLE_OK;
}

/* ---------------------------------------------------------------------------
 * Parameter-space mix over the active set (Theorem 1, mixed streams):
 *   BC[t,:] = sum_j w[t,j] * (W_e[idx[t,j]] u_t).
 * Only the k selected experts are projected.
 * ------------------------------------------------------------------------- */
int oracle_mix_topk(const double *u, const double *W_e, long T, int F, int S, int E, int k,
                    const int *idx, const double *w, double *BC)
{
    if (!u || !W_e || !idx || !w || !BC || T < 0 || F <= 0 || S <= 0 || E <= 0 || k <= 0)
        return ORACLE_BAD_ARG;
    for (long i = 0; i < T * k; ++i) if (idx[i] < 0 || idx[i] >= E) return ORACLE_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t)
        for (int s = 0; s < S; ++s) {
            double mixed = 0.0;
            for (int j = 0; j < k; ++j) {
                const double *wrow = W_e + ((long)idx[t * k + j] * S + s) * F;
                double proj = 0.0;
                for (int f = 0; f < F; ++f) proj += wrow[f] * u[t * F + f];
                mixed += w[t * k + j] * proj;
            }
            BC[t * S + s] = mixed;
        }
    return ORACLE_OK;
}

/* Same mix with arbitrary dense weights pi[T,E] (zero = inactive expert). */
int oracle_mix_dense(const double *u, const double *W_e, long T, int F, int S, int E,
                     const double *pi, double *BC)
{
    if (!u || !W_e || !pi || !BC || T < 0 || F <= 0 || S <= 0 || E <= 0) return ORACLE_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t)
        for (int s = 0; s < S; ++s) {
            double mixed = 0.0;
            for (int e = 0; e < E; ++e) {
                if (pi[t * E + e] == 0.0) continue;
                const double *wrow = W_e + ((long)e * S + s) * F;
                double proj = 0.0;
                for (int f = 0; f < F; ++f) proj += wrow[f] * u[t * F + f];
                mixed += pi[t * E + e] * proj;
            }
            BC[t * S + s] = mixed;
        }
    return ORACLE_OK;
}

/* ---------------------------------------------------------------------------
 * The single selective-SSM recurrence on given (already mixed) streams
 * (selective-SSM equation with the channelwise convention; Theorem 1).
 *   for t = 0..L-1, every head h, channel p, state index n:
 *     Delta = softplus(dt[b,t,h] + dt_bias[h])   (dt == NULL -> dt = 0)
 *     a     = exp(Delta * A[h])
 *     h[p,n] <- a * h[p,n] + Delta * x[b,t,h,p] * Btilde[b,t,g(h),n]
 *     y[b,t,h,p] = sum_n Ctilde[b,t,g(h),n] * h[p,n] + D[h] * x[b,t,h,p]
 *   h0 == NULL -> zero initial state; D == NULL -> no skip term.
 *   h_final[B,H,P,N] optional; h_traj[B,L,H,P,N] optional (tiny cases).
 * ------------------------------------------------------------------------- */
int oracle_ssm_recurrence(const double *x, const double *BC, const double *dt,
                          const double *A, const double *dt_bias, const double *D,
                          const double *h0, int B, int L, int H, int P, int N, int G,
                          double *y, double *h_final, double *h_traj)
{
    if (!x || !BC || !A || !dt_bias || !y || B < 0 || L < 0 || H <= 0 || P <= 0 || N <= 0 ||
        G <= 0 || H % G != 0)
        return ORACLE_BAD_ARG;
    const int S = 2 * G * N, hpg = H / G;
    int fail = 0;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            double *st = (double *)malloc(sizeof(double) * (size_t)P * N);
            if (!st) { fail = 1; continue; }
            for (int i = 0; i < P * N; ++i)
                st[i] = h0 ? h0[((long)b * H + h) * P * N + i] : 0.0;
            const int g = h / hpg;
            for (int t = 0; t < L; ++t) {
                const long bt = (long)b * L + t;
                const double *Bt = BC + bt * S + (long)g * N;
                const double *Ct = BC + bt * S + (long)(G + g) * N;
                const double delta = softplus((dt ? dt[bt * H + h] : 0.0) + dt_bias[h]);
                const double a = exp(delta * A[h]);
                for (int p = 0; p < P; ++p) {
                    const double xv = x[(bt * H + h) * P + p];
                    double *sp = st + (long)p * N;
                    double acc = 0.0;
                    for (int n = 0; n < N; ++n) {
                        sp[n] = a * sp[n] + delta * xv * Bt[n];
                        acc += Ct[n] * sp[n];
                    }
                    y[(bt * H + h) * P + p] = acc + (D ? D[h] * xv : 0.0);
                }
                if (h_traj)
                    memcpy(h_traj + ((bt * H + h) * (long)P) * N, st, sizeof(double) * (size_t)P * N);
            }
            if (h_final)
                memcpy(h_final + ((long)b * H + h) * P * N, st, sizeof(double) * (size_t)P * N);
            free(st);
        }
    return fail ? ORACLE_NO_MEM : ORACLE_OK;
}

/* ---------------------------------------------------------------------------
 * General mixed model with expert-specific input streams (state and output
 * equations of Section "MoE-parameterized SSM"):
 *     h_t = a_t h_{t-1} + Delta_t sum_e pi_{t,e} B_t^(e) x_t^(e)T
 *     y_t = (sum_e pi_{t,e} C_t^(e))^T h_t
 *   BCe[B,L,E,S] expert streams, xe[B,L,E,H,P] expert inputs, pi[B,L,E] dense
 *   weights (zero outside the active set).  No skip term.
 *   h_traj[B,L,H,P,N] optional.
 * ------------------------------------------------------------------------- */
int oracle_mixed_general(const double *xe, const double *BCe, const double *pi,
                         const double *dt, const double *A, const double *dt_bias,
                         const double *h0, int B, int L, int E, int H, int P, int N, int G,
                         double *y, double *h_final, double *h_traj)
{
    if (!xe || !BCe || !pi || !A || !dt_bias || !y || H <= 0 || G <= 0 || H % G != 0 || E <= 0)
        return ORACLE_BAD_ARG;
    const int S = 2 * G * N, hpg = H / G;
    int fail = 0;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            double *st = (double *)malloc(sizeof(double) * (size_t)P * N);
            if (!st) { fail = 1; continue; }
            for (int i = 0; i < P * N; ++i)
                st[i] = h0 ? h0[((long)b * H + h) * P * N + i] : 0.0;
            const int g = h / hpg;
            for (int t = 0; t < L; ++t) {
                const long bt = (long)b * L + t;
                const double delta = softplus((dt ? dt[bt * H + h] : 0.0) + dt_bias[h]);
                const double a = exp(delta * A[h]);
                for (int p = 0; p < P; ++p) {
                    double *sp = st + (long)p * N;
                    double acc = 0.0;
                    for (int n = 0; n < N; ++n) {
                        double inj = 0.0, cmix = 0.0;
                        for (int e = 0; e < E; ++e) {
                            const double pe = pi[bt * E + e];
                            if (pe == 0.0) continue;
                            const double *row = BCe + (bt * E + e) * S;
                            inj += pe * row[(long)g * N + n] * xe[((bt * E + e) * H + h) * P + p];
                            cmix += pe * row[(long)(G + g) * N + n];
                        }
                        sp[n] = a * sp[n] + delta * inj;
                        acc += cmix * sp[n];
                    }
                    y[(bt * H + h) * P + p] = acc;
                }
                if (h_traj)
                    memcpy(h_traj + ((bt * H + h) * (long)P) * N, st, sizeof(double) * (size_t)P * N);
            }
            if (h_final)
                memcpy(h_final + ((long)b * H + h) * P * N, st, sizeof(double) * (size_t)P * N);
            free(st);
        }
    return fail ? ORACLE_NO_MEM : ORACLE_OK;
}

/* ---------------------------------------------------------------------------
 * MoE over separated SSMs (Section "Alternative: MoE of separated SSMs"):
 * every expert advances its own state at every step; only the readout is
 * restricted to the active set through pi (zero outside it).
 *   he_traj[B,L,E,H,P,N] optional (tiny cases); he_final[B,E,H,P,N] optional.
 *   All expert states start from zero (Theorem 4's assumption) unless h0e
 *   [B,E,H,P,N] is given.
 * ------------------------------------------------------------------------- */
int oracle_separated(const double *xe, const double *BCe, const double *pi,
                     const double *dt, const double *A, const double *dt_bias,
                     const double *h0e, int B, int L, int E, int H, int P, int N, int G,
                     double *y, double *he_final, double *he_traj)
{
    if (!xe || !BCe || !pi || !A || !dt_bias || !y || H <= 0 || G <= 0 || H % G != 0 || E <= 0)
        return ORACLE_BAD_ARG;
    const int S = 2 * G * N, hpg = H / G;
    const long PN = (long)P * N;
    int fail = 0;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H; ++h) {
            double *st = (double *)malloc(sizeof(double) * (size_t)E * PN);
            if (!st) { fail = 1; continue; }
            for (int e = 0; e < E; ++e)
                for (long i = 0; i < PN; ++i)
                    st[e * PN + i] = h0e ? h0e[(((long)b * E + e) * H + h) * PN + i] : 0.0;
            const int g = h / hpg;
            for (int t = 0; t < L; ++t) {
                const long bt = (long)b * L + t;
                const double delta = softplus((dt ? dt[bt * H + h] : 0.0) + dt_bias[h]);
                const double a = exp(delta * A[h]);
                for (int p = 0; p < P; ++p) {
                    double out = 0.0;
                    for (int e = 0; e < E; ++e) {
                        const double *row = BCe + (bt * E + e) * S;
                        const double xv = xe[((bt * E + e) * H + h) * P + p];
                        double *sp = st + e * PN + (long)p * N;
                        double read = 0.0;
                        for (int n = 0; n < N; ++n) {
                            sp[n] = a * sp[n] + delta * row[(long)g * N + n] * xv;
                            read += row[(long)(G + g) * N + n] * sp[n];
                        }
                        out += pi[bt * E + e] * read;
                    }
                    y[(bt * H + h) * P + p] = out;
                }
                if (he_traj)
                    for (int e = 0; e < E; ++e)
                        memcpy(he_traj + (((bt * E + e) * H + h) * PN), st + e * PN,
                               sizeof(double) * (size_t)PN);
            }
            if (he_final)
                for (int e = 0; e < E; ++e)
                    memcpy(he_final + (((long)b * E + e) * H + h) * PN, st + e * PN,
                           sizeof(double) * (size_t)PN);
            free(st);
        }
    return fail ? ORACLE_NO_MEM : ORACLE_OK;
}

/* ---------------------------------------------------------------------------
 * Whole layer forward: router -> top-k -> project the selected experts ->
 * mix -> one recurrence.  forced_idx/forced_w (both or neither) replace the
 * router's decision; the router outputs are then copies of them.
 *   Outputs idx[T,k], w[T,k], BC[T,S] are optional.
 * ------------------------------------------------------------------------- */
int oracle_swimba_forward(const double *u, const double *x, const double *dt, const double *h0,
                          const double *W_r, const double *W_e, const double *A,
                          const double *dt_bias, const double *D,
                          int B, int L, int F, int H, int P, int N, int G, int E, int k,
                          const int *forced_idx, const double *forced_w,
                          double *y, double *h_final, int *idx_out, double *w_out, double *BC_out)
{
    if (!u || !x || !W_e || !A || !dt_bias || !y || B < 0 || L < 0 || F <= 0 || E <= 0 ||
        k <= 0 || k > E || N <= 0 || G <= 0)
        return ORACLE_BAD_ARG;
    if ((forced_idx == NULL) != (forced_w == NULL)) return ORACLE_BAD_ARG;
    if (!forced_idx && !W_r) return ORACLE_BAD_ARG;
    const long T = (long)B * L;
    const int S = 2 * G * N;
    int *idx = (int *)malloc(sizeof(int) * (size_t)(T * k + 1));
    double *w = (double *)malloc(sizeof(double) * (size_t)(T * k + 1));
    double *BC = (double *)malloc(sizeof(double) * (size_t)(T * S + 1));
    int rc = ORACLE_OK;
    if (!idx || !w || !BC) rc = ORACLE_NO_MEM;
    if (rc == ORACLE_OK) {
        if (forced_idx) {
            memcpy(idx, forced_idx, sizeof(int) * (size_t)(T * k));
            memcpy(w, forced_w, sizeof(double) * (size_t)(T * k));
        } else {
            rc = oracle_router(u, W_r, T, F, E, k, idx, w, NULL, NULL, NULL);
        }
    }
    if (rc == ORACLE_OK) rc = oracle_mix_topk(u, W_e, T, F, S, E, k, idx, w, BC);
    if (rc == ORACLE_OK)
        rc = oracle_ssm_recurrence(x, BC, dt, A, dt_bias, D, h0, B, L, H, P, N, G, y, h_final, NULL);
    if (rc == ORACLE_OK) {
        if (idx_out) memcpy(idx_out, idx, sizeof(int) * (size_t)(T * k));
        if (w_out) memcpy(w_out, w, sizeof(double) * (size_t)(T * k));
        if (BC_out) memcpy(BC_out, BC, sizeof(double) * (size_t)(T * S));
    }
    free(idx); free(w); free(BC);
    return rc;
}

/* ---------------------------------------------------------------------------
 * Gradients of  loss = sum_{b,t,h,p} dy[b,t,h,p] * y[b,t,h,p]  with respect to the router matrix
 * W_r and the expert matrices W_e (Section "Training": only the router and the expert
 * parameters that the conversion adds are trained, the rest of the layer is frozen), by
 * reverse-mode differentiation of oracle_swimba_forward's steps, taken in reverse order:
 *   recurrence   lambda_t = a_{t+1} lambda_{t+1} + dy_t Ctilde_t^T      (adjoint of the state)
 *                dCtilde_t[g,n] = sum_{h in g, p} dy_t[h,p] h_t[h,p,n]
 *                dBtilde_t[g,n] = Delta_t sum_{h in g, p} x_t[h,p] lambda_t[h,p,n]
 *   mix          dpi_{t,j} = <dBC_t, W_e[e_j] u_t>,   dW_e[e_j] += pi_{t,e_j} dBC_t u_t^T
 *   softmax      dg_{t,i} = pi_{t,i} ( [i in K_t] dpi_{t,i} - sum_{j in K_t} pi_{t,j} dpi_{t,j} )
 *   logits       dW_r += dg_t u_t^T
 * The active sets K_t are constants of the differentiation (the selection itself has no
 * derivative); the kept weights are the softmax values over all E, not renormalised, and are
 * differentiated as such.  forced_idx (may be NULL) replaces the router's selection; the
 * weights are always the softmax values of the selected experts.
 *   Outputs: dW_r[E,F] (may be NULL when W_r is NULL and E == 1), dW_e[E,S,F]; optional
 *   dBC[T,S], dpi[T,k].
 * ------------------------------------------------------------------------- */
int oracle_swimba_backward_weights(const double *u, const double *x, const double *dt,
                                   const double *h0, const double *W_r, const double *W_e,
                                   const double *A, const double *dt_bias, const double *dy,
                                   int B, int L, int F, int H, int P, int N, int G, int E, int k,
                                   const int *forced_idx, double *dW_r, double *dW_e,
                                   double *dBC_out, double *dpi_out)
{
    if (!u || !x || !W_e || !W_r || !A || !dt_bias || !dy || !dW_e || !dW_r || B < 0 || L < 0 ||
        F <= 0 || E <= 0 || k <= 0 || k > E || N <= 0 || G <= 0 || H % G != 0)
        return ORACLE_BAD_ARG;
    const long T = (long)B * L;
    const int S = 2 * G * N, hpg = H / G;
    const long PN = (long)P * N;
    int *idx = (int *)malloc(sizeof(int) * (size_t)(T * k + 1));
    double *w = (double *)malloc(sizeof(double) * (size_t)(T * k + 1));
    double *pi = (double *)malloc(sizeof(double) * (size_t)(T * E + 1));
    double *BC = (double *)malloc(sizeof(double) * (size_t)(T * S + 1));
    double *dBC = (double *)calloc((size_t)(T * S + 1), sizeof(double));
    double *dg = (double *)calloc((size_t)(T * E + 1), sizeof(double));
    int rc = ORACLE_OK;
    if (!idx || !w || !pi || !BC || !dBC || !dg) rc = ORACLE_NO_MEM;
    if (rc == ORACLE_OK) rc = oracle_router(u, W_r, T, F, E, k, idx, w, pi, NULL, NULL);
    if (rc == ORACLE_OK && forced_idx) {
        memcpy(idx, forced_idx, sizeof(int) * (size_t)(T * k));
        for (long r = 0; r < T * k; ++r) w[r] = pi[(r / k) * E + idx[r]];
    }
    if (rc == ORACLE_OK) rc = oracle_mix_topk(u, W_e, T, F, S, E, k, idx, w, BC);
    int fail = 0;
    if (rc == ORACLE_OK) {
        /* the recurrence, one (sequence, head) at a time: forward in time for h_t, then backward
         * in time for lambda_t */
#pragma omp parallel for collapse(2) schedule(dynamic)
        for (int b = 0; b < B; ++b)
            for (int h = 0; h < H; ++h) {
                double *st = (double *)malloc(sizeof(double) * (size_t)PN);
                if (!st) { fail = 1; continue; }
                const int g = h / hpg;
                for (long i = 0; i < PN; ++i) st[i] = h0 ? h0[((long)b * H + h) * PN + i] : 0.0;
                for (int t = 0; t < L; ++t) {
                    const long bt = (long)b * L + t;
                    const double *Bt = BC + bt * S + (long)g * N;
                    const double delta = softplus((dt ? dt[bt * H + h] : 0.0) + dt_bias[h]);
                    const double a = exp(delta * A[h]);
                    for (int n = 0; n < N; ++n) {
                        double acc = 0.0;
                        for (int p = 0; p < P; ++p) {
                            double *sp = st + (long)p * N + n;
                            *sp = a * (*sp) + delta * x[(bt * H + h) * P + p] * Bt[n];
                            acc += dy[(bt * H + h) * P + p] * (*sp);
                        }
#pragma omp atomic
                        dBC[bt * S + (long)(G + g) * N + n] += acc;
                    }
                }
                for (long i = 0; i < PN; ++i) st[i] = 0.0;          /* lambda past the last token */
                double a_next = 0.0;
                for (int t = L - 1; t >= 0; --t) {
                    const long bt = (long)b * L + t;
                    const double *Ct = BC + bt * S + (long)(G + g) * N;
                    const double delta = softplus((dt ? dt[bt * H + h] : 0.0) + dt_bias[h]);
                    for (int n = 0; n < N; ++n) {
                        double acc = 0.0;
                        for (int p = 0; p < P; ++p) {
                            double *sp = st + (long)p * N + n;
                            *sp = a_next * (*sp) + dy[(bt * H + h) * P + p] * Ct[n];
                            acc += x[(bt * H + h) * P + p] * (*sp);
                        }
#pragma omp atomic
                        dBC[bt * S + (long)g * N + n] += delta * acc;
                    }
                    a_next = exp(delta * A[h]);
                }
                free(st);
            }
        if (fail) rc = ORACLE_NO_MEM;
    }
    if (rc == ORACLE_OK) {
        /* mix and softmax, token by token */
#pragma omp parallel for schedule(static)
        for (long t = 0; t < T; ++t) {
            double dpi[64], inner = 0.0;
            for (int j = 0; j < k && j < 64; ++j) {
                const int e = idx[t * k + j];
                double acc = 0.0;
                for (int srow = 0; srow < S; ++srow) {
                    double proj = 0.0;
                    for (int f = 0; f < F; ++f) proj += W_e[((long)e * S + srow) * F + f] * u[t * F + f];
                    acc += dBC[t * S + srow] * proj;
                }
                dpi[j] = acc;
                inner += w[t * k + j] * acc;
                if (dpi_out) dpi_out[t * k + j] = acc;
            }
            for (int i = 0; i < E; ++i) dg[t * E + i] = -pi[t * E + i] * inner;
            for (int j = 0; j < k && j < 64; ++j) dg[t * E + idx[t * k + j]] += w[t * k + j] * dpi[j];
        }
        /* weight gradients, one expert at a time (no two threads touch the same rows) */
#pragma omp parallel for schedule(dynamic)
        for (int e = 0; e < E; ++e) {
            for (long i = 0; i < (long)S * F; ++i) dW_e[(long)e * S * F + i] = 0.0;
            for (int f = 0; f < F; ++f) dW_r[(long)e * F + f] = 0.0;
            for (long t = 0; t < T; ++t) {
                for (int f = 0; f < F; ++f) dW_r[(long)e * F + f] += dg[t * E + e] * u[t * F + f];
                for (int j = 0; j < k; ++j) {
                    if (idx[t * k + j] != e) continue;
                    for (int srow = 0; srow < S; ++srow) {
                        const double c = w[t * k + j] * dBC[t * S + srow];
                        for (int f = 0; f < F; ++f) dW_e[((long)e * S + srow) * F + f] += c * u[t * F + f];
                    }
                }
            }
        }
        if (dBC_out) memcpy(dBC_out, dBC, sizeof(double) * (size_t)(T * S));
    }
    free(idx); free(w); free(pi); free(BC); free(dBC); free(dg);
    return rc;
}

/* ---------------------------------------------------------------------------
 * One autoregressive step: the layer above with one token per sequence and the
 * carried state updated in place (state[B,H,P,N]).
 * ------------------------------------------------------------------------- */
int oracle_swimba_decode_step(const double *u, const double *x, const double *dt,
                              const double *W_r, const double *W_e, const double *A,
                              const double *dt_bias, const double *D,
                              int B, int F, int H, int P, int N, int G, int E, int k,
                              const int *forced_idx, const double *forced_w,
                              double *state, double *y, int *idx_out, double *w_out)
{
    if (!state) return ORACLE_BAD_ARG;
    const size_t n = (size_t)B * H * P * N;
    double *next = (double *)malloc(sizeof(double) * (n + 1));
    if (!next) return ORACLE_NO_MEM;
    int rc = oracle_swimba_forward(u, x, dt, state, W_r, W_e, A, dt_bias, D, B, 1, F, H, P, N, G,
                                   E, k, forced_idx, forced_w, y, next, idx_out, w_out, NULL);
    if (rc == ORACLE_OK) memcpy(state, next, sizeof(double) * n);
    free(next);
    return rc;
}

/* ===========================================================================
 * The rest of the block around the mixer (Section "Swimba layer": the in-projection becomes a
 * mixture of experts and "the rest of the Mamba-2 layer is kept unchanged"; the paper does not
 * restate that rest, so these three functions write out the public Mamba-2 block conventions:
 * causal depthwise convolution + SiLU on the [x | B | C] stream, the gated RMS norm
 * norm(y * silu(z)) * weight, and plain linear maps).
 * ======================================================================== */
static double silu(double v) { return v / (1.0 + exp(-v)); }

/* Causal depthwise convolution of width K followed by SiLU, channel by channel:
 *   out[b,t,c] = silu( bias[c] + sum_{i<K} w[c,i] * in[b, t-(K-1)+i, c] ),
 * i.e. w[c,K-1] multiplies the current token.  Positions before the call are taken from
 * state_in[b,i,c] (the K-1 tokens preceding the call, oldest first; zeros when NULL); the last
 * K-1 inputs of the call (or of state + call when L < K-1) are returned in state_out. */
int oracle_conv_silu(const double *in, const double *w, const double *bias, const double *state_in,
                     int B, int L, int C, int K, double *out, double *state_out)
{
    if (!in || !w || !out || B <= 0 || L < 0 || C <= 0 || K <= 0) return ORACLE_BAD_ARG;
    for (int b = 0; b < B; ++b)
        for (int t = 0; t < L; ++t)
            for (int c = 0; c < C; ++c) {
                double acc = bias ? bias[c] : 0.0;
                for (int i = 0; i < K; ++i) {
                    const int tt = t - (K - 1) + i;
                    double v;
                    if (tt >= 0) v = in[((long)b * L + tt) * C + c];
                    else v = state_in ? state_in[((long)b * (K - 1) + (K - 1 + tt)) * C + c] : 0.0;
                    acc += w[(long)c * K + i] * v;
                }
                out[((long)b * L + t) * C + c] = silu(acc);
            }
    if (state_out)
        for (int b = 0; b < B; ++b)
            for (int i = 0; i < K - 1; ++i)
                for (int c = 0; c < C; ++c) {
                    const int tt = L - (K - 1) + i;      /* position of the i-th kept token */
                    double v;
                    if (tt >= 0) v = in[((long)b * L + tt) * C + c];
                    else v = state_in ? state_in[((long)b * (K - 1) + (K - 1 + tt)) * C + c] : 0.0;
                    state_out[((long)b * (K - 1) + i) * C + c] = v;
                }
    return ORACLE_OK;
}

/* Gated RMS norm over groups of D/ngroups channels:
 *   v = y * silu(z),  out = v / sqrt(mean_group(v^2) + eps) * weight. */
int oracle_gated_rmsnorm(const double *y, const double *z, const double *weight, long T, int D,
                         int ngroups, double eps, double *out)
{
    if (!y || !z || !weight || !out || D <= 0 || ngroups <= 0 || D % ngroups != 0) return ORACLE_BAD_ARG;
    const int gs = D / ngroups;
    for (long t = 0; t < T; ++t)
        for (int g = 0; g < ngroups; ++g) {
            double ss = 0.0;
            for (int c = g * gs; c < (g + 1) * gs; ++c) {
                const double v = y[t * D + c] * silu(z[t * D + c]);
                ss += v * v;
            }
            const double r = 1.0 / sqrt(ss / gs + eps);
            for (int c = g * gs; c < (g + 1) * gs; ++c)
                out[t * D + c] = y[t * D + c] * silu(z[t * D + c]) * r * weight[c];
        }
    return ORACLE_OK;
}

/* out[T,O] = x[T,F] W[O,F]^T */
int oracle_linear(const double *x, const double *W, long T, int F, int O, double *out)
{
    if (!x || !W || !out || F <= 0 || O <= 0) return ORACLE_BAD_ARG;
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t)
        for (int o = 0; o < O; ++o) {
            double acc = 0.0;
            for (int f = 0; f < F; ++f) acc += W[(long)o * F + f] * x[t * F + f];
            out[t * O + o] = acc;
        }
    return ORACLE_OK;
}

int oracle_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}
