"""Pins for the CPU oracle: every check compares it with something the paper or
the mathematics fixes independently of the oracle's own code (closed forms, the
SSD matrix form, library routines on special cases, the theorems' identities,
the worked example of Theorem 5).  CPU only.
"""
import math
import os

import numpy as np
import pytest
import scipy.special

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
rng = np.random.default_rng


def np_softplus(v):
    return np.logaddexp(0.0, v)


def ssd_matrix_form(x, BC, dt, A, dt_bias, D, h0, G=1):
    """Background section, SSD: with a scalar-identity transition the sequence map is
    Y = M X with M[t,s] = (C_t . B_s) * prod_{r=s+1..t} a_r for s <= t (semiseparable,
    masked by the decay), plus the carried-in state and the skip term.  O(L^2)."""
    Bsz, L, H, P = x.shape
    N = BC.shape[-1] // (2 * G)
    y = np.zeros_like(x)
    for b in range(Bsz):
        for h in range(H):
            g = h // (H // G)
            Bm = BC[b, :, g * N:(g + 1) * N]
            Cm = BC[b, :, (G + g) * N:(G + g + 1) * N]
            delta = np_softplus((dt[b, :, h] if dt is not None else 0.0) + dt_bias[h]) * np.ones(L)
            loga = delta * A[h]
            cum = np.cumsum(loga)                       # log prod_{r<=t} a_r
            M = (Cm @ Bm.T) * np.tril(np.exp(cum[:, None] - cum[None, :]))
            y[b, :, h, :] = M @ (delta[:, None] * x[b, :, h, :])
            if h0 is not None:
                y[b, :, h, :] += np.exp(cum)[:, None] * (Cm @ h0[b, h].T)
            if D is not None:
                y[b, :, h, :] += D[h] * x[b, :, h, :]
    return y


def rand_layer(seed, B=2, L=9, F=6, H=4, P=3, N=5, G=1, E=3):
    r = rng(seed)
    S = 2 * G * N
    return dict(
        u=r.normal(size=(B, L, F)), x=r.normal(size=(B, L, H, P)),
        dt=0.5 * r.normal(size=(B, L, H)),
        W_r=r.normal(size=(E, F)), W_e=r.normal(size=(E, S, F)) * 0.3,
        A=-np.exp(r.uniform(0, math.log(16), size=H)),
        dt_bias=r.normal(size=H) - 2.0, D=1 + 0.1 * r.normal(size=H),
        h0=r.normal(size=(B, H, P, N)),
    )


# ------------------------------------------------------------------ recurrence
@pytest.mark.parametrize("G", [1, 2])
@pytest.mark.parametrize("use_dt,use_h0,use_D", [(True, True, True), (False, False, False),
                                                 (True, False, True)])
def test_recurrence_equals_ssd_matrix_form(G, use_dt, use_h0, use_D):
    d = rand_layer(1, B=2, L=17, H=4, P=3, N=5, G=G)
    r = rng(2)
    BC = r.normal(size=(2, 17, 2 * G * 5))
    dt = d["dt"] if use_dt else None
    h0 = d["h0"] if use_h0 else None
    D = d["D"] if use_D else None
    y, hf = oracle.ssm_recurrence(d["x"], BC, dt, d["A"], d["dt_bias"], D, h0, G=G)
    y_ref = ssd_matrix_form(d["x"], BC, dt, d["A"], d["dt_bias"], D, h0, G=G)
    np.testing.assert_allclose(y, y_ref, rtol=1e-10, atol=1e-11)


def test_recurrence_closed_form_constant_streams():
    # x = 1, Btilde = b, Ctilde = c, Delta constant:  h_t = Delta b (1-a^t)/(1-a),
    # y_t = (c.b) Delta (1-a^t)/(1-a) + D  (the geometric series of the stability proof).
    L, H, P, N = 40, 2, 2, 3
    b = np.array([0.5, -1.0, 2.0])
    c = np.array([1.5, 0.25, -0.75])
    A = np.array([-1.0, -3.0])
    dt_bias = np.array([0.3, -1.2])
    D = np.array([0.7, -0.2])
    x = np.ones((1, L, H, P))
    BC = np.tile(np.concatenate([b, c]), (1, L, 1))
    y, hf = oracle.ssm_recurrence(x, BC, None, A, dt_bias, D)
    for h in range(H):
        delta = math.log1p(math.exp(dt_bias[h]))
        a = math.exp(delta * A[h])
        t = np.arange(1, L + 1)
        geo = (1 - a ** t) / (1 - a)
        np.testing.assert_allclose(y[0, :, h, 0], (c @ b) * delta * geo + D[h], rtol=1e-12)
        np.testing.assert_allclose(hf[0, h, 1], delta * b * geo[-1], rtol=1e-12)


def test_state_carry_split_equals_one_call():
    d = rand_layer(3, L=12)
    BC = rng(4).normal(size=(2, 12, 10))
    y, hf = oracle.ssm_recurrence(d["x"], BC, d["dt"], d["A"], d["dt_bias"], d["D"], d["h0"])
    y1, h1 = oracle.ssm_recurrence(d["x"][:, :5], BC[:, :5], d["dt"][:, :5], d["A"], d["dt_bias"],
                                   d["D"], d["h0"])
    y2, h2 = oracle.ssm_recurrence(d["x"][:, 5:], BC[:, 5:], d["dt"][:, 5:], d["A"], d["dt_bias"],
                                   d["D"], h1)
    np.testing.assert_allclose(np.concatenate([y1, y2], 1), y, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(h2, hf, rtol=1e-13, atol=1e-13)


def test_trajectory_last_equals_final_and_group_mapping():
    d = rand_layer(5, H=4, G=1)
    BC = rng(6).normal(size=(2, 9, 2 * 2 * 5))
    y, hf, traj = oracle.ssm_recurrence(d["x"], BC, d["dt"], d["A"], d["dt_bias"], None, None, G=2,
                                        want_traj=True)
    np.testing.assert_array_equal(traj[:, -1], hf)
    # heads 0,1 read group 0 and heads 2,3 group 1: a G=1 call on each half must agree
    for g, heads in enumerate([[0, 1], [2, 3]]):
        BCg = np.concatenate([BC[..., g * 5:(g + 1) * 5], BC[..., (2 + g) * 5:(3 + g) * 5]], -1)
        yg, _ = oracle.ssm_recurrence(d["x"][:, :, heads], BCg, d["dt"][:, :, heads],
                                      d["A"][heads], d["dt_bias"][heads], None, None, G=1)
        np.testing.assert_allclose(y[:, :, heads], yg, rtol=1e-13, atol=1e-13)


# ---------------------------------------------------------------------- router
def test_router_is_softmax_and_topk_keeps_values_without_renorm():
    r = rng(7)
    u = r.normal(size=(50, 8))
    W_r = r.normal(size=(6, 8))
    out = oracle.router(u, W_r, 2)
    logits = u @ W_r.T
    pi = scipy.special.softmax(logits, axis=-1)
    np.testing.assert_allclose(out["pi"], pi, rtol=1e-12)
    np.testing.assert_allclose(out["pi"].sum(-1), 1.0, rtol=1e-12)
    order = np.argsort(-logits, axis=-1, kind="stable")[:, :2]
    np.testing.assert_array_equal(out["idx"], order)
    np.testing.assert_allclose(out["w"], np.take_along_axis(pi, order, -1), rtol=1e-12)
    assert np.all(out["w"].sum(-1) < 1.0)             # mass of the dropped experts is lost
    srt = -np.sort(-logits, axis=-1)
    gaps = np.minimum(srt[:, 0] - srt[:, 1], srt[:, 1] - srt[:, 2])
    np.testing.assert_allclose(out["margin"], gaps, rtol=1e-9, atol=1e-12)
    absdot = np.max(np.abs(u[:, None, :] * W_r[None]).sum(-1), axis=-1)
    np.testing.assert_allclose(out["absdot"], absdot, rtol=1e-12)


def test_router_tie_break_prefers_lower_index_and_dense_k():
    u = rng(8).normal(size=(5, 4))
    row = rng(9).normal(size=4)
    W_r = np.stack([row * 0.5, row, row, row * 0.1])     # experts 1 and 2 tie exactly
    out = oracle.router(u, W_r, 2)
    logit = u @ row
    for t in range(5):
        if logit[t] > 0:
            assert list(out["idx"][t]) == [1, 2]
            assert out["margin"][t] == 0.0
    dense = oracle.router(u, W_r, 4)
    np.testing.assert_allclose(dense["w"].sum(-1), 1.0, rtol=1e-12)
    assert sorted(dense["idx"][0]) == [0, 1, 2, 3]


# ------------------------------------------------------------------------ mix
def test_mix_topk_matches_library_matmul():
    r = rng(10)
    T, F, S, E, k = 20, 7, 6, 4, 2
    u = r.normal(size=(T, F))
    W_e = r.normal(size=(E, S, F))
    idx = np.stack([r.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    w = r.uniform(size=(T, k))
    BC = oracle.mix_topk(u, W_e, idx, w)
    streams = np.einsum("esf,tf->tes", W_e, u)
    ref = sum(w[:, j, None] * streams[np.arange(T), idx[:, j]] for j in range(k))
    np.testing.assert_allclose(BC, ref, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(oracle.expert_streams(u, W_e), streams, rtol=1e-12, atol=1e-13)
    pi = np.zeros((T, E))
    for j in range(k):
        pi[np.arange(T), idx[:, j]] = w[:, j]
    np.testing.assert_allclose(oracle.mix_dense(u, W_e, pi), ref, rtol=1e-12, atol=1e-13)


# --------------------------------------------------------------- whole layer
def test_single_expert_is_plain_mamba2_ssm():
    d = rand_layer(11, E=1)
    out = oracle.swimba_forward(d["u"], d["x"], d["dt"], d["W_r"], d["W_e"], d["A"], d["dt_bias"],
                                d["D"], k=1, h0=d["h0"])
    np.testing.assert_array_equal(out["w"], 1.0)          # softmax over one expert
    BC = d["u"] @ d["W_e"][0].T                           # B = W_B u, C = W_C u
    np.testing.assert_allclose(out["BC"], BC, rtol=1e-12, atol=1e-13)
    y_ref = ssd_matrix_form(d["x"], BC, d["dt"], d["A"], d["dt_bias"], d["D"], d["h0"])
    np.testing.assert_allclose(out["y"], y_ref, rtol=1e-10, atol=1e-11)


@pytest.mark.parametrize("k", [1, 2, 3])
def test_identical_experts_scale_streams_by_retained_mass(k):
    d = rand_layer(12, E=3)
    W_e = np.repeat(d["W_e"][:1], 3, axis=0)
    out = oracle.swimba_forward(d["u"], d["x"], d["dt"], d["W_r"], W_e, d["A"], d["dt_bias"],
                                d["D"], k=k)
    pi = scipy.special.softmax(d["u"] @ d["W_r"].T, axis=-1)
    s_t = -np.sort(-pi, axis=-1)[..., :k].sum(-1)         # mass kept by top-k, <= 1
    BC = (d["u"] @ W_e[0].T) * s_t[..., None]
    if k == 3:
        np.testing.assert_allclose(s_t, 1.0, rtol=1e-12)
    y_ref = ssd_matrix_form(d["x"], BC, d["dt"], d["A"], d["dt_bias"], d["D"], None)
    np.testing.assert_allclose(out["y"], y_ref, rtol=1e-10, atol=1e-11)


def test_readout_only_mixing_is_linear_in_router_weights():
    # all experts share the injection map; dense weights: y - D x is linear in pi
    d = rand_layer(13, E=3)
    N = 5
    W_e = d["W_e"].copy()
    W_e[:, :N] = W_e[0, :N]
    r = rng(14)
    T = 2 * 9
    u2 = d["u"].reshape(T, -1)
    pi1, pi2 = r.uniform(size=(T, 3)), r.uniform(size=(T, 3))
    al, be = 0.7, -1.3

    def run(pi):
        # the injection must not depend on pi for linearity: give B the weights of a
        # fixed reference mixture and only C the tested one
        BC_ref = oracle.mix_dense(u2, W_e, np.full((T, 3), 1.0 / 3))
        BC = oracle.mix_dense(u2, W_e, pi)
        BC[:, :N] = BC_ref[:, :N]
        y, _ = oracle.ssm_recurrence(d["x"], BC.reshape(2, 9, -1), d["dt"], d["A"], d["dt_bias"],
                                     None, None)
        return y

    np.testing.assert_allclose(run(al * pi1 + be * pi2), al * run(pi1) + be * run(pi2),
                               rtol=1e-10, atol=1e-11)


def test_forced_routing_reproduces_free_routing():
    d = rand_layer(15)
    free = oracle.swimba_forward(d["u"], d["x"], d["dt"], d["W_r"], d["W_e"], d["A"], d["dt_bias"],
                                 d["D"], k=2, h0=d["h0"])
    forced = oracle.swimba_forward(d["u"], d["x"], d["dt"], None, d["W_e"], d["A"], d["dt_bias"],
                                   d["D"], k=2, h0=d["h0"], forced_idx=free["idx"],
                                   forced_w=free["w"])
    np.testing.assert_array_equal(free["y"], forced["y"])
    r = oracle.router(d["u"].reshape(18, -1), d["W_r"], 2)
    np.testing.assert_array_equal(free["idx"].reshape(18, 2), r["idx"])
    BC = oracle.mix_topk(d["u"].reshape(18, -1), d["W_e"], r["idx"], r["w"])
    y_ref = ssd_matrix_form(d["x"], BC.reshape(2, 9, -1), d["dt"], d["A"], d["dt_bias"], d["D"],
                            d["h0"])
    np.testing.assert_allclose(free["y"], y_ref, rtol=1e-10, atol=1e-11)


def test_decode_steps_equal_forward():
    d = rand_layer(16, L=11)
    full = oracle.swimba_forward(d["u"], d["x"], d["dt"], d["W_r"], d["W_e"], d["A"], d["dt_bias"],
                                 d["D"], k=2, h0=d["h0"])
    state = d["h0"].copy()
    for t in range(11):
        o = oracle.swimba_decode_step(d["u"][:, t], d["x"][:, t], d["dt"][:, t], d["W_r"],
                                      d["W_e"], d["A"], d["dt_bias"], d["D"], 2, state)
        np.testing.assert_allclose(o["y"], full["y"][:, t], rtol=1e-12, atol=1e-13)
        np.testing.assert_array_equal(o["idx"], full["idx"][:, t])
    np.testing.assert_allclose(state, full["h_final"], rtol=1e-12, atol=1e-13)


# ------------------------------------------------------- theorems 3, 4 and 5
def _general_case(seed, B=1, L=10, E=3, H=2, P=2, N=3, F=4, shared_C=False, uniform_pi=False):
    r = rng(seed)
    S = 2 * N
    u = r.normal(size=(B * L, F))
    W_e = r.normal(size=(E, S, F)) * 0.5
    if shared_C:
        W_e[:, N:] = W_e[0, N:]
    BCe = oracle.expert_streams(u, W_e).reshape(B, L, E, S)
    xe = r.normal(size=(B, L, E, H, P))
    if uniform_pi:
        pi = oracle.router(u, np.zeros((E, F)), E)["pi"].reshape(B, L, E)
    else:
        ro = oracle.router(u, r.normal(size=(E, F)), 2)
        pi = np.zeros((B * L, E))
        np.put_along_axis(pi, ro["idx"], ro["w"], axis=-1)
        pi = pi.reshape(B, L, E)
    dt = 0.5 * r.normal(size=(B, L, H))
    A = -np.exp(r.uniform(0, 2, size=H))
    dt_bias = r.normal(size=H) - 1
    return dict(xe=xe, BCe=BCe, pi=pi, dt=dt, A=A, dt_bias=dt_bias, N=N)


def test_theorem4_equality_regime():
    # time-invariant weights (zero router => uniform), shared readout, zero initial states
    c = _general_case(20, shared_C=True, uniform_pi=True)
    np.testing.assert_allclose(c["pi"], 1.0 / 3, rtol=1e-14)
    y_mix, _ = oracle.mixed_general(c["xe"], c["BCe"], c["pi"], c["dt"], c["A"], c["dt_bias"])
    y_sep, _ = oracle.separated(c["xe"], c["BCe"], c["pi"], c["dt"], c["A"], c["dt_bias"])
    np.testing.assert_allclose(y_sep, y_mix, rtol=1e-11, atol=1e-12)
    # and the regime is sharp: a time-varying router breaks the equality
    c2 = _general_case(20, shared_C=True, uniform_pi=False)
    y_mix2, _ = oracle.mixed_general(c2["xe"], c2["BCe"], c2["pi"], c2["dt"], c2["A"], c2["dt_bias"])
    y_sep2, _ = oracle.separated(c2["xe"], c2["BCe"], c2["pi"], c2["dt"], c2["A"], c2["dt_bias"])
    assert np.max(np.abs(y_sep2 - y_mix2)) > 1e-3


def test_theorem4_difference_identity_recursion_and_bound():
    c = _general_case(21)
    N = c["N"]
    y_mix, _, h = oracle.mixed_general(c["xe"], c["BCe"], c["pi"], c["dt"], c["A"], c["dt_bias"],
                                       want_traj=True)
    y_sep, _, he = oracle.separated(c["xe"], c["BCe"], c["pi"], c["dt"], c["A"], c["dt_bias"],
                                    want_traj=True)
    B, L, E, H, P = c["xe"].shape
    Ce = c["BCe"][..., N:]                                  # [B,L,E,N]
    delta_e = he - h[:, :, None]                            # h^(e)_t - h_t   [B,L,E,H,P,N]
    # Y_sep - Y_mix = sum_e pi_e C^(e)T (h^(e) - h)
    rhs = np.einsum("ble,blen,blehpn->blhp", c["pi"], Ce, delta_e)
    np.testing.assert_allclose(y_sep - y_mix, rhs, rtol=1e-10, atol=1e-11)
    # delta_t = a_t delta_{t-1} + (B^(e) X^(e) - Utilde_t), with the Delta-scaled injection
    dlt = np_softplus(c["dt"] + c["dt_bias"])               # [B,L,H]
    a = np.exp(dlt * c["A"])
    inj_e = np.einsum("blh,blen,blehp->blehpn", dlt, c["BCe"][..., :N], c["xe"])
    u_mix = np.einsum("ble,blehpn->blhpn", c["pi"], inj_e)
    prev = np.zeros_like(delta_e[:, 0])
    for t in range(L):
        expect = a[:, t, None, :, None, None] * prev + (inj_e[:, t] - u_mix[:, t, None])
        np.testing.assert_allclose(delta_e[:, t], expect, rtol=1e-10, atol=1e-11)
        prev = delta_e[:, t]
    # ||Y_sep - Y_mix|| <= C sum_e pi_e ||h^(e) - h||   per head and channel
    Cmax = np.max(np.linalg.norm(Ce, axis=-1))
    lhs = np.abs(y_sep - y_mix)
    bound = Cmax * np.einsum("ble,blehp->blhp", c["pi"], np.linalg.norm(delta_e, axis=-1))
    assert np.all(lhs <= bound * (1 + 1e-12) + 1e-14)


def test_theorem3_bibo_bound():
    d = rand_layer(22, B=1, L=60, H=3, P=2, N=4)
    BC = rng(23).normal(size=(1, 60, 8))
    y, hf, traj = oracle.ssm_recurrence(d["x"], BC, d["dt"], d["A"], d["dt_bias"], None, d["h0"],
                                        want_traj=True)
    dlt = np_softplus(d["dt"] + d["dt_bias"])
    a = np.exp(dlt * d["A"])                                # [1,L,H]
    for h in range(3):
        rho = a[0, :, h].max()
        for p in range(2):
            inj = dlt[0, :, h, None] * d["x"][0, :, h, p, None] * BC[0, :, :4]
            U = np.linalg.norm(inj, axis=-1).max()
            Cn = np.linalg.norm(BC[0, :, 4:], axis=-1).max()
            t = np.arange(1, 61)
            bound = rho ** t * np.linalg.norm(d["h0"][0, h, p]) + (1 - rho ** t) / (1 - rho) * U
            hn = np.linalg.norm(traj[0, :, h, p], axis=-1)
            assert np.all(hn <= bound * (1 + 1e-12))
            assert np.all(np.abs(y[0, :, h, p]) <= Cn * bound * (1 + 1e-12))


def test_theorem5_worked_example_is_logistic_sigmoid():
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "thm5_sigmoid.txt"))
            if ln.strip() and not ln.startswith("#")]
    for r_str, expect in rows:
        xin = math.log(float(r_str))
        u = np.array([[[xin, 1.0]]])                        # appended constant feature
        W_r = np.array([[0.0, 0.0], [1.0, 0.0]])            # g = (0, x)
        # N = 1: rows of W_e are [B ; C]; expert 1 injects 0, expert 2 injects 1; C = 1
        W_e = np.array([[[0.0, 0.0], [0.0, 1.0]], [[0.0, 1.0], [0.0, 1.0]]])
        x = np.ones((1, 1, 1, 1))
        dt_bias = np.array([math.log(math.e - 1)])          # softplus -> Delta = 1
        for A in (0.0, -3.0):                               # h0 = 0: A cannot matter
            out = oracle.swimba_forward(u, x, None, W_r, W_e, np.array([A]), dt_bias,
                                        np.array([0.0]), k=2)
            assert abs(out["y"][0, 0, 0, 0] - float(expect)) < 1e-13
            assert abs(out["h_final"][0, 0, 0, 0] - float(expect)) < 1e-13


def test_mixed_general_reduces_to_shared_input_layer():
    # with X^(e) = x for every expert the general injection is Btilde x^T: same as the layer
    d = rand_layer(24)
    B, L, E = 2, 9, 3
    out = oracle.swimba_forward(d["u"], d["x"], d["dt"], d["W_r"], d["W_e"], d["A"], d["dt_bias"],
                                None, k=2, h0=d["h0"])
    pi = np.zeros((B * L, E))
    np.put_along_axis(pi, out["idx"].reshape(B * L, 2), out["w"].reshape(B * L, 2), axis=-1)
    BCe = oracle.expert_streams(d["u"].reshape(B * L, -1), d["W_e"])
    xe = np.repeat(d["x"][:, :, None], E, axis=2)
    y, hf = oracle.mixed_general(xe, BCe, pi, d["dt"], d["A"], d["dt_bias"], h0=d["h0"])
    np.testing.assert_allclose(y, out["y"], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(hf, out["h_final"], rtol=1e-11, atol=1e-12)


def test_bad_arguments_are_rejected():
    with pytest.raises(ValueError):
        oracle.router(np.zeros((2, 3)), np.zeros((2, 3)), 3)        # k > E
    with pytest.raises(ValueError):
        oracle.mix_topk(np.zeros((2, 3)), np.zeros((2, 4, 3)), np.array([[5], [0]]),
                        np.ones((2, 1)))                            # expert index out of range


# ------------------------------------------------------------------ the rest of the block
def test_conv_silu_equals_numpy_convolution_and_carries_its_state():
    rng = np.random.default_rng(5)
    B, L, C, K = 2, 37, 5, 4
    xin = rng.standard_normal((B, L, C))
    w = rng.standard_normal((C, K))
    bias = rng.standard_normal(C)
    out, st = oracle.conv_silu(xin, w, bias)
    for b in range(B):
        for c in range(C):
            # np.convolve flips its second argument: w[c, K-1] multiplies the current token
            full = np.convolve(xin[b, :, c], w[c, ::-1])[:L] + bias[c]
            np.testing.assert_allclose(out[b, :, c], full / (1.0 + np.exp(-full)), rtol=1e-12, atol=1e-12)
    np.testing.assert_array_equal(st, xin[:, L - (K - 1):, :])
    # two calls with the carried state equal one call; a call shorter than the window keeps older tokens
    cut = 11
    o1, s1 = oracle.conv_silu(xin[:, :cut], w, bias)
    o2, s2 = oracle.conv_silu(xin[:, cut:], w, bias, state=s1)
    np.testing.assert_allclose(np.concatenate([o1, o2], 1), out, rtol=1e-12, atol=1e-12)
    np.testing.assert_array_equal(s2, st)
    o3, s3 = oracle.conv_silu(xin[:, :2], w, bias, state=np.ones((B, K - 1, C)))
    np.testing.assert_array_equal(s3[:, 0], np.ones((B, C)))
    np.testing.assert_array_equal(s3[:, 1:], xin[:, :2])


def test_gated_rmsnorm_and_linear_equal_their_numpy_definitions():
    rng = np.random.default_rng(6)
    T, D, G = 9, 24, 3
    y, z, wt = rng.standard_normal((T, D)), rng.standard_normal((T, D)), rng.standard_normal(D)
    v = (y * z / (1.0 + np.exp(-z))).reshape(T, G, D // G)
    ref = (v / np.sqrt((v * v).mean(-1, keepdims=True) + 1e-5)).reshape(T, D) * wt
    np.testing.assert_allclose(oracle.gated_rmsnorm(y, z, wt, ngroups=G), ref, rtol=1e-12, atol=1e-12)
    # unit weight, one group, no gate effect (z large: silu(z) ~ z): output has unit mean square
    out = oracle.gated_rmsnorm(y, np.full((T, D), 50.0), np.ones(D), ngroups=1, eps=0.0)
    np.testing.assert_allclose((out * out).mean(-1), 1.0, rtol=1e-9)
    W = rng.standard_normal((7, D))
    np.testing.assert_allclose(oracle.linear(y, W), y @ W.T, rtol=1e-12, atol=1e-12)


def test_block_forward_is_the_composition_of_its_steps_and_reduces_to_a_plain_block():
    rng = np.random.default_rng(7)
    B, L, F, H, P, N, G, E, k, K = 2, 19, 12, 2, 4, 8, 1, 3, 2, 4
    Dm, S = H * P, 2 * G * N
    u = rng.standard_normal((B, L, F))
    W_in = rng.standard_normal((2 * Dm + H, F)) * 0.3
    W_r = rng.standard_normal((E, F))
    W_e = rng.standard_normal((E, S, F)) * 0.3
    conv_w, conv_b = rng.standard_normal((Dm + S, K)) * 0.5, rng.standard_normal(Dm + S) * 0.1
    A, dt_bias, D = -np.exp(rng.uniform(0, 2, H)), rng.standard_normal(H), rng.standard_normal(H)
    norm_w, W_out = rng.standard_normal(Dm), rng.standard_normal((F, Dm)) * 0.3
    r = oracle.block_forward(u, W_in, W_r, W_e, conv_w, conv_b, A, dt_bias, D, norm_w, W_out, H=H, k=k, G=G)
    # the mixer inside the block is the layer itself on the convolved streams
    y2, h2 = oracle.ssm_recurrence(r["x"], r["BC"], r["dt"], A, dt_bias, D, G=G)
    np.testing.assert_array_equal(y2, r["y"])
    # identical experts and dense routing: the block is a plain Mamba-2 block whose B / C projection is
    # that one expert matrix, written here with numpy only
    W1 = np.repeat(W_e[:1], E, 0)
    rb = oracle.block_forward(u, W_in, W_r, W1, conv_w, conv_b, A, dt_bias, D, norm_w, W_out, H=H, k=E, G=G)
    T = B * L
    zxdt = u.reshape(T, F) @ W_in.T
    pre = np.concatenate([zxdt[:, Dm:2 * Dm], u.reshape(T, F) @ W_e[0].T], -1).reshape(B, L, Dm + S)
    pad = np.concatenate([np.zeros((B, K - 1, Dm + S)), pre], 1)
    acc = sum(conv_w[:, i] * pad[:, i:i + L] for i in range(K)) + conv_b
    xbc = acc / (1.0 + np.exp(-acc))
    y_ref, _ = oracle.ssm_recurrence(xbc[..., :Dm].reshape(B, L, H, P), xbc[..., Dm:], zxdt[:, 2 * Dm:].reshape(B, L, H),
                                     A, dt_bias, D, G=G)
    z = zxdt[:, :Dm]
    v = y_ref.reshape(T, Dm) * z / (1.0 + np.exp(-z))
    g = v / np.sqrt((v * v).mean(-1, keepdims=True) + 1e-5) * norm_w
    np.testing.assert_allclose(rb["out"], (g @ W_out.T).reshape(B, L, F), rtol=1e-9, atol=1e-11)
    # chunked prefill: two calls carrying the convolution window and the SSM state equal one call
    cut = 7
    r1 = oracle.block_forward(u[:, :cut], W_in, W_r, W_e, conv_w, conv_b, A, dt_bias, D, norm_w, W_out, H=H, k=k, G=G)
    r2 = oracle.block_forward(u[:, cut:], W_in, W_r, W_e, conv_w, conv_b, A, dt_bias, D, norm_w, W_out, H=H, k=k, G=G,
                              conv_state=r1["conv_state"], h0=r1["h_final"])
    np.testing.assert_allclose(np.concatenate([r1["out"], r2["out"]], 1), r["out"], rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(r2["h_final"], r["h_final"], rtol=1e-9, atol=1e-12)


# ----------------------------------------------------------------- gradients of the trained weights
def _loss(lay, dy, k, G, idx, W_r=None, W_e=None, h0=None):
    """sum(dy * y) of the oracle's forward with the active sets held at idx and the weights taken
    from the softmax of the (possibly perturbed) router matrix."""
    W_r = lay["W_r"] if W_r is None else W_r
    W_e = lay["W_e"] if W_e is None else W_e
    T = idx.shape[0] * idx.shape[1]
    pi = oracle.router(lay["u"].reshape(T, -1), W_r, k)["pi"]
    fw = np.take_along_axis(pi, idx.reshape(T, k).astype(np.int64), -1)
    out = oracle.swimba_forward(lay["u"], lay["x"], lay["dt"], W_r, W_e, lay["A"], lay["dt_bias"], lay["D"],
                                k=k, G=G, h0=h0, forced_idx=idx, forced_w=fw)
    return float(np.sum(dy * out["y"]))


@pytest.mark.parametrize("G,k", [(1, 2), (2, 1), (1, 3)])
def test_backward_matches_central_differences_of_the_forward(G, k):
    lay = rand_layer(31 + k, B=2, L=7, F=5, H=4, P=3, N=4, G=G, E=3)
    r = rng(77)
    h0 = 0.3 * r.standard_normal((2, 4, 3, 4))
    dy = r.standard_normal(lay["x"].shape)
    fwd = oracle.swimba_forward(lay["u"], lay["x"], lay["dt"], lay["W_r"], lay["W_e"], lay["A"], lay["dt_bias"],
                                lay["D"], k=k, G=G, h0=h0)
    idx = fwd["idx"]
    got = oracle.backward_weights(lay["u"], lay["x"], lay["dt"], lay["W_r"], lay["W_e"], lay["A"], lay["dt_bias"],
                                  dy, k=k, G=G, h0=h0)
    eps = 1e-6
    for name, grad in (("W_e", got["dW_e"]), ("W_r", got["dW_r"])):
        base = lay[name]
        flat = r.choice(base.size, size=min(base.size, 24), replace=False)
        for pos in flat:
            where = np.unravel_index(pos, base.shape)
            up, dn = base.copy(), base.copy()
            up[where] += eps
            dn[where] -= eps
            fd = (_loss(lay, dy, k, G, idx, h0=h0, **{name: up}) - _loss(lay, dy, k, G, idx, h0=h0, **{name: dn})) / (2 * eps)
            assert abs(fd - grad[where]) <= 1e-6 * max(1.0, abs(fd)), (name, where, fd, grad[where])


def test_backward_single_token_closed_form():
    # L = 1, zero initial state: y[h,p] = Delta_h x[h,p] (Ctilde . Btilde) + D_h x[h,p], so with
    # c = sum_{h,p} dy Delta x:  dBtilde = c Ctilde, dCtilde = c Btilde, dW_e[e] = pi_e [dB; dC] u^T
    lay = rand_layer(41, B=1, L=1, F=4, H=2, P=3, N=5, G=1, E=3)
    k = 2
    dy = rng(5).standard_normal(lay["x"].shape)
    fwd = oracle.swimba_forward(lay["u"], lay["x"], lay["dt"], lay["W_r"], lay["W_e"], lay["A"], lay["dt_bias"],
                                lay["D"], k=k)
    got = oracle.backward_weights(lay["u"], lay["x"], lay["dt"], lay["W_r"], lay["W_e"], lay["A"], lay["dt_bias"],
                                  dy, k=k)
    delta = np_softplus(lay["dt"][0, 0] + lay["dt_bias"])
    c = float(np.sum(dy[0, 0] * delta[:, None] * lay["x"][0, 0]))
    Bt, Ct = fwd["BC"][0, 0, :5], fwd["BC"][0, 0, 5:]
    dBC = np.concatenate([c * Ct, c * Bt])
    np.testing.assert_allclose(got["dBC"][0, 0], dBC, rtol=1e-12, atol=1e-14)
    want = np.zeros_like(lay["W_e"])
    for j in range(k):
        e = fwd["idx"][0, 0, j]
        want[e] += fwd["w"][0, 0, j] * np.outer(dBC, lay["u"][0, 0])
    np.testing.assert_allclose(got["dW_e"], want, rtol=1e-12, atol=1e-14)


def test_backward_invariants():
    lay = rand_layer(43, B=2, L=8, F=6, H=4, P=3, N=4, G=2, E=4)
    r = rng(9)
    dy1, dy2 = r.standard_normal(lay["x"].shape), r.standard_normal(lay["x"].shape)
    args = (lay["u"], lay["x"], lay["dt"], lay["W_r"], lay["W_e"], lay["A"], lay["dt_bias"])
    g1 = oracle.backward_weights(*args, dy1, k=2, G=2)
    g2 = oracle.backward_weights(*args, dy2, k=2, G=2)
    g12 = oracle.backward_weights(*args, 2.0 * dy1 - 3.0 * dy2, k=2, G=2)
    # linear in dy
    np.testing.assert_allclose(g12["dW_e"], 2.0 * g1["dW_e"] - 3.0 * g2["dW_e"], rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(g12["dW_r"], 2.0 * g1["dW_r"] - 3.0 * g2["dW_r"], rtol=1e-10, atol=1e-12)
    # the softmax values sum to one: the logit gradients of a token sum to zero, hence the columns of dW_r
    np.testing.assert_allclose(g1["dW_r"].sum(axis=0), 0.0, atol=1e-12 * np.abs(g1["dW_r"]).max())
    # experts outside every active set receive no gradient; k == E (dense) reaches all of them
    idx = oracle.swimba_forward(*args, lay["D"], k=2, G=2)["idx"]
    unused = [e for e in range(4) if not np.any(idx == e)]
    for e in unused:
        assert not np.any(g1["dW_e"][e])
    # one expert: the softmax is constant, the router receives nothing
    one = rand_layer(44, E=1)
    g = oracle.backward_weights(one["u"], one["x"], one["dt"], one["W_r"], one["W_e"], one["A"], one["dt_bias"],
                                r.standard_normal(one["x"].shape), k=1)
    assert not np.any(g["dW_r"])
    assert np.any(g["dW_e"])
