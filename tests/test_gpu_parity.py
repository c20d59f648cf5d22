"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element,
on the same seeded inputs.  Tolerances: routing indices bit-exact (see helpers.check_routing for
near-ties); fp32 path 1e-4 max relative error; bf16 inputs with fp32 accumulation 2e-2 on y and
1e-2 on the final state.  The error is max|got-ref| / max|ref| taken inside every (sequence, head)
(helpers.check_outputs): heads differ by orders of magnitude in step size and decay.  Every shape
runs twice, with the skip term D x and without it; without it y is the readout Ctilde^T h alone.
"""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2603_06938_b200 import binding as sb
from paper_2603_06938_b200 import synth

import helpers as hp

pytestmark = pytest.mark.gpu


def cfg_of(dtype="bf16", **kw):
    base = dict(name="case", dtype=dtype, B=2, L=300, F=64, H=4, P=64, N=128, G=1, E=4, k=2, Q=128)
    base.update(kw)
    return synth.LayerConfig(**base)


# ------------------------------------------------------------------ config 0, whole tensor
def test_tiny_fp32_config_full_parity():
    cfg = synth.CONFIGS["tiny_fp32"]
    inp = synth.make_inputs(cfg, seed=0)
    got = hp.gpu_forward(cfg, inp)
    res = hp.compare_forward(cfg, inp, got, 1e-4, 1e-4, require_all_certified=True)
    assert got["launches"] > 0
    assert res["ambiguous"] == 0


# ------------------------------------------------------------ small, odd and ragged shapes
CASES = [
    cfg_of("bf16"),                                        # several tiles + ragged tail
    cfg_of("bf16", L=77, B=3),                             # shorter than one tile
    cfg_of("bf16", L=128, B=1),                            # exactly one tile
    cfg_of("bf16", L=1, B=2),                              # single token
    cfg_of("bf16", L=513, k=4, E=4),                       # dense routing (k == E)
    cfg_of("bf16", L=260, k=1, E=8),                       # switch routing
    cfg_of("bf16", L=260, k=1, E=1),                       # plain Mamba-2 (router skipped)
    cfg_of("bf16", L=200, H=4, G=2),                       # two B/C groups
    cfg_of("bf16", L=300, H=3, P=32, N=64, F=40),          # other head/state sizes
    cfg_of("bf16", L=700, H=2, E=16, k=3, F=136),
    cfg_of("fp32", L=150, N=16, P=64, H=3, F=48),
    cfg_of("fp32", L=97, N=32, P=16, H=2, G=2, E=3, k=2, F=24),
    cfg_of("fp32", L=64, N=128, P=64, H=2, E=5, k=5, F=72),
    cfg_of("fp32", L=100, N=16, P=16, H=2, F=32),          # a block of 16 threads per (sequence, head)
    cfg_of("bf16", L=70, N=32, P=8, H=4, F=32),            # the same through the bf16 per-timestep path
    cfg_of("bf16", L=130, B=1, H=2, F=2048, E=8, k=2),     # router matrix of 32 KB in shared memory
    cfg_of("bf16", L=150, B=1, H=2, F=1024, E=64, k=8),    # router matrix too large to stage
    cfg_of("bf16", L=2100, B=1, H=2, F=256, E=16, k=2),    # several router chunks per block
    cfg_of("bf16", L=390, B=2, H=3),                       # odd head count: one CTA with a single head
    cfg_of("bf16", L=257, B=1, H=6, G=2),                  # three heads per group: a pair and a single
    cfg_of("bf16", L=129, B=1, H=2),                       # one token past a tile boundary
    cfg_of("bf16", L=5000, B=1, H=2, h0_std=0.3),          # segmented sequence with an initial state
    # enough 64-token tiles for the streaming router (three per SM): ragged last tile and feature
    # block, 2 / 4 / 8 expert column tiles
    cfg_of("bf16", L=14420, B=2, H=2, F=200, E=16, k=2),
    cfg_of("bf16", L=28810, B=1, H=2, F=72, E=32, k=3),
    cfg_of("bf16", L=28900, B=1, H=2, F=128, E=64, k=8),
    # between half an SM count and one SM count of (sequence, head pair) CTAs: every pair is worked by
    # two CTAs (leading tiles / whole sequence with a state-only lead); even and odd head counts
    cfg_of("bf16", L=700, B=40, H=4, h0_std=0.3),
    cfg_of("bf16", L=650, B=45, H=3),
    cfg_of("bf16", L=520, B=40, H=4, G=2),                 # the same with two B/C groups
]


@pytest.mark.parametrize("skip_term", [True, False], ids=["D", "noD"])
@pytest.mark.parametrize("i", range(len(CASES)))
def test_small_shapes_full_parity(i, skip_term):
    cfg = CASES[i]
    inp = synth.make_inputs(cfg, seed=100 + i)
    if not skip_term:
        inp["D"] = None
    got = hp.gpu_forward(cfg, inp)
    hp.compare_forward(cfg, inp, got, *hp.tolerances(cfg))


def test_alias_mode_features_are_the_ssm_input():
    # the paper writes one symbol X_t for what the router / experts read and what the SSM is fed:
    # u and x are the same buffer, d_model = H * P
    cfg = cfg_of("bf16", L=333, B=2, H=4, P=64, F=256, E=4, k=2)
    inp = synth.make_inputs(cfg, seed=61)
    inp["D"] = None
    inp["u"] = inp["x"].reshape(cfg.B, cfg.L, cfg.F).clone()
    h = hp.create_handle(cfg)
    w, keep = hp.device_weights(inp)
    x = hp.dev(inp["x"])
    dt = hp.dev(inp["dt"])
    y = torch.full_like(x, float("nan"))
    hf = torch.full((cfg.B, cfg.H, cfg.P, cfg.N), float("nan"), device="cuda")
    idx = torch.full((cfg.B, cfg.L, cfg.k), -1, dtype=torch.int32, device="cuda")
    wt = torch.full((cfg.B, cfg.L, cfg.k), float("nan"), device="cuda")
    ws = torch.empty(sb.swimba_workspace_bytes(h, cfg.B, cfg.L), dtype=torch.uint8, device="cuda")
    sb.swimba_forward(h, w, x, x, dt, None, cfg.B, cfg.L, y, hf, idx, wt, ws)     # u is x
    assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
    sb.swimba_destroy(h)
    got = dict(y=y.cpu(), h_final=hf.cpu(), idx=idx.cpu(), w=wt.cpu())
    hp.compare_forward(cfg, inp, got, *hp.tolerances(cfg))


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_optional_arguments_and_initial_state(dtype):
    cfg = cfg_of(dtype, L=210, h0_std=0.5, N=64 if dtype == "fp32" else 128)
    inp = synth.make_inputs(cfg, seed=7, with_dt=False)     # dt == NULL: time-invariant transition
    inp["D"] = None                                         # no skip term
    got = hp.gpu_forward(cfg, inp, want_topk=False)
    ref = hp.oracle_forward(cfg, inp)
    hp.check_outputs(cfg, inp, got["y"], got["h_final"], ref, *hp.tolerances(cfg))


def test_empty_inputs_are_a_no_op():
    cfg = cfg_of("bf16")
    h = hp.create_handle(cfg)
    inp = synth.make_inputs(dataclasses.replace(cfg, L=4), seed=1)
    w, keep = hp.device_weights(inp)
    assert sb.swimba_workspace_bytes(h, 0, 10) == 0
    assert sb.swimba_forward(h, w, None, None, None, None, 0, 5, None, None, None, None, None) == 0
    assert sb.swimba_forward(h, w, None, None, None, None, 3, 0, None, None, None, None, None) == 0
    assert sb.swimba_status(h) == 0
    sb.swimba_destroy(h)


# ------------------------------------------------------------------------------ properties
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_result_does_not_depend_on_chunk_length(dtype):
    cfg = cfg_of(dtype, L=600, N=64 if dtype == "fp32" else 128)
    inp = synth.make_inputs(cfg, seed=11)
    inp["D"] = None
    ref = hp.oracle_forward(cfg, inp)
    for Q in (64, 128, 256):
        got = hp.gpu_forward(cfg, inp, chunk=Q)
        hp.check_outputs(cfg, inp, got["y"], got["h_final"], ref, *hp.tolerances(cfg))


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_two_calls_with_carried_state_equal_one_call(dtype):
    cfg = cfg_of(dtype, L=500, B=2, N=64 if dtype == "fp32" else 128)
    inp = synth.make_inputs(cfg, seed=12)
    inp["D"] = None
    whole = hp.gpu_forward(cfg, inp)
    cut = 207
    first = {k: (v[:, :cut] if k in ("u", "x", "dt") else v) for k, v in inp.items()}
    second = {k: (v[:, cut:] if k in ("u", "x", "dt") else v) for k, v in inp.items()}
    g1 = hp.gpu_forward(dataclasses.replace(cfg, L=cut), {k: (v.contiguous() if torch.is_tensor(v) else v) for k, v in first.items()})
    g2 = hp.gpu_forward(dataclasses.replace(cfg, L=cfg.L - cut), {k: (v.contiguous() if torch.is_tensor(v) else v) for k, v in second.items()}, h0=g1["h_final"])
    y12 = torch.cat([g1["y"], g2["y"]], 1)
    ty, th = hp.tolerances(cfg)
    assert hp.max_rel(y12.double().numpy(), whole["y"].double().numpy()) <= ty
    assert hp.max_rel(g2["h_final"].numpy(), whole["h_final"].numpy()) <= th
    ref = hp.oracle_forward(cfg, inp)
    hp.check_outputs(cfg, inp, y12, g2["h_final"], ref, ty, th)


def test_forward_is_bitwise_reproducible():
    cfg = cfg_of("bf16", L=400)
    inp = synth.make_inputs(cfg, seed=13)
    a = hp.gpu_forward(cfg, inp)
    b = hp.gpu_forward(cfg, inp)
    assert torch.equal(a["y"].view(torch.int16), b["y"].view(torch.int16))
    assert torch.equal(a["h_final"], b["h_final"])
    assert torch.equal(a["idx"], b["idx"])


@pytest.mark.parametrize("shape", [dict(L=400), dict(L=700, B=40, H=4), dict(L=5000, B=1, H=2)])
def test_calls_queued_back_to_back_do_not_disturb_each_other(shape):
    """Three forwards on one handle, one workspace and one stream with no host synchronisation in
    between (inputs A, B, A): the kernels of a call start under the tail of the kernel before them,
    but never under an earlier call.  Each result must equal that of the same call made alone.
    Shapes: one CTA per head pair, the split launch, the segmented launch."""
    cfg = cfg_of("bf16", **shape)
    ia = synth.make_inputs(cfg, seed=21)
    ib = dict(synth.make_inputs(cfg, seed=22), **{n: ia[n] for n in ("W_r", "W_e", "A", "dt_bias", "D")})
    alone = [hp.gpu_forward(cfg, ia), hp.gpu_forward(cfg, ib)]
    h = hp.create_handle(cfg)
    w, keep = hp.device_weights(ia)
    dev_in = [{n: hp.dev(i[n]) for n in ("u", "x", "dt")} for i in (ia, ib)]
    ws = torch.empty(sb.swimba_workspace_bytes(h, cfg.B, cfg.L), dtype=torch.uint8, device="cuda")
    outs = []
    for which in (0, 1, 0):
        d = dev_in[which]
        y = torch.full_like(d["x"], float("nan"))
        hf = torch.full((cfg.B, cfg.H, cfg.P, cfg.N), float("nan"), device="cuda")
        idx = torch.full((cfg.B, cfg.L, cfg.k), -1, dtype=torch.int32, device="cuda")
        wt = torch.full((cfg.B, cfg.L, cfg.k), float("nan"), device="cuda")
        sb.swimba_forward(h, w, d["u"], d["x"], d["dt"], None, cfg.B, cfg.L, y, hf, idx, wt, ws)
        outs.append((y, hf, idx))
    assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
    sb.swimba_destroy(h)
    for (y, hf, idx), ref in zip(outs, (alone[0], alone[1], alone[0])):
        assert torch.equal(y.cpu().view(torch.int16), ref["y"].view(torch.int16))
        assert torch.equal(hf.cpu(), ref["h_final"])
        assert torch.equal(idx.cpu(), ref["idx"])


def test_theorem3_state_bound_holds_on_device():
    # ||h_T|| <= rho^T ||h_0|| + (1-rho^T)/(1-rho) U, per (head, channel), with the mixed streams
    cfg = cfg_of("fp32", L=256, B=1, N=32, P=16, H=2, h0_std=1.0)
    inp = synth.make_inputs(cfg, seed=14)
    got = hp.gpu_forward(cfg, inp)
    ref = hp.oracle_forward(cfg, inp)
    dlt = np.logaddexp(0.0, synth.f64(inp["dt"]) + synth.f64(inp["dt_bias"]))
    a = np.exp(dlt * synth.f64(inp["A"]))
    Bt = ref["BC"][0, :, :cfg.N]
    x = synth.f64(inp["x"])
    for h in range(cfg.H):
        rho = a[0, :, h].max()
        for p in range(cfg.P):
            U = np.linalg.norm(dlt[0, :, h, None] * x[0, :, h, p, None] * Bt, axis=-1).max()
            bound = rho ** cfg.L * np.linalg.norm(synth.f64(inp["h0"])[0, h, p]) + \
                (1 - rho ** cfg.L) / (1 - rho) * U
            assert np.linalg.norm(got["h_final"][0, h, p].double().numpy()) <= bound * (1 + 1e-4)


# ------------------------------------------------------------------------- split entry points
def test_route_mix_and_ssd_entry_points():
    cfg = cfg_of("bf16", L=300)
    inp = synth.make_inputs(cfg, seed=15)
    B, L = cfg.B, cfg.L
    h = hp.create_handle(cfg)
    w, keep = hp.device_weights(inp)
    u, x, dt = hp.dev(inp["u"]), hp.dev(inp["x"]), hp.dev(inp["dt"])
    ws = torch.empty(sb.swimba_workspace_bytes(h, B, L), dtype=torch.uint8, device="cuda")
    BC = torch.empty(B, L, cfg.S, dtype=torch.bfloat16, device="cuda")
    idx = torch.empty(B, L, cfg.k, dtype=torch.int32, device="cuda")
    wt = torch.empty(B, L, cfg.k, device="cuda")
    sb.swimba_route_mix(h, w, u, B * L, BC, idx, wt, ws)
    assert sb.swimba_status(h) == 0
    hp.check_routing(cfg, inp, idx.cpu(), wt.cpu())
    ref_bc = oracle.mix_topk(synth.f64(inp["u"]).reshape(B * L, -1), synth.f64(inp["W_e"]),
                             idx.cpu().numpy().reshape(B * L, -1), wt.cpu().double().numpy().reshape(B * L, -1))
    assert hp.max_rel(BC.cpu().double().numpy().reshape(B * L, -1), ref_bc) <= 1e-2
    # SSD on the library's own (bf16-rounded) mixed streams against the oracle recurrence on them
    y = torch.empty_like(x)
    hf = torch.empty(B, cfg.H, cfg.P, cfg.N, device="cuda")
    sb.swimba_ssd(h, w, x, BC, dt, None, B, L, y, hf, ws)
    assert sb.swimba_status(h) == 0
    yr, hr = oracle.ssm_recurrence(synth.f64(inp["x"]), BC.cpu().double().numpy(), synth.f64(inp["dt"]),
                                   synth.f64(inp["A"]), synth.f64(inp["dt_bias"]), synth.f64(inp["D"]))
    hp.check_outputs(cfg, inp, y.cpu(), hf.cpu(), dict(y=yr, h_final=hr), 2e-2, 1e-2)
    sb.swimba_destroy(h)


# -------------------------------------------------------------------------------- decode
# F = 128: grouped GEMM (bf16) / SIMT (fp32) front end; F a multiple of 256 with k <= 2 and E <= 16:
# the two-kernel front end for a handful of tokens (ragged token tiles, k = 1, E = 16, several passes)
@pytest.mark.parametrize("dtype,F,k,B,E", [("fp32", 128, 2, 5, 8), ("bf16", 128, 2, 5, 8), ("bf16", 256, 2, 5, 8),
                                           ("bf16", 512, 1, 37, 16), ("bf16", 256, 2, 150, 4)])
def test_decode_steps_match_oracle_and_forward(dtype, F, k, B, E):
    cfg = cfg_of(dtype, B=B, L=40 if B < 100 else 12, H=4, P=64, N=128 if dtype == "bf16" else 32, E=E, k=k, F=F,
                 h0_std=0.1)
    inp = synth.make_inputs(cfg, seed=21)
    B, L = cfg.B, cfg.L
    h = hp.create_handle(cfg)
    w, keep = hp.device_weights(inp)
    state = hp.dev(inp["h0"]).clone()
    ws = torch.empty(sb.swimba_decode_workspace_bytes(h, B), dtype=torch.uint8, device="cuda")
    ys, idxs, wts = [], [], []
    for t in range(L):
        u = hp.dev(inp["u"][:, t])
        x = hp.dev(inp["x"][:, t])
        dt = hp.dev(inp["dt"][:, t])
        y = torch.empty_like(x)
        idx = torch.empty(B, cfg.k, dtype=torch.int32, device="cuda")
        wt = torch.empty(B, cfg.k, device="cuda")
        sb.swimba_decode_step(h, w, u, x, dt, state, B, y, idx, wt, ws)
        ys.append(y.cpu())
        idxs.append(idx.cpu())
        wts.append(wt.cpu())
    assert sb.swimba_status(h) == 0
    y_dec = torch.stack(ys, 1)
    idx_dec = torch.stack(idxs, 1)
    ty, th = hp.tolerances(cfg)
    # (a) against the oracle's decode loop == oracle forward (pinned on the CPU side)
    res = hp.compare_forward(cfg, inp, dict(y=y_dec, h_final=state.cpu(), idx=idx_dec, w=torch.stack(wts, 1)),
                             ty, th)
    # (b) against the library's own forward over the same L tokens (the two paths may use different
    # router kernels: only tokens too close to a tie to be certified may be routed differently)
    fwd = hp.gpu_forward(cfg, inp)
    differ = int((idx_dec != fwd["idx"]).any(-1).sum())
    assert differ <= res["ambiguous"]
    if differ == 0:
        assert hp.max_rel(y_dec.double().numpy(), fwd["y"].double().numpy()) <= ty
        assert hp.max_rel(state.cpu().numpy(), fwd["h_final"].numpy()) <= th
    sb.swimba_destroy(h)


# ------------------------------------------------------------------- device-detected errors
def test_bounded_wait_runs_out_and_the_handle_stays_usable():
    """The failure path of the tensor-core kernels' waits, exercised on a barrier nothing signals:
    the wait gives up after its cycle limit, the status word carries DEVICE_TIMEOUT, later waits of
    the same block return at once, the kernel exits normally, and a forward on the same handle
    afterwards is correct."""
    cfg = cfg_of("bf16", L=300)
    h = hp.create_handle(cfg)
    rc, (first, second, cycles2) = sb.swimba_selftest_wait(h, 2000000)      # about 1 ms
    assert rc == 0 and first == 1 and second == 1
    assert cycles2 < 200000, "the second wait must not spin for the limit again"
    assert sb.swimba_status(h) == sb.ERR_DEVICE_TIMEOUT
    assert "device reported error" in sb.swimba_last_error(h)
    assert sb.swimba_status(h) == 0                      # reading the status cleared it
    assert sb.swimba_selftest_wait(h, 10, check=False)[0] == sb.ERR_UNSUPPORTED_SHAPE
    sb.swimba_destroy(h)
    inp = synth.make_inputs(cfg, seed=71)
    got = hp.gpu_forward(cfg, inp)
    hp.compare_forward(cfg, inp, got, *hp.tolerances(cfg))


@pytest.mark.parametrize("dtype,k", [("bf16", 2), ("bf16", 3), ("fp32", 2)])
def test_index_checks_stay_silent_on_valid_calls(dtype, k):
    # SWIMBA_FLAG_CHECK_INDICES: the kernels validate expert indices and per-expert lists before
    # following them; on a healthy call nothing fires and the results are unchanged
    cfg = cfg_of(dtype, L=400, E=8, k=k, N=64 if dtype == "fp32" else 128)
    inp = synth.make_inputs(cfg, seed=72)
    plain = hp.gpu_forward(cfg, inp)
    checked = hp.gpu_forward(cfg, inp, flags=sb.FLAG_CHECK_INDICES)
    assert torch.equal(plain["idx"], checked["idx"])
    assert torch.equal(plain["y"].float(), checked["y"].float())
    assert torch.equal(plain["h_final"], checked["h_final"])
    hp.compare_forward(cfg, inp, checked, *hp.tolerances(cfg))
    with pytest.raises(sb.SwimbaError) as e:
        sb.swimba_create(64, 4, 64, 128, 1, 4, 2, 128, sb.DTYPE_BF16, 2)    # reserved flag bit
    assert e.value.code == sb.ERR_BAD_CONFIG


# ------------------------------------------------------------------- host-detected errors
def test_host_side_errors_leave_outputs_untouched():
    cfg = cfg_of("bf16", L=64)
    inp = synth.make_inputs(cfg, seed=31)
    B, L = cfg.B, cfg.L
    h = hp.create_handle(cfg)
    w, keep = hp.device_weights(inp)
    u, x, dt = hp.dev(inp["u"]), hp.dev(inp["x"]), hp.dev(inp["dt"])
    y = torch.full_like(x, 7.0)
    ws = torch.empty(sb.swimba_workspace_bytes(h, B, L) + 64, dtype=torch.uint8, device="cuda")

    def call(**kw):
        a = dict(u=u, x=x, dt=dt, y=y, ws=ws, B=B, L=L)
        a.update(kw)
        return sb.swimba_forward(h, w, a["u"], a["x"], a["dt"], None, a["B"], a["L"], a["y"], None,
                                 None, None, a["ws"], check=False)

    assert call(u=None) == sb.ERR_NULL_ARG
    assert call(y=None) == sb.ERR_NULL_ARG
    assert call(ws=ws[:128]) == sb.ERR_WORKSPACE_TOO_SMALL
    assert call(ws=ws[8:]) == sb.ERR_MISALIGNED
    assert call(B=-1) == sb.ERR_UNSUPPORTED_SHAPE
    assert "workspace" in sb.swimba_last_error(h) or sb.swimba_last_error(h) != ""
    torch.cuda.synchronize()
    assert torch.all(y == 7.0)
    assert call() == 0 and sb.swimba_status(h) == 0
    assert not torch.any(y == 7.0)
    sb.swimba_destroy(h)
    for bad in (dict(top_k=5), dict(chunk=100), dict(n_groups=3), dict(dtype=3), dict(n_experts=0),
                dict(n_experts=65, top_k=1)):
        args = dict(d_model=64, n_heads=4, head_dim=64, d_state=128, n_groups=1, n_experts=4,
                    top_k=2, chunk=128, dtype=1)
        args.update(bad)
        with pytest.raises(sb.SwimbaError) as e:
            sb.swimba_create(**args)
        assert e.value.code == sb.ERR_BAD_CONFIG
    with pytest.raises(sb.SwimbaError) as e:
        sb.swimba_create(d_model=60, n_heads=4, head_dim=64, d_state=128, n_groups=1, n_experts=4,
                         top_k=2, chunk=128, dtype=1)
    assert e.value.code == sb.ERR_UNSUPPORTED_SHAPE


def test_host_buffer_entry_point_matches_device_entry_point():
    cfg = cfg_of("bf16", L=300)
    inp = synth.make_inputs(cfg, seed=41)
    B, L = cfg.B, cfg.L
    dev_out = hp.gpu_forward(cfg, inp)
    h = hp.create_handle(cfg)
    w, keep = hp.device_weights(inp)
    ws = torch.empty(sb.swimba_host_workspace_bytes(h, B, L), dtype=torch.uint8, device="cuda")
    u, x, dt = inp["u"].pin_memory(), inp["x"].pin_memory(), inp["dt"].pin_memory()
    y = torch.empty_like(x).pin_memory()
    hf = torch.empty(B, cfg.H, cfg.P, cfg.N).pin_memory()
    idx = torch.empty(B, L, cfg.k, dtype=torch.int32).pin_memory()
    sb.swimba_forward_host(h, w, u, x, dt, B, L, y, hf, idx, None, ws)
    assert sb.swimba_status(h) == 0
    # the host path runs the batch in slices; a slice may be cut into other SSD segments than the
    # whole batch, so the floats agree within the parity tolerance, the routing exactly
    assert hp.max_rel(y.double().numpy(), dev_out["y"].double().numpy()) <= 2e-2
    assert hp.max_rel(hf.numpy(), dev_out["h_final"].numpy()) <= 1e-2
    assert torch.equal(idx, dev_out["idx"])
    ref = hp.oracle_forward(cfg, inp)
    hp.check_outputs(cfg, inp, y, hf, ref, 2e-2, 1e-2)
    sb.swimba_destroy(h)


def test_decode_steps_replay_from_a_cuda_graph():
    """The decode step enqueues kernels and nothing else (no allocation, no synchronisation), so a
    run of steps can be captured once and replayed: the replay must reproduce the eager steps bit
    for bit (same kernels, same order)."""
    cfg = cfg_of("bf16", B=16, L=1, F=256, H=4, E=8, k=2)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(6)
    wts = {n: v.cuda() for n, v in synth.make_weights(cfg, gen).items()}
    w = sb.make_weights(wts["W_r"], wts["W_e"], wts["A"], wts["dt_bias"], wts["D"])
    toks = [{n: v.cuda() for n, v in synth.make_decode_step_inputs(cfg, gen).items()} for _ in range(4)]
    state0 = (0.1 * torch.randn(cfg.B, cfg.H, cfg.P, cfg.N, generator=gen)).cuda()
    state = state0.clone()
    y = torch.empty(4, *toks[0]["x"].shape, dtype=toks[0]["x"].dtype, device="cuda")
    h = hp.create_handle(cfg)
    try:
        ws = torch.empty(sb.swimba_decode_workspace_bytes(h, cfg.B), dtype=torch.uint8, device="cuda")

        def run(stream=None):
            for i, t in enumerate(toks):
                sb.swimba_decode_step(h, w, t["u"], t["x"], t["dt"], state, cfg.B, y[i], None, None, ws, stream=stream)

        run()                                      # eager (also warms the handle's caches)
        torch.cuda.synchronize()
        y_eager, s_eager = y.clone(), state.clone()
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                run(side)
        torch.cuda.synchronize()
        state.copy_(state0)
        y.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
        assert torch.equal(y, y_eager) and torch.equal(state, s_eager)
    finally:
        sb.swimba_destroy(h)
