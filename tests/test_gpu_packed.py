"""GPU parity of the packed (variable-length) forward: sequences of different lengths back to back
in one [T, ...] batch, every sequence against the oracle run on its own slice (its own recurrence,
its own initial state), plus the properties that hold at any size: no row of one sequence depends
on another sequence's tokens, and the packed call equals the dense call when all lengths agree.
Tolerances as in test_gpu_parity (routing bit-exact on certified tokens, bf16 2e-2 / 1e-2 per
(sequence, head), fp32 1e-4)."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2603_06938_b200 import binding as sb
from paper_2603_06938_b200 import synth

import helpers as hp

pytestmark = pytest.mark.gpu


def cfg_of(dtype="bf16", **kw):
    base = dict(name="packed", dtype=dtype, B=1, L=1, F=64, H=4, P=64, N=128, G=1, E=4, k=2, Q=128)
    base.update(kw)
    return synth.LayerConfig(**base)


def packed_forward(cfg, inp, lens, h0=None, flags=0):
    """inp: a B = 1 batch of T = sum(lens) tokens.  Returns host y [T,H,P], h_final [nseq,H,P,N], idx,
    w, segments."""
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    T, nseq = int(cu[-1]), len(lens)
    h = hp.create_handle(cfg, None, flags)
    try:
        w, keep = hp.device_weights(inp)
        u, x, dt = hp.dev(inp["u"][0]), hp.dev(inp["x"][0]), hp.dev(inp["dt"][0] if inp["dt"] is not None else None)
        h0d = hp.dev(h0)
        y, y_raw = hp.with_canary((max(T, 1), cfg.H, cfg.P), x.dtype, float("nan"))
        hf, hf_raw = hp.with_canary((nseq, cfg.H, cfg.P, cfg.N), torch.float32, float("nan"))
        idx = torch.full((max(T, 1), cfg.k), -1, dtype=torch.int32, device="cuda")
        wt = torch.full((max(T, 1), cfg.k), float("nan"), device="cuda")
        nws = max(sb.swimba_packed_workspace_bytes(h, cu), 16)
        ws, ws_raw = hp.with_canary((nws,), torch.uint8, 0)
        sb.swimba_forward_packed(h, w, u, x, dt, h0d, cu, y, hf, idx, wt, ws)
        rc = sb.swimba_status(h)
        assert rc == 0, sb.swimba_last_error(h)
        assert hp.canary_intact(y_raw) and hp.canary_intact(hf_raw) and hp.canary_intact(ws_raw), \
            "a kernel wrote past the end of y, h_final or the workspace"
        return dict(y=y[:T].cpu(), h_final=hf.cpu(), idx=idx[:T].cpu(), w=wt[:T].cpu(),
                    segments=sb.swimba_packed_segments(h, cu), launches=sb.swimba_last_launch_count(h))
    finally:
        sb.swimba_destroy(h)


def slice_inputs(inp, a, b, h0):
    out = dict(inp)
    out["u"] = inp["u"][:, a:b]
    out["x"] = inp["x"][:, a:b]
    out["dt"] = None if inp["dt"] is None else inp["dt"][:, a:b]
    out["h0"] = h0
    return out


def check_packed(cfg, inp, lens, got, h0=None):
    tol_y, tol_h = hp.tolerances(cfg)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    worst = dict(err_y=0.0, err_h=0.0, ambiguous=0)
    for b, n in enumerate(lens):
        a, e = int(cu[b]), int(cu[b + 1])
        h0b = None if h0 is None else h0[b:b + 1]
        if n == 0:
            ref_h = np.zeros((cfg.H, cfg.P, cfg.N)) if h0b is None else synth.f64(h0b)[0]
            assert np.array_equal(got["h_final"][b].double().numpy(), ref_h), "an empty sequence must pass its state through"
            continue
        sub = slice_inputs(inp, a, e, h0b)
        sub_cfg = dataclasses.replace(cfg, B=1, L=n)
        sub_got = dict(y=got["y"][a:e][None], h_final=got["h_final"][b:b + 1],
                       idx=got["idx"][a:e][None], w=got["w"][a:e][None])
        res = hp.compare_forward(sub_cfg, sub, sub_got, tol_y, tol_h, h0=h0b)
        worst["err_y"] = max(worst["err_y"], res["err_y"])
        worst["err_h"] = max(worst["err_h"], res["err_h"])
        worst["ambiguous"] += res["ambiguous"]
    return worst


LENGTH_MIXES = [
    [300, 77, 128, 1, 513],                 # ragged tails, one tile exactly, a single token
    [1, 1, 1, 1, 1, 1, 1, 1],               # decode-shaped: one token per sequence
    [127, 129, 0, 256, 5],                  # an empty sequence in the middle
    [0, 200],                               # an empty sequence first
    [640],                                  # one sequence: the dense case
]


@pytest.mark.parametrize("lens", LENGTH_MIXES, ids=lambda v: "-".join(map(str, v)))
@pytest.mark.parametrize("skip", ["D", "noD"])
def test_packed_matches_oracle_per_sequence(lens, skip):
    cfg = cfg_of(L=int(sum(lens)))
    inp = synth.make_inputs(cfg, seed=41)
    if skip == "noD":
        inp["D"] = None
    gen = torch.Generator().manual_seed(5)
    h0 = (0.1 * torch.randn(len(lens), cfg.H, cfg.P, cfg.N, generator=gen)).float()
    got = packed_forward(cfg, inp, lens, h0=h0, flags=sb.FLAG_CHECK_INDICES)
    check_packed(cfg, inp, lens, got, h0=h0)
    assert got["launches"] > 0


def test_packed_other_shapes_and_paths():
    # odd head count (a CTA with one head), two groups, k = 3; then the per-timestep fp32 path
    for cfg, lens in [(cfg_of(H=3, E=8, k=3, F=136, L=700), [150, 390, 160]),
                      (cfg_of(H=6, G=2, L=515), [257, 258]),
                      (cfg_of("fp32", H=3, P=64, N=16, F=48, L=250), [100, 0, 149, 1]),
                      (cfg_of(H=4, P=8, N=32, F=32, L=140), [70, 70])]:
        inp = synth.make_inputs(cfg, seed=43)
        got = packed_forward(cfg, inp, lens)
        check_packed(cfg, inp, lens, got)


def test_packed_long_sequence_among_short_ones_is_segmented():
    # one sequence far above the batch's per-SM share of tiles: it is cut into segments (state-only
    # pass, scan, full pass) while the short ones stay whole
    lens = [128 * 40 + 37, 100, 260, 128, 3]
    cfg = cfg_of(H=2, L=int(sum(lens)))
    inp = synth.make_inputs(cfg, seed=47)
    gen = torch.Generator().manual_seed(7)
    h0 = (0.1 * torch.randn(len(lens), cfg.H, cfg.P, cfg.N, generator=gen)).float()
    got = packed_forward(cfg, inp, lens, h0=h0)
    assert got["segments"] > len(lens), "the long sequence was expected to be cut"
    check_packed(cfg, inp, lens, got, h0=h0)


def test_packed_equals_dense_when_lengths_agree_and_sequences_do_not_mix():
    cfg = cfg_of(B=3, L=384, H=4)
    inp = synth.make_inputs(cfg, seed=53)
    dense = hp.gpu_forward(cfg, inp)
    flat = dict(inp)
    T = cfg.B * cfg.L
    flat["u"] = inp["u"].reshape(1, T, cfg.F)
    flat["x"] = inp["x"].reshape(1, T, cfg.H, cfg.P)
    flat["dt"] = inp["dt"].reshape(1, T, cfg.H)
    pcfg = dataclasses.replace(cfg, B=1, L=T)
    got = packed_forward(pcfg, flat, [cfg.L] * cfg.B)
    # tiles coincide (384 = 3 * 128), so the two calls run the same arithmetic
    assert torch.equal(got["y"].view(cfg.B, cfg.L, cfg.H, cfg.P), dense["y"])
    assert torch.equal(got["h_final"], dense["h_final"])
    assert torch.equal(got["idx"].view(cfg.B, cfg.L, cfg.k), dense["idx"])
    # changing one sequence's tokens leaves the other sequences' rows bit-identical, ragged tails included
    lens = [200, 333, 619]
    cu = np.concatenate([[0], np.cumsum(lens)])
    base = packed_forward(pcfg, flat, lens)
    changed = dict(flat)
    changed["x"] = flat["x"].clone()
    changed["u"] = flat["u"].clone()
    changed["x"][0, cu[1]:cu[2]] = 3.0
    changed["u"][0, cu[1]:cu[2]] = -flat["u"][0, cu[1]:cu[2]]
    other = packed_forward(pcfg, changed, lens)
    for b in (0, 2):
        assert torch.equal(other["y"][cu[b]:cu[b + 1]], base["y"][cu[b]:cu[b + 1]])
        assert torch.equal(other["h_final"][b], base["h_final"][b])
    assert not torch.equal(other["y"][cu[1]:cu[2]], base["y"][cu[1]:cu[2]])


def test_packed_rejects_bad_offsets():
    cfg = cfg_of(L=256)
    inp = synth.make_inputs(cfg, seed=3)
    h = hp.create_handle(cfg)
    try:
        w, keep = hp.device_weights(inp)
        u, x, dt = hp.dev(inp["u"][0]), hp.dev(inp["x"][0]), hp.dev(inp["dt"][0])
        y = torch.zeros_like(x)
        ws = torch.zeros(1 << 22, dtype=torch.uint8, device="cuda")
        for cu in ([1, 256], [0, 200, 100]):
            rc = sb.swimba_forward_packed(h, w, u, x, dt, None, cu, y, None, None, None, ws, check=False)
            assert rc == sb.ERR_UNSUPPORTED_SHAPE
            assert sb.swimba_packed_workspace_bytes(h, cu) == 0
        small = torch.zeros(64, dtype=torch.uint8, device="cuda")
        rc = sb.swimba_forward_packed(h, w, u, x, dt, None, [0, 256], y, None, None, None, small, check=False)
        assert rc == sb.ERR_WORKSPACE_TOO_SMALL
        assert float(y.abs().max()) == 0.0
    finally:
        sb.swimba_destroy(h)


def test_packed_without_step_sizes_initial_states_or_final_states():
    # dt == NULL (the literal time-invariant transition), h0 == NULL, h_final == NULL, two B/C groups
    lens = [140, 2, 391]
    cfg = cfg_of(H=4, G=2, L=int(sum(lens)))
    inp = synth.make_inputs(cfg, seed=59, with_dt=False)
    cu = np.concatenate([[0], np.cumsum(lens)])
    h = hp.create_handle(cfg)
    try:
        w, keep = hp.device_weights(inp)
        u, x = hp.dev(inp["u"][0]), hp.dev(inp["x"][0])
        y = torch.full_like(x, float("nan"))
        idx = torch.full((cfg.L, cfg.k), -1, dtype=torch.int32, device="cuda")
        wt = torch.full((cfg.L, cfg.k), float("nan"), device="cuda")
        ws = torch.zeros(sb.swimba_packed_workspace_bytes(h, cu), dtype=torch.uint8, device="cuda")
        sb.swimba_forward_packed(h, w, u, x, None, None, cu, y, None, idx, wt, ws)
        assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
        hf = torch.full((len(lens), cfg.H, cfg.P, cfg.N), float("nan"), device="cuda")
        y2 = torch.full_like(x, float("nan"))
        sb.swimba_forward_packed(h, w, u, x, None, None, cu, y2, hf, idx, wt, ws)
        assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
        assert torch.equal(y, y2)
    finally:
        sb.swimba_destroy(h)
    got = dict(y=y.cpu(), h_final=hf.cpu(), idx=idx.cpu(), w=wt.cpu())
    check_packed(cfg, inp, lens, got)
