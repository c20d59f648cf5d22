"""GPU parity of the sequence-sharded forward.  The ranks of a job are emulated one after the
other on one device (no kernel of one rank waits for another: the summaries are complete before any
rank's second half starts); the all-gather is a stack of the ranks' summaries.  The concatenated
outputs are compared with the oracle run on the whole sequences, the state after every rank's shard
with the oracle run on the prefix."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2603_06938_b200 import binding as sb
from paper_2603_06938_b200 import synth

import helpers as hp

pytestmark = pytest.mark.gpu


def cfg_of(**kw):
    base = dict(name="sharded", dtype="bf16", B=2, L=512, F=64, H=4, P=64, N=128, G=1, E=4, k=2, Q=128)
    base.update(kw)
    return synth.LayerConfig(**base)


def sharded_forward(cfg, inp, shard_lens, h0=None):
    """Splits every sequence into len(shard_lens) runs of tokens; returns host y [B,L,H,P], the state
    after every rank's shard, idx, w."""
    R, B = len(shard_lens), cfg.B
    cu = np.concatenate([[0], np.cumsum(shard_lens)])
    assert cu[-1] == cfg.L
    h = hp.create_handle(cfg)
    try:
        w, keep = hp.device_weights(inp)
        h0d = hp.dev(h0)
        ranks = []
        for r in range(R):
            a, e = int(cu[r]), int(cu[r + 1])
            L = e - a
            u, x, dt = hp.dev(inp["u"][:, a:e]), hp.dev(inp["x"][:, a:e]), hp.dev(inp["dt"][:, a:e])
            ws, ws_raw = hp.with_canary((sb.swimba_shard_workspace_bytes(h, B, L),), torch.uint8, 0)
            st, st_raw = hp.with_canary((B, cfg.H, cfg.P, cfg.N), torch.float32, float("nan"))
            dc, dc_raw = hp.with_canary((B, cfg.H), torch.float32, float("nan"))
            idx = torch.full((B, L, cfg.k), -1, dtype=torch.int32, device="cuda")
            wt = torch.full((B, L, cfg.k), float("nan"), device="cuda")
            sb.swimba_shard_summary(h, w, u, x, dt, B, L, st, dc, idx, wt, ws)
            ranks.append(dict(u=u, x=x, dt=dt, ws=ws, raws=[ws_raw, st_raw, dc_raw], st=st, dc=dc, idx=idx, wt=wt, L=L))
        assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
        all_state = torch.stack([r_["st"] for r_ in ranks]).contiguous()      # the all-gather
        all_decay = torch.stack([r_["dc"] for r_ in ranks]).contiguous()
        ys, ends = [], []
        for r, r_ in enumerate(ranks):
            y, y_raw = hp.with_canary(tuple(r_["x"].shape), r_["x"].dtype, float("nan"))
            he, he_raw = hp.with_canary((B, cfg.H, cfg.P, cfg.N), torch.float32, float("nan"))
            sb.swimba_shard_finish(h, w, r_["x"], h0d, all_state, all_decay, r, R, B, r_["L"], y, he, r_["ws"])
            assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
            for raw in r_["raws"] + [y_raw, he_raw]:
                assert hp.canary_intact(raw), "a kernel wrote past the end of a buffer"
            ys.append(y.cpu())
            ends.append(he.cpu())
        return dict(y=torch.cat(ys, dim=1), ends=ends, idx=torch.cat([r_["idx"].cpu() for r_ in ranks], dim=1),
                    w=torch.cat([r_["wt"].cpu() for r_ in ranks], dim=1),
                    decay=all_decay.cpu())
    finally:
        sb.swimba_destroy(h)


CASES = [
    (cfg_of(), [256, 256]),
    (cfg_of(L=640), [128, 384, 128]),
    (cfg_of(L=505, B=1, H=3), [300, 128, 77]),                 # ragged shards of different lengths
    (cfg_of(L=4, B=3), [1, 1, 1, 1]),                          # one token per rank
    (cfg_of(L=6144, B=1, H=2), [2048, 2048, 2048]),            # every shard is cut into local segments
    (cfg_of(L=700, H=6, G=2, E=8, k=3, F=136), [350, 350]),
]


@pytest.mark.parametrize("case", range(len(CASES)))
@pytest.mark.parametrize("skip", ["D", "noD"])
def test_sharded_forward_matches_oracle(case, skip):
    cfg, shard_lens = CASES[case]
    inp = synth.make_inputs(cfg, seed=61 + case)
    if skip == "noD":
        inp["D"] = None
    gen = torch.Generator().manual_seed(13)
    h0 = (0.1 * torch.randn(cfg.B, cfg.H, cfg.P, cfg.N, generator=gen)).float()
    got = sharded_forward(cfg, inp, shard_lens, h0=h0)
    tol_y, tol_h = hp.tolerances(cfg)
    full = dict(y=got["y"], h_final=got["ends"][-1], idx=got["idx"], w=got["w"])
    res = hp.compare_forward(cfg, inp, full, tol_y, tol_h, h0=h0)
    # the state after every rank's shard: the oracle on the prefix, with the library's routing
    cu = np.cumsum(shard_lens)
    for r in range(len(shard_lens) - 1):
        e = int(cu[r])
        sub = dict(inp)
        sub["u"], sub["x"], sub["dt"] = inp["u"][:, :e], inp["x"][:, :e], inp["dt"][:, :e]
        fi = np.ascontiguousarray(got["idx"][:, :e].numpy())
        pi = oracle.router(synth.f64(sub["u"]).reshape(-1, cfg.F), synth.f64(inp["W_r"]), cfg.k)["pi"]
        fw = np.take_along_axis(pi, fi.reshape(-1, cfg.k).astype(np.int64), -1)
        ref = hp.oracle_forward(dataclasses.replace(cfg, L=e), sub, h0=h0, forced_idx=fi, forced_w=fw)
        assert hp.per_head_rel(got["ends"][r].double().numpy(), ref["h_final"], 1) <= tol_h


def test_sharded_equals_the_plain_forward_for_one_rank():
    cfg = cfg_of(L=384, B=3)
    inp = synth.make_inputs(cfg, seed=71)
    dense = hp.gpu_forward(cfg, inp)
    got = sharded_forward(cfg, inp, [cfg.L])
    tol_y, tol_h = hp.tolerances(cfg)
    # same routing; y and the final state agree to rounding (the segmentation may differ)
    assert torch.equal(got["idx"], dense["idx"])
    assert hp.per_head_rel(got["y"].double().numpy(), dense["y"].double().numpy(), 2) <= 2 * hp.BF16_EPS
    assert hp.per_head_rel(got["ends"][0].double().numpy(), dense["h_final"].double().numpy(), 1) <= 1e-5


def test_shard_entry_points_reject_what_they_do_not_take():
    cfg = synth.LayerConfig("fp32", "fp32", 1, 64, 32, 2, 16, 16, 1, 2, 1, 64)
    h = hp.create_handle(cfg)
    try:
        assert sb.swimba_shard_workspace_bytes(h, 1, 64) == 0
        inp = synth.make_inputs(cfg, seed=1)
        w, keep = hp.device_weights(inp)
        u, x, dt = hp.dev(inp["u"]), hp.dev(inp["x"]), hp.dev(inp["dt"])
        st = torch.zeros(1, 2, 16, 16, device="cuda")
        dc = torch.zeros(1, 2, device="cuda")
        ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
        rc = sb.swimba_shard_summary(h, w, u, x, dt, 1, 64, st, dc, None, None, ws, check=False)
        assert rc == sb.ERR_UNSUPPORTED_SHAPE
    finally:
        sb.swimba_destroy(h)
    cfg = cfg_of(L=128, B=1)
    h = hp.create_handle(cfg)
    try:
        inp = synth.make_inputs(cfg, seed=2)
        w, keep = hp.device_weights(inp)
        x = hp.dev(inp["x"])
        y = torch.zeros_like(x)
        ws = torch.zeros(sb.swimba_shard_workspace_bytes(h, 1, 128), dtype=torch.uint8, device="cuda")
        for rank, world in ((2, 2), (-1, 2), (0, 0)):
            rc = sb.swimba_shard_finish(h, w, x, None, None, None, rank, world, 1, 128, y, None, ws, check=False)
            assert rc == sb.ERR_UNSUPPORTED_SHAPE
        rc = sb.swimba_shard_finish(h, w, x, None, None, None, 1, 2, 1, 128, y, None, ws, check=False)
        assert rc == sb.ERR_NULL_ARG
        assert float(y.abs().max()) == 0.0
    finally:
        sb.swimba_destroy(h)
