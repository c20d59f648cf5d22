"""GPU parity of the whole block around the mixer (shared in-projection, routed B / C projection,
causal convolution + SiLU, the single recurrence, gated RMS norm, out-projection) against the
oracle's step-by-step composition.  Routing is checked under the margin protocol of helpers.py and
the oracle then runs with the library's routing, so that every token's floats are compared.
Tolerances: the final state as everywhere (1e-2 bf16 / 1e-4 fp32, inside every (sequence, head));
the block output passes through six more bf16-stored intermediates than y does, so it is held to
3e-2 of its largest magnitude (2e-4 on the fp32 path).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_06938_b200 import binding as sb
from paper_2603_06938_b200 import synth

import helpers as hp

pytestmark = pytest.mark.gpu


def make_block(cfg, seed, d_conv=4, bias=True):
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    dt_ = synth.torch_dtype(cfg.dtype)
    D = cfg.H * cfg.P
    W_in = (torch.randn(2 * D + cfg.H, cfg.F, generator=gen) * (1.0 / cfg.F ** 0.5)).to(dt_)
    # the step-size rows are small, as a trained dt projection's are
    W_in[2 * D:] = (W_in[2 * D:].float() * 0.3).to(dt_)
    conv_w = (torch.randn(D + cfg.S, d_conv, generator=gen) * 0.5).float()
    conv_b = (torch.randn(D + cfg.S, generator=gen) * 0.1).float() if bias else None
    norm_w = (1.0 + 0.1 * torch.randn(D, generator=gen)).float()
    W_out = (torch.randn(cfg.F, D, generator=gen) * (1.0 / D ** 0.5)).to(dt_)
    return dict(W_in=W_in, conv_w=conv_w, conv_b=conv_b, norm_w=norm_w, W_out=W_out, d_conv=d_conv)


def gpu_block(cfg, inp, blk, u, conv_state=None, h0=None):
    B, L = u.shape[:2]
    h = hp.create_handle(cfg)
    w, keep = hp.device_weights(inp)
    dblk = {n: hp.dev(v) if torch.is_tensor(v) else v for n, v in blk.items()}
    bw = sb.make_block_weights(dblk["W_in"], dblk["conv_w"], dblk["conv_b"], dblk["norm_w"], dblk["W_out"], blk["d_conv"])
    ud = hp.dev(u)
    out, out_raw = hp.with_canary((B, L, cfg.F), ud.dtype, float("nan"))
    C = cfg.H * cfg.P + cfg.S
    cst, cst_raw = hp.with_canary((B, blk["d_conv"] - 1, C), ud.dtype, float("nan"))
    hf, hf_raw = hp.with_canary((B, cfg.H, cfg.P, cfg.N), torch.float32, float("nan"))
    idx = torch.full((B, L, cfg.k), -1, dtype=torch.int32, device="cuda")
    wt = torch.full((B, L, cfg.k), float("nan"), device="cuda")
    ws, ws_raw = hp.with_canary((sb.swimba_block_workspace_bytes(h, B, L),), torch.uint8, 0)
    sb.swimba_block_forward(h, w, bw, ud, hp.dev(conv_state), hp.dev(h0), B, L, out, cst, hf, idx, wt, ws)
    assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
    assert all(hp.canary_intact(r) for r in (out_raw, cst_raw, hf_raw, ws_raw))
    sb.swimba_destroy(h)
    return dict(out=out.cpu(), conv_state=cst.cpu(), h_final=hf.cpu(), idx=idx.cpu(), w=wt.cpu())


def oracle_block(cfg, inp, blk, u, idx, conv_state=None, h0=None):
    B, L = u.shape[:2]
    r = oracle.router(synth.f64(u).reshape(B * L, cfg.F), synth.f64(inp["W_r"]), cfg.k)
    fi = idx.numpy().reshape(B * L, cfg.k)
    fw = np.take_along_axis(r["pi"], fi.astype(np.int64), -1)
    return oracle.block_forward(synth.f64(u), synth.f64(blk["W_in"]), synth.f64(inp["W_r"]), synth.f64(inp["W_e"]),
                                synth.f64(blk["conv_w"]), synth.f64(blk["conv_b"]), synth.f64(inp["A"]),
                                synth.f64(inp["dt_bias"]), synth.f64(inp["D"]), synth.f64(blk["norm_w"]),
                                synth.f64(blk["W_out"]), H=cfg.H, k=cfg.k, G=cfg.G, conv_state=synth.f64(conv_state),
                                h0=synth.f64(h0), forced_idx=fi, forced_w=fw)


def tolerances(cfg):
    return (3e-2, 1e-2) if cfg.dtype == "bf16" else (2e-4, 1e-4)


CASES = [
    dict(dtype="bf16"),                                             # tensor-core linear maps and SSD tiles
    dict(dtype="bf16", L=700, B=1, H=2, G=1, E=8, k=1, d_conv=2, bias=False),
    dict(dtype="bf16", L=200, H=4, G=2, F=128),                      # two B / C groups: two norm groups
    dict(dtype="fp32", L=150, N=32, P=16, H=2, F=48, E=3),
]


@pytest.mark.parametrize("i", range(len(CASES)))
def test_block_forward_matches_the_oracle_composition(i):
    kw = dict(CASES[i])
    d_conv, bias = kw.pop("d_conv", 4), kw.pop("bias", True)
    base = dict(name="block", dtype="bf16", B=2, L=300, F=64, H=4, P=64, N=128, G=1, E=4, k=2, Q=128)
    base.update(kw)
    cfg = synth.LayerConfig(**base)
    inp = synth.make_inputs(cfg, seed=90 + i)
    blk = make_block(cfg, 190 + i, d_conv, bias)
    got = gpu_block(cfg, inp, blk, inp["u"])
    hp.check_routing(cfg, inp, got["idx"], got["w"])
    ref = oracle_block(cfg, inp, blk, inp["u"], got["idx"])
    ty, th = tolerances(cfg)
    assert hp.max_rel(got["out"].double().numpy(), ref["out"]) <= ty
    assert hp.per_head_rel(got["h_final"].double().numpy(), ref["h_final"], 1) <= th
    tol_c = 2.0 ** -7 if cfg.dtype == "bf16" else 1e-5
    assert hp.max_rel(got["conv_state"].double().numpy(), ref["conv_state"]) <= tol_c


def test_block_carries_convolution_window_and_state_across_calls():
    cfg = synth.LayerConfig("block", "bf16", 2, 400, 64, 4, 64, 128, 1, 4, 2, 128)
    inp = synth.make_inputs(cfg, seed=95)
    blk = make_block(cfg, 195)
    whole = gpu_block(cfg, inp, blk, inp["u"])
    cut = 130
    g1 = gpu_block(cfg, inp, blk, inp["u"][:, :cut].contiguous())
    g2 = gpu_block(cfg, inp, blk, inp["u"][:, cut:].contiguous(), conv_state=g1["conv_state"], h0=g1["h_final"])
    out12 = torch.cat([g1["out"], g2["out"]], 1)
    assert hp.max_rel(out12.double().numpy(), whole["out"].double().numpy()) <= 3e-2
    assert hp.per_head_rel(g2["h_final"].numpy(), whole["h_final"].numpy(), 1) <= 1e-2
    assert torch.equal(g2["conv_state"].view(torch.int16), whole["conv_state"].view(torch.int16))
    ref = oracle_block(cfg, inp, blk, inp["u"], torch.cat([g1["idx"], g2["idx"]], 1))
    assert hp.max_rel(out12.double().numpy(), ref["out"]) <= 3e-2
