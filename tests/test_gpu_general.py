"""GPU parity of the general form of the layer, with expert-specific SSM inputs X^(e) (the state
equation of the paper's Section "MoE-parameterized SSM" as printed): the library's two calls
(router + projection without the mix, then the single recurrence on per-slot streams) against the
oracle's direct statement of that equation, and against the MoE over separated SSMs in the regime
where Theorem 4 says the two designs coincide.  Tolerances as elsewhere: routing bit-exact on
certified tokens; 1e-4 (fp32) or 2e-2 on y / 1e-2 on the final state (bf16), inside every
(sequence, head).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_06938_b200 import binding as sb
from paper_2603_06938_b200 import synth

import helpers as hp

pytestmark = pytest.mark.gpu


def cfg_of(dtype="bf16", **kw):
    base = dict(name="general", dtype=dtype, B=2, L=300, F=64, H=4, P=64, N=128, G=1, E=4, k=2, Q=128)
    base.update(kw)
    return synth.LayerConfig(**base)


def run_general(cfg, inp, xe, h0=None):
    """xe [B,L,E,H,P] (config dtype, host).  Returns y, h_final, idx, w (host tensors)."""
    B, L, T = cfg.B, cfg.L, cfg.B * cfg.L
    h = hp.create_handle(cfg)
    w, keep = hp.device_weights(inp)
    u, dt = hp.dev(inp["u"]), hp.dev(inp["dt"])
    ws = torch.empty(sb.swimba_workspace_bytes(h, B, L), dtype=torch.uint8, device="cuda")
    BCs, bc_raw = hp.with_canary((T, cfg.k, cfg.S), u.dtype, float("nan"))
    idx = torch.full((B, L, cfg.k), -1, dtype=torch.int32, device="cuda")
    wt = torch.full((B, L, cfg.k), float("nan"), device="cuda")
    sb.swimba_route_project_slots(h, w, u, T, BCs, idx, wt, ws)
    assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
    assert hp.canary_intact(bc_raw)
    # the caller's experts: slot j of a token gets X^(e) of its j-th active expert
    gather = idx.cpu().long()[..., None, None].expand(B, L, cfg.k, cfg.H, cfg.P)
    x_slots = torch.gather(xe, 2, gather).permute(2, 0, 1, 3, 4).contiguous().cuda()      # [k,B,L,H,P]
    ws2 = torch.empty(sb.swimba_ssd_slots_workspace_bytes(h, B, L), dtype=torch.uint8, device="cuda")
    y, y_raw = hp.with_canary((B, L, cfg.H, cfg.P), u.dtype, float("nan"))
    hf, hf_raw = hp.with_canary((B, cfg.H, cfg.P, cfg.N), torch.float32, float("nan"))
    sb.swimba_ssd_slots(h, w, x_slots, BCs, dt, hp.dev(h0), B, L, y, hf, ws2)
    assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
    assert hp.canary_intact(y_raw) and hp.canary_intact(hf_raw)
    sb.swimba_destroy(h)
    return y.cpu(), hf.cpu(), idx.cpu(), wt.cpu()


def dense_pi(cfg, inp, idx):
    """fp64 mixture weights of the library's routing, dense over E (zero outside the active set)."""
    T = cfg.B * cfg.L
    r = oracle.router(synth.f64(inp["u"]).reshape(T, cfg.F), synth.f64(inp["W_r"]), cfg.k)
    ii = idx.numpy().reshape(T, cfg.k).astype(np.int64)
    pi = np.zeros((T, cfg.E))
    np.put_along_axis(pi, ii, np.take_along_axis(r["pi"], ii, -1), -1)
    return pi.reshape(cfg.B, cfg.L, cfg.E)


@pytest.mark.parametrize("dtype,k,E,L", [("bf16", 2, 8, 300), ("bf16", 3, 4, 200), ("bf16", 1, 4, 260),
                                        ("fp32", 2, 4, 150)])
def test_general_injection_matches_the_state_equation(dtype, k, E, L):
    cfg = cfg_of(dtype, k=k, E=E, L=L, N=128 if dtype == "bf16" else 32, h0_std=0.3)
    inp = synth.make_inputs(cfg, seed=81)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(82)
    xe = torch.randn(cfg.B, cfg.L, cfg.E, cfg.H, cfg.P, generator=gen).to(synth.torch_dtype(dtype))
    y, hf, idx, wt = run_general(cfg, inp, xe, h0=inp["h0"])
    hp.check_routing(cfg, inp, idx, wt)
    T = cfg.B * cfg.L
    BCe = oracle.expert_streams(synth.f64(inp["u"]).reshape(T, cfg.F), synth.f64(inp["W_e"]))
    y_ref, h_ref = oracle.mixed_general(synth.f64(xe), BCe.reshape(cfg.B, cfg.L, cfg.E, cfg.S), dense_pi(cfg, inp, idx),
                                        synth.f64(inp["dt"]), synth.f64(inp["A"]), synth.f64(inp["dt_bias"]),
                                        h0=synth.f64(inp["h0"]), G=cfg.G)
    hp.check_outputs(cfg, dict(inp, D=None), y, hf, dict(y=y_ref, h_final=h_ref), *hp.tolerances(cfg))


def test_theorem4_equality_regime_on_device():
    # time-invariant routing (W_r = 0: pi = 1/E), dense mixture (k = E), one readout shared by all
    # experts, zero initial states: the mixed model equals the MoE over separated SSMs
    cfg = cfg_of("bf16", k=4, E=4, L=260)
    inp = synth.make_inputs(cfg, seed=83)
    inp["W_r"] = torch.zeros_like(inp["W_r"])
    gn = cfg.G * cfg.N
    inp["W_e"][:, gn:, :] = inp["W_e"][0:1, gn:, :]
    gen = torch.Generator(device="cpu")
    gen.manual_seed(84)
    xe = torch.randn(cfg.B, cfg.L, cfg.E, cfg.H, cfg.P, generator=gen).to(torch.bfloat16)
    y, hf, idx, wt = run_general(cfg, inp, xe)
    assert torch.equal(idx, torch.arange(cfg.E, dtype=torch.int32).expand(cfg.B, cfg.L, cfg.E))   # ties: lower index first
    np.testing.assert_allclose(wt.numpy(), 1.0 / cfg.E, rtol=1e-6)
    T = cfg.B * cfg.L
    BCe = oracle.expert_streams(synth.f64(inp["u"]).reshape(T, cfg.F), synth.f64(inp["W_e"]))
    pi = np.full((cfg.B, cfg.L, cfg.E), 1.0 / cfg.E)
    y_sep, _ = oracle.separated(synth.f64(xe), BCe.reshape(cfg.B, cfg.L, cfg.E, cfg.S), pi, synth.f64(inp["dt"]),
                                synth.f64(inp["A"]), synth.f64(inp["dt_bias"]), G=cfg.G)
    assert hp.per_head_rel(y.double().numpy(), y_sep, 2) <= 2e-2
