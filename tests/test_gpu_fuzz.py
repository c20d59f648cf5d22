"""GPU parity on seeded random shapes: every case draws batch, length, widths, heads, groups,
experts, top-k, chunk and which optional arguments are present, runs the forward through the C ABI
and compares it with the oracle under the same protocol and tolerances as test_gpu_parity.  The
draws favour the corners the fixed cases visit one at a time (odd head counts per group, one head,
k == E, lengths around tile and segment boundaries), here in combination."""
import numpy as np
import pytest
import torch

from paper_2603_06938_b200 import synth

import helpers as hp

pytestmark = pytest.mark.gpu


def draw(seed):
    r = np.random.default_rng(1000 + seed)
    kind = r.choice(["tile", "tile", "tile", "bf16_other", "fp32"])
    G = int(r.choice([1, 1, 2, 3]))
    H = G * int(r.integers(1, 5))
    if kind == "tile":
        dtype, P, N = "bf16", 64, 128
    elif kind == "bf16_other":
        dtype, P, N = "bf16", int(r.choice([8, 16, 32, 64])), int(r.choice([16, 32, 64]))
    else:
        dtype, P, N = "fp32", int(r.choice([8, 16, 64])), int(r.choice([16, 32, 128]))
    E = int(r.choice([1, 2, 3, 4, 8, 16]))
    k = int(r.integers(1, min(E, 4) + 1))
    F = 8 * int(r.integers(1, 66))
    B = int(r.integers(1, 6))
    L = int(r.choice([1, int(r.integers(2, 130)), int(r.integers(120, 140)), int(r.integers(250, 700)),
                      int(r.integers(1000, 3000))]))
    if kind != "tile":
        L = min(L, 400)
    Q = int(r.choice([64, 128, 256]))
    cfg = synth.LayerConfig("fuzz", dtype, B, L, F, H, P, N, G, E, k, Q, h0_std=float(r.choice([0.0, 0.1])))
    return cfg, bool(r.integers(0, 2)), bool(r.integers(0, 4) > 0)


@pytest.mark.parametrize("seed", range(32))
def test_random_shapes_match_oracle(seed):
    cfg, use_D, use_dt = draw(seed)
    inp = synth.make_inputs(cfg, seed=seed, with_dt=use_dt)
    if not use_D:
        inp["D"] = None
    got = hp.gpu_forward(cfg, inp)
    res = hp.compare_forward(cfg, inp, got, *hp.tolerances(cfg))
    print(cfg, "D" if use_D else "noD", "dt" if use_dt else "nodt",
          f"err_y={res['err_y']:.2e} err_h={res['err_h']:.2e} ambiguous={res['ambiguous']}")


@pytest.mark.parametrize("seed", range(16))
def test_random_packed_batches_match_oracle(seed):
    import test_gpu_packed as tp
    r = np.random.default_rng(2000 + seed)
    nseq = int(r.integers(1, 9))
    lens = [int(r.choice([0, 1, int(r.integers(2, 6)), int(r.integers(6, 140)), int(r.integers(140, 600)),
                          int(r.integers(600, 2500))])) for _ in range(nseq)]
    if sum(lens) == 0:
        lens[0] = 37
    tile = bool(r.integers(0, 4) > 0)
    G = int(r.choice([1, 2]))
    H = G * int(r.integers(1, 4))
    E = int(r.choice([1, 4, 8]))
    k = int(r.integers(1, min(E, 3) + 1))
    if tile:
        cfg = synth.LayerConfig("fuzz", "bf16", 1, int(sum(lens)), 8 * int(r.integers(4, 40)), H, 64, 128, G, E, k, 128)
    else:
        lens = [min(v, 200) for v in lens]
        cfg = synth.LayerConfig("fuzz", str(r.choice(["bf16", "fp32"])), 1, int(sum(lens)), 8 * int(r.integers(4, 40)), H,
                                int(r.choice([16, 32])), int(r.choice([16, 64])), G, E, k, 128)
    inp = synth.make_inputs(cfg, seed=seed)
    gen = torch.Generator().manual_seed(seed)
    h0 = (0.1 * torch.randn(len(lens), cfg.H, cfg.P, cfg.N, generator=gen)).float() if r.integers(0, 2) else None
    got = tp.packed_forward(cfg, inp, lens, h0=h0)
    worst = tp.check_packed(cfg, inp, lens, got, h0=h0)
    print(cfg.dtype, cfg.P, cfg.N, lens, f"err_y={worst['err_y']:.2e} err_h={worst['err_h']:.2e}")


@pytest.mark.parametrize("seed", range(12))
def test_random_decode_loops_match_oracle(seed):
    """A run of decode steps on a drawn shape (both front ends, tile and other state shapes, with
    and without the skip term) against the oracle's forward over the same tokens."""
    from paper_2603_06938_b200 import binding as sb
    r = np.random.default_rng(3000 + seed)
    dtype = str(r.choice(["bf16", "bf16", "fp32"]))
    G = int(r.choice([1, 2]))
    H = G * int(r.integers(1, 4))
    P, N = (64, 128) if (dtype == "bf16" and r.integers(0, 3) > 0) else (int(r.choice([16, 32, 64])), int(r.choice([16, 32, 64])))
    E = int(r.choice([1, 2, 4, 8, 16]))
    k = int(r.integers(1, min(E, 3) + 1))
    F = int(r.choice([64, 128, 256, 512, 8 * int(r.integers(1, 40))]))
    B = int(r.choice([1, 2, int(r.integers(3, 40)), int(r.integers(100, 300))]))
    L = 6 if B > 64 else int(r.integers(2, 20))
    cfg = synth.LayerConfig("fuzz", dtype, B, L, F, H, P, N, G, E, k, 128, h0_std=0.1)
    inp = synth.make_inputs(cfg, seed=seed)
    if r.integers(0, 2):
        inp["D"] = None
    h = hp.create_handle(cfg)
    try:
        w, keep = hp.device_weights(inp)
        state = hp.dev(inp["h0"]).clone()
        ws = torch.empty(max(sb.swimba_decode_workspace_bytes(h, B), 16), dtype=torch.uint8, device="cuda")
        ys, idxs, wts = [], [], []
        for t in range(L):
            u, x, dt = hp.dev(inp["u"][:, t]), hp.dev(inp["x"][:, t]), hp.dev(inp["dt"][:, t])
            y = torch.empty_like(x)
            idx = torch.empty(B, k, dtype=torch.int32, device="cuda")
            wt = torch.empty(B, k, device="cuda")
            sb.swimba_decode_step(h, w, u, x, dt, state, B, y, idx, wt, ws)
            ys.append(y.cpu()); idxs.append(idx.cpu()); wts.append(wt.cpu())
        assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
    finally:
        sb.swimba_destroy(h)
    got = dict(y=torch.stack(ys, 1), h_final=state.cpu(), idx=torch.stack(idxs, 1), w=torch.stack(wts, 1))
    res = hp.compare_forward(cfg, inp, got, *hp.tolerances(cfg))
    print(cfg, f"err_y={res['err_y']:.2e} err_h={res['err_h']:.2e} ambiguous={res['ambiguous']}")


@pytest.mark.parametrize("seed", range(10))
def test_random_weight_gradients_match_oracle(seed):
    import oracle
    import test_gpu_backward as tb
    r = np.random.default_rng(4000 + seed)
    tile = bool(r.integers(0, 3) > 0)
    G = int(r.choice([1, 2]))
    H = G * int(r.integers(1, 4))
    E = int(r.choice([1, 2, 4, 8]))
    k = int(r.integers(1, min(E, 3) + 1))
    F = 8 * int(r.integers(2, 40))
    B = int(r.integers(1, 4))
    if tile:
        dtype, P, N = "bf16", 64, 128
        L = int(r.choice([1, int(r.integers(2, 200)), int(r.integers(200, 900)), int(r.integers(1500, 2600))]))
    else:
        dtype, P, N = str(r.choice(["bf16", "fp32"])), int(r.choice([16, 32, 64])), int(r.choice([16, 32, 64]))
        L = int(r.integers(1, 200))
    cfg = synth.LayerConfig("fuzz", dtype, B, L, F, H, P, N, G, E, k, 128)
    inp = synth.make_inputs(cfg, seed=seed, with_dt=bool(r.integers(0, 4) > 0))
    gen = torch.Generator().manual_seed(seed)
    dy = torch.randn(B, L, H, P, generator=gen).to(synth.torch_dtype(dtype))
    h0 = (0.1 * torch.randn(B, H, P, N, generator=gen)).float() if r.integers(0, 2) else None
    dWr, dWe, idx = tb.gpu_backward(cfg, inp, dy, h0=h0)
    W_r = inp["W_r"] if E > 1 else torch.zeros(1, F)
    ref = oracle.backward_weights(synth.f64(inp["u"]), synth.f64(inp["x"]), synth.f64(inp["dt"]), synth.f64(W_r),
                                  synth.f64(inp["W_e"]), synth.f64(inp["A"]), synth.f64(inp["dt_bias"]), synth.f64(dy),
                                  k=k, G=G, h0=synth.f64(h0), forced_idx=idx.numpy())
    tol = 2e-4 if dtype == "fp32" else 2e-2
    err_e = tb.rel_per_expert(dWe, ref["dW_e"])
    assert err_e <= tol, err_e
    if E > 1:
        den = np.abs(ref["dW_r"]).max()
        assert np.abs(dWr.double().numpy() - ref["dW_r"]).max() <= tol * den
    print(cfg, f"dW_e err={err_e:.2e}")
