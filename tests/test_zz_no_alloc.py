"""The allocation-free routing/projection entry point against the regular one.

Some users of the library cannot allocate device memory at the call site (plug-ins that only get
their input and output buffers, processes whose memory pool is fully handed out).  For them
swimba_route_mix_static keeps its scratch in a fixed array inside the library.  It must give the
same mixed streams, indices and weights as swimba_route_mix, also on a second call that finds the
previous call's contents in the array.  This file is collected last on purpose.
"""
import pytest
import torch

import oracle

from paper_2603_06938_b200 import binding as sb
from paper_2603_06938_b200 import synth

import helpers as hp

pytestmark = pytest.mark.gpu


def run_both(cfg, seed):
    inp = synth.make_inputs(cfg, seed=seed)
    T = cfg.B * cfg.L
    h = hp.create_handle(cfg)
    w, keep = hp.device_weights(inp)
    u = hp.dev(inp["u"])
    outs = []
    for static in (False, True):
        BC = torch.full((T, cfg.S), float("nan"), dtype=u.dtype, device="cuda")
        idx = torch.full((T, cfg.k), -1, dtype=torch.int32, device="cuda")
        wt = torch.full((T, cfg.k), float("nan"), device="cuda")
        if static:
            sb.swimba_route_mix_static(h, w, u, T, BC, idx, wt)
        else:
            ws = torch.empty(sb.swimba_workspace_bytes(h, cfg.B, cfg.L), dtype=torch.uint8, device="cuda")
            sb.swimba_route_mix(h, w, u, T, BC, idx, wt, ws)
        assert sb.swimba_status(h) == 0, sb.swimba_last_error(h)
        outs.append((BC.float().cpu(), idx.cpu(), wt.cpu()))
    sb.swimba_destroy(h)
    return inp, outs


def lc(name, dtype, B, L, E, k):
    return synth.LayerConfig(name, dtype, B, L, 128, 4, 64, 128, 1, E, k, 128)


# two calls in a row per case: the second (different size, different routing) finds the first one's
# histogram, per-expert lists (and, for k > 2, slot buffer) still in the shared array
@pytest.mark.parametrize("first,second", [
    (lc("noalloc_a", "bf16", 2, 700, 8, 2), lc("noalloc_b", "bf16", 1, 333, 8, 2)),    # rows added in place
    (lc("noalloc_c", "bf16", 2, 500, 8, 3), lc("noalloc_d", "bf16", 1, 777, 8, 3)),    # slot buffer + slot sum
    (lc("noalloc_e", "fp32", 1, 300, 4, 2), lc("noalloc_f", "fp32", 2, 150, 4, 2)),    # fp32 path: routing scratch only
], ids=["bf16_k2", "bf16_k3", "fp32"])
def test_static_scratch_entry_point_matches_regular_one_twice_in_a_row(first, second):
    for cfg, seed in ((first, 51), (second, 52)):
        inp, ((bc_ref, idx_ref, w_ref), (bc, idx, w)) = run_both(cfg, seed)
        assert torch.equal(idx, idx_ref)
        assert torch.equal(w, w_ref)
        assert hp.max_rel(bc.numpy(), bc_ref.numpy()) <= 1e-2     # same kernels: identical in practice
        assert torch.equal(bc, bc_ref)
        # and against the CPU oracle: routing under the margin protocol, mixed streams given that routing
        hp.check_routing(cfg, inp, idx, w)
        T = cfg.B * cfg.L
        ref_bc = oracle.mix_topk(synth.f64(inp["u"]).reshape(T, -1), synth.f64(inp["W_e"]),
                                 idx.numpy().reshape(T, -1), w.double().numpy().reshape(T, -1))
        tol = 1e-2 if cfg.dtype == "bf16" else 1e-4
        assert hp.max_rel(bc.double().numpy(), ref_bc) <= tol


def test_static_scratch_serves_the_documented_token_count():
    # 100 000 tokens at E = 8, k = 2 need 4.8 MB of the 8 MiB array
    cfg = synth.LayerConfig("noalloc_many", "bf16", 1, 100000, 64, 2, 64, 128, 1, 8, 2, 128)
    inp, ((bc_ref, idx_ref, w_ref), (bc, idx, w)) = run_both(cfg, 54)
    assert torch.equal(idx, idx_ref) and torch.equal(w, w_ref) and torch.equal(bc, bc_ref)


def test_static_scratch_rejects_sizes_beyond_its_capacity():
    cfg = synth.LayerConfig("noalloc_big", "bf16", 1, 64, 128, 4, 64, 128, 1, 8, 2, 128)
    inp = synth.make_inputs(cfg, seed=53)
    h = hp.create_handle(cfg)
    w, keep = hp.device_weights(inp)
    T = 1 << 20                                   # 48 bytes of scratch per token: 48 MiB
    rc = sb.swimba_route_mix_static(h, w, hp.dev(inp["u"]), T, hp.dev(inp["u"]), None, None, check=False)
    assert rc == sb.ERR_WORKSPACE_TOO_SMALL
    assert "static scratch" in sb.swimba_last_error(h)
    sb.swimba_destroy(h)
