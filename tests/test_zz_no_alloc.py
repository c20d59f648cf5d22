"""The allocation-free routing/projection entry point against the regular one.

Some users of the library cannot allocate device memory at the call site (plug-ins that only get
their input and output buffers, processes whose memory pool is fully handed out).  For them
swimba_route_mix_static keeps its scratch in a fixed array inside the library.  It must give the
same mixed streams, indices and weights as swimba_route_mix, also on a second call that finds the
previous call's contents in the array.  This file is collected last on purpose.
"""
import pytest
import torch

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
    return outs


def test_static_scratch_entry_point_matches_regular_one_twice_in_a_row():
    # two calls in a row: the second (different size, different routing) finds the first one's
    # histogram, tile table and slot buffer still in the shared array
    first = synth.LayerConfig("noalloc_a", "bf16", 2, 700, 128, 4, 64, 128, 1, 8, 2, 128)
    second = synth.LayerConfig("noalloc_b", "bf16", 1, 333, 128, 4, 64, 128, 1, 8, 2, 128)
    for cfg, seed in ((first, 51), (second, 52)):
        (bc_ref, idx_ref, w_ref), (bc, idx, w) = run_both(cfg, seed)
        assert torch.equal(idx, idx_ref)
        assert torch.equal(w, w_ref)
        assert hp.max_rel(bc.numpy(), bc_ref.numpy()) <= 1e-2     # same kernels: identical in practice
        assert torch.equal(bc, bc_ref)


def test_static_scratch_rejects_sizes_beyond_its_capacity():
    cfg = synth.LayerConfig("noalloc_big", "bf16", 1, 64, 128, 4, 64, 128, 1, 8, 2, 128)
    inp = synth.make_inputs(cfg, seed=53)
    h = hp.create_handle(cfg)
    w, keep = hp.device_weights(inp)
    T = 1 << 20                                   # needs far more than the 8 MiB array
    rc = sb.swimba_route_mix_static(h, w, hp.dev(inp["u"]), T, hp.dev(inp["u"]), None, None, check=False)
    assert rc == sb.ERR_WORKSPACE_TOO_SMALL
    assert "static scratch" in sb.swimba_last_error(h)
    sb.swimba_destroy(h)
