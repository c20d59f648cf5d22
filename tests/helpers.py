"""Shared test plumbing: run one layer through the CUDA library and through the CPU oracle on the
same seeded host arrays, and compare under the routing protocol.

Routing protocol.  The library computes router logits from the same (bf16 or fp32) inputs in fp32,
the oracle in fp64.  A token is *certified* when the smallest gap among its k+1 largest oracle
logits exceeds twice the worst-case fp32 summation error F * 2^-24 * sum_f |W_r[e,f] u[t,f]|; for
those tokens indices must match bit for bit, order included.  The few remaining near-tied tokens
may differ; the oracle is then re-run with the library's routing forced so that every token's
float outputs are still compared.
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2603_06938_b200 import binding as sb
from paper_2603_06938_b200 import synth


def dtype_code(cfg: synth.LayerConfig) -> int:
    return sb.DTYPE_FP32 if cfg.dtype == "fp32" else sb.DTYPE_BF16


def create_handle(cfg: synth.LayerConfig, chunk=None, flags: int = 0) -> sb.Handle:
    return sb.swimba_create(cfg.F, cfg.H, cfg.P, cfg.N, cfg.G, cfg.E, cfg.k,
                            chunk if chunk is not None else cfg.Q, dtype_code(cfg), flags)


CANARY_BYTES = 1024


def with_canary(shape, dtype, fill):
    """A device tensor of the given shape followed in memory by CANARY_BYTES of a fixed pattern:
    returns (tensor view, whole byte buffer).  A kernel that writes past the end of its output or
    workspace damages the pattern."""
    n = 1
    for d in shape:
        n *= d
    es = torch.empty((), dtype=dtype).element_size()
    raw = torch.full((n * es + CANARY_BYTES,), 0xA5, dtype=torch.uint8, device="cuda")
    view = raw[:n * es].view(dtype).view(*shape)
    view.fill_(fill)
    return view, raw


def canary_intact(raw) -> bool:
    return bool((raw[-CANARY_BYTES:] == 0xA5).all())


def dev(t):
    return None if t is None else t.cuda().contiguous()


def device_weights(inp):
    keep = {n: dev(inp[n]) for n in ("W_r", "W_e", "A", "dt_bias", "D")}
    return sb.make_weights(keep["W_r"], keep["W_e"], keep["A"], keep["dt_bias"], keep["D"]), keep


def gpu_forward(cfg: synth.LayerConfig, inp, chunk=None, h0=None, want_topk=True, flags: int = 0):
    """Runs swimba_forward; returns host tensors dict(y, h_final, idx, w).  Outputs and workspace
    are followed by canary bytes, which must come back untouched."""
    h = create_handle(cfg, chunk, flags)
    try:
        B, L = inp["u"].shape[0], inp["u"].shape[1]
        w, keep = device_weights(inp)
        u, x, dt = dev(inp["u"]), dev(inp["x"]), dev(inp["dt"])
        h0d = dev(h0 if h0 is not None else inp.get("h0"))
        y, y_raw = with_canary(x.shape, x.dtype, float("nan"))
        hf, hf_raw = with_canary((B, cfg.H, cfg.P, cfg.N), torch.float32, float("nan"))
        idx = torch.full((B, L, cfg.k), -1, dtype=torch.int32, device="cuda") if want_topk else None
        wt = torch.full((B, L, cfg.k), float("nan"), device="cuda") if want_topk else None
        nws = max(sb.swimba_workspace_bytes(h, B, L), 16)
        ws, ws_raw = with_canary((nws,), torch.uint8, 0)
        sb.swimba_forward(h, w, u, x, dt, h0d, B, L, y, hf, idx, wt, ws)
        rc = sb.swimba_status(h)
        assert rc == 0, sb.swimba_last_error(h)
        assert canary_intact(y_raw) and canary_intact(hf_raw) and canary_intact(ws_raw), \
            "a kernel wrote past the end of y, h_final or the workspace"
        launches = sb.swimba_last_launch_count(h)
        return dict(y=y.cpu(), h_final=hf.cpu(), idx=None if idx is None else idx.cpu(),
                    w=None if wt is None else wt.cpu(), launches=launches)
    finally:
        sb.swimba_destroy(h)


def oracle_forward(cfg: synth.LayerConfig, inp, h0=None, forced_idx=None, forced_w=None):
    h0 = h0 if h0 is not None else inp.get("h0")
    return oracle.swimba_forward(
        synth.f64(inp["u"]), synth.f64(inp["x"]), synth.f64(inp["dt"]), synth.f64(inp["W_r"]),
        synth.f64(inp["W_e"]), synth.f64(inp["A"]), synth.f64(inp["dt_bias"]), synth.f64(inp["D"]),
        k=cfg.k, G=cfg.G, h0=synth.f64(h0), forced_idx=forced_idx, forced_w=forced_w)


def max_rel(got, ref) -> float:
    """max |got - ref| / max |ref| over the whole tensor."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    den = np.max(np.abs(ref))
    return float(np.max(np.abs(got - ref)) / (den if den > 0 else 1.0))


def _head_max(a, head_axis):
    """max |a| per (sequence, head): a is [B, ..., H, ...] with the head index at head_axis."""
    axes = tuple(i for i in range(a.ndim) if i not in (0, head_axis))
    return np.max(np.abs(a), axis=axes)


def per_head_rel(got, ref, head_axis) -> float:
    """max over (sequence, head) of max|got - ref| / max|ref|, both maxima taken inside that
    (sequence, head).  Heads differ by orders of magnitude in step size and decay, so one scale
    for the whole tensor would hide the small ones.  A (sequence, head) whose reference is
    identically zero must be reproduced as zero."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    err = _head_max(got - ref, head_axis)
    den = _head_max(ref, head_axis)
    rel = np.where(den > 0, err / np.where(den > 0, den, 1.0), np.where(err > 0, np.inf, 0.0))
    return float(rel.max())


def elementwise_rel(got, ref):
    """(max, 99.9th percentile) of |got - ref| / (|ref| + 1e-3 rms(ref)) over all elements."""
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    rms = float(np.sqrt(np.mean(ref * ref)))
    r = np.abs(got - ref) / (np.abs(ref) + 1e-3 * rms + 1e-300)
    return float(r.max()), float(np.percentile(r, 99.9))


BF16_EPS = 2.0 ** -8      # unit roundoff of a bf16 store
FP32_EPS = 2.0 ** -22     # the skip product and the final sum, each rounded once to fp32


def check_outputs(cfg: synth.LayerConfig, inp, got_y, got_h, ref, tol_y, tol_h):
    """y and final state against the oracle at the resolution of one (sequence, head).

    Final state: per (sequence, head) max-norm relative error <= tol_h.
    y, call without skip term (D is None): y is the readout Ctilde^T h alone; per (sequence, head)
    max-norm relative error <= tol_y.
    y, call with a skip term: y is dominated by D x, so the whole-tensor measure alone could not
    see the readout.  Here every element must satisfy
        |y - yref| <= tol_y * max_{(b,h)} |Ctilde^T h| + eps_out * |yref|
    i.e. the readout part is held to tol_y of its own per-head scale, and the only extra slack is
    the rounding of the stored y (eps_out = 2^-8 for bf16 outputs, 2^-22 for fp32: D x and the
    final sum are each rounded once).
    Sequences shorter than one 128-token tile are the one place where the readout of a whole
    (sequence, head) can nearly cancel (with a single token, y is one 128-term dot product
    Ctilde . Btilde of streams that are stored in bf16, times Delta x): there the per-head scale
    is floored by 1/16 of the same readout evaluated on absolute values, the scale a forward
    error bound is relative to.
    Also returned (not asserted): the elementwise measure |y - yref| / (|yref| + 1e-3 rms), its
    maximum and 99.9th percentile (the largest over sequences).  got_y / got_h: torch tensors."""
    D = inp.get("D")
    Dv = None if D is None else synth.f64(D)[None, :, None]
    eps_out = BF16_EPS if cfg.dtype == "bf16" else FP32_EPS
    floor = None
    if ref["y"].shape[1] < 128 and "BC" in ref:
        h0 = inp.get("h0")
        y_abs, _ = oracle.ssm_recurrence(np.abs(synth.f64(inp["x"])), np.abs(ref["BC"]), synth.f64(inp["dt"]),
                                         synth.f64(inp["A"]), synth.f64(inp["dt_bias"]), None,
                                         None if h0 is None else np.abs(synth.f64(h0)), G=cfg.G)
        floor = np.max(np.abs(y_abs), axis=(1, 3)) / 16.0                   # [B,H]
    eh = per_head_rel(got_h.double().numpy(), ref["h_final"], 1)
    y_den = float(np.max(np.abs(ref["y"])))
    ey, ey_whole, emax, e999 = 0.0, 0.0, 0.0, 0.0
    for b in range(ref["y"].shape[0]):           # one sequence at a time keeps the temporaries small
        gy = got_y[b].double().numpy()           # [L,H,P]
        ry = ref["y"][b]
        diff = np.abs(gy - ry)
        ey_whole = max(ey_whole, float(diff.max()) / (y_den if y_den > 0 else 1.0))
        ssm = ry if Dv is None else ry - Dv * synth.f64(inp["x"][b])
        scale = np.max(np.abs(ssm), axis=(0, 2))                          # [H]
        if floor is not None:
            scale = np.maximum(scale, floor[b])
        scale = scale[None, :, None]
        room = diff - (eps_out * np.abs(ry) if Dv is not None else 0.0)
        rel = np.where(scale > 0, room / np.where(scale > 0, scale, 1.0), np.where(room > 0, np.inf, 0.0))
        ey = max(ey, float(rel.max()))
        m, p = elementwise_rel(gy, ry)
        emax, e999 = max(emax, m), max(e999, p)
    assert ey_whole <= tol_y, f"y whole-tensor max-rel error {ey_whole:.3e} > {tol_y}"
    assert ey <= tol_y, f"y per-(sequence, head) error {ey:.3e} > {tol_y}"
    assert eh <= tol_h, f"h_final per-(sequence, head) error {eh:.3e} > {tol_h}"
    return dict(err_y=ey, err_y_whole=ey_whole, err_h=eh, err_y_elem_max=emax, err_y_elem_p999=e999)


def check_routing(cfg: synth.LayerConfig, inp, idx_gpu, w_gpu, require_all_certified=False):
    """Certified tokens must match exactly; returns (#uncertified tokens, oracle router output).
    r["mismatch"] counts the tokens (necessarily uncertified) whose routing differs from the
    oracle's own."""
    F = cfg.F
    u2 = synth.f64(inp["u"]).reshape(-1, F)
    r = oracle.router(u2, synth.f64(inp["W_r"]), cfg.k)
    idx_gpu = idx_gpu.numpy().reshape(-1, cfg.k)
    w_gpu = w_gpu.numpy().reshape(-1, cfg.k)
    bound = 2.0 * F * 2.0 ** -24 * r["absdot"]
    certified = r["margin"] > bound
    if cfg.E == cfg.k == 1:
        certified[:] = True
    assert np.array_equal(idx_gpu[certified], r["idx"][certified]), "certified routing differs"
    n_amb = int((~certified).sum())
    r["mismatch"] = int(np.any(idx_gpu != r["idx"], axis=-1).sum())
    if require_all_certified:
        assert n_amb == 0
    # ambiguous tokens must still pick k distinct valid experts
    assert idx_gpu.min() >= 0 and idx_gpu.max() < cfg.E
    if cfg.k > 1:
        srt = np.sort(idx_gpu, axis=-1)
        assert np.all(srt[:, 1:] != srt[:, :-1])
    # weights: softmax values of the chosen experts (no renormalisation)
    chosen = np.take_along_axis(r["pi"], idx_gpu.astype(np.int64), axis=-1)
    np.testing.assert_allclose(w_gpu, chosen, rtol=2e-5, atol=1e-7)
    return n_amb, r


def compare_forward(cfg: synth.LayerConfig, inp, got, tol_y, tol_h, h0=None,
                    require_all_certified=False):
    n_amb, r0 = check_routing(cfg, inp, got["idx"], got["w"], require_all_certified)
    B, L = inp["u"].shape[:2]
    forced_idx = got["idx"].numpy().reshape(B, L, cfg.k)
    forced_w = None
    if n_amb:
        # weights for the library's routing, in fp64, from the oracle's own softmax
        r = oracle.router(synth.f64(inp["u"]).reshape(-1, cfg.F), synth.f64(inp["W_r"]), cfg.k)
        forced_w = np.take_along_axis(r["pi"], forced_idx.reshape(-1, cfg.k).astype(np.int64), -1)
        ref = oracle_forward(cfg, inp, h0=h0, forced_idx=forced_idx, forced_w=forced_w)
    else:
        ref = oracle_forward(cfg, inp, h0=h0)
    res = check_outputs(cfg, inp, got["y"], got["h_final"], ref, tol_y, tol_h)
    res.update(ambiguous=n_amb, mismatch=r0["mismatch"], ref=ref)
    return res


def tolerances(cfg: synth.LayerConfig):
    """fp32 path: 1e-4 on everything; bf16 inputs with fp32 accumulation: 2e-2 on y, 1e-2 on state."""
    return (1e-4, 1e-4) if cfg.dtype == "fp32" else (2e-2, 1e-2)
