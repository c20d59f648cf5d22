"""Double-precision CPU oracle of the Swimba token mixer.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library and its Python binding never
import this package, and this package never imports them.

`build()` compiles `swimba_oracle.c` into `liboracle.so` beside it; the
functions below are thin numpy/ctypes wrappers (argument marshalling only, all
arithmetic is in the C file).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "swimba_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over independent sequences/heads)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
    return _lib


def _d(a, shape=None) -> Optional[np.ndarray]:
    if a is None:
        return None
    a = np.ascontiguousarray(np.asarray(a, dtype=np.float64))
    if shape is not None:
        assert a.shape == tuple(shape), (a.shape, shape)
    return a


def _i(a, shape=None) -> Optional[np.ndarray]:
    if a is None:
        return None
    a = np.ascontiguousarray(np.asarray(a, dtype=np.int32))
    if shape is not None:
        assert a.shape == tuple(shape), (a.shape, shape)
    return a


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check(rc: int, name: str):
    if rc != 0:
        raise ValueError(f"{name} failed with code {rc}")


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def router(u, W_r, k: int):
    """Router softmax over all E experts + top-k without renormalisation.

    u[T,F], W_r[E,F] -> dict(idx[T,k], w[T,k], pi[T,E], margin[T], absdot[T]).
    """
    u = _d(u)
    W_r = _d(W_r)
    T, F = u.shape
    E = W_r.shape[0]
    assert W_r.shape == (E, F)
    idx = np.zeros((T, k), np.int32)
    w = np.zeros((T, k), np.float64)
    pi = np.zeros((T, E), np.float64)
    margin = np.zeros((T,), np.float64)
    absdot = np.zeros((T,), np.float64)
    rc = _load().oracle_router(_p(u), _p(W_r), ctypes.c_long(T), F, E, k,
                               _p(idx), _p(w), _p(pi), _p(margin), _p(absdot))
    _check(rc, "oracle_router")
    return dict(idx=idx, w=w, pi=pi, margin=margin, absdot=absdot)


def expert_streams(u, W_e):
    """u[T,F], W_e[E,S,F] -> BCe[T,E,S] (every expert projected)."""
    u = _d(u)
    W_e = _d(W_e)
    T, F = u.shape
    E, S, F2 = W_e.shape
    assert F2 == F
    out = np.zeros((T, E, S), np.float64)
    _check(_load().oracle_expert_streams(_p(u), _p(W_e), ctypes.c_long(T), F, S, E, _p(out)),
           "oracle_expert_streams")
    return out


def mix_topk(u, W_e, idx, w):
    """BC[T,S] = sum_j w[t,j] * W_e[idx[t,j]] u_t."""
    u = _d(u)
    W_e = _d(W_e)
    T, F = u.shape
    E, S, _ = W_e.shape
    idx = _i(idx)
    k = idx.shape[1]
    w = _d(w, (T, k))
    out = np.zeros((T, S), np.float64)
    _check(_load().oracle_mix_topk(_p(u), _p(W_e), ctypes.c_long(T), F, S, E, k, _p(idx), _p(w),
                                   _p(out)), "oracle_mix_topk")
    return out


def mix_dense(u, W_e, pi):
    """BC[T,S] = sum_e pi[t,e] * W_e[e] u_t for arbitrary dense weights."""
    u = _d(u)
    W_e = _d(W_e)
    T, F = u.shape
    E, S, _ = W_e.shape
    pi = _d(pi, (T, E))
    out = np.zeros((T, S), np.float64)
    _check(_load().oracle_mix_dense(_p(u), _p(W_e), ctypes.c_long(T), F, S, E, _p(pi), _p(out)),
           "oracle_mix_dense")
    return out


def ssm_recurrence(x, BC, dt, A, dt_bias, D=None, h0=None, G: int = 1, want_traj: bool = False):
    """Per-timestep recurrence on given mixed streams.

    x[B,L,H,P], BC[B,L,2GN], dt[B,L,H] or None -> y, h_final (and h_traj[B,L,H,P,N]).
    """
    x = _d(x)
    B, L, H, P = x.shape
    BC = _d(BC)
    S = BC.shape[-1]
    N = S // (2 * G)
    BC = BC.reshape(B, L, S)
    dt = _d(dt, (B, L, H)) if dt is not None else None
    A = _d(A, (H,))
    dt_bias = _d(dt_bias, (H,))
    D = _d(D, (H,)) if D is not None else None
    h0 = _d(h0, (B, H, P, N)) if h0 is not None else None
    y = np.zeros((B, L, H, P), np.float64)
    hf = np.zeros((B, H, P, N), np.float64)
    traj = np.zeros((B, L, H, P, N), np.float64) if want_traj else None
    _check(_load().oracle_ssm_recurrence(_p(x), _p(BC), _p(dt), _p(A), _p(dt_bias), _p(D), _p(h0),
                                         B, L, H, P, N, G, _p(y), _p(hf), _p(traj)),
           "oracle_ssm_recurrence")
    return (y, hf, traj) if want_traj else (y, hf)


def mixed_general(xe, BCe, pi, dt, A, dt_bias, h0=None, G: int = 1, want_traj: bool = False):
    """General mixed model with expert-specific inputs xe[B,L,E,H,P]."""
    xe = _d(xe)
    B, L, E, H, P = xe.shape
    BCe = _d(BCe).reshape(B, L, E, -1)
    S = BCe.shape[-1]
    N = S // (2 * G)
    pi = _d(pi).reshape(B, L, E)
    dt = _d(dt, (B, L, H)) if dt is not None else None
    A = _d(A, (H,))
    dt_bias = _d(dt_bias, (H,))
    h0 = _d(h0, (B, H, P, N)) if h0 is not None else None
    y = np.zeros((B, L, H, P), np.float64)
    hf = np.zeros((B, H, P, N), np.float64)
    traj = np.zeros((B, L, H, P, N), np.float64) if want_traj else None
    _check(_load().oracle_mixed_general(_p(xe), _p(BCe), _p(pi), _p(dt), _p(A), _p(dt_bias),
                                        _p(h0), B, L, E, H, P, N, G, _p(y), _p(hf), _p(traj)),
           "oracle_mixed_general")
    return (y, hf, traj) if want_traj else (y, hf)


def separated(xe, BCe, pi, dt, A, dt_bias, h0e=None, G: int = 1, want_traj: bool = False):
    """MoE over separated SSMs: one state per expert, readout weighted by pi."""
    xe = _d(xe)
    B, L, E, H, P = xe.shape
    BCe = _d(BCe).reshape(B, L, E, -1)
    S = BCe.shape[-1]
    N = S // (2 * G)
    pi = _d(pi).reshape(B, L, E)
    dt = _d(dt, (B, L, H)) if dt is not None else None
    A = _d(A, (H,))
    dt_bias = _d(dt_bias, (H,))
    h0e = _d(h0e, (B, E, H, P, N)) if h0e is not None else None
    y = np.zeros((B, L, H, P), np.float64)
    hf = np.zeros((B, E, H, P, N), np.float64)
    traj = np.zeros((B, L, E, H, P, N), np.float64) if want_traj else None
    _check(_load().oracle_separated(_p(xe), _p(BCe), _p(pi), _p(dt), _p(A), _p(dt_bias), _p(h0e),
                                    B, L, E, H, P, N, G, _p(y), _p(hf), _p(traj)),
           "oracle_separated")
    return (y, hf, traj) if want_traj else (y, hf)


def swimba_forward(u, x, dt, W_r, W_e, A, dt_bias, D, k: int, G: int = 1, h0=None,
                   forced_idx=None, forced_w=None):
    """Whole layer: u[B,L,F], x[B,L,H,P] -> dict(y, h_final, idx, w, BC)."""
    u = _d(u)
    x = _d(x)
    B, L, F = u.shape
    _, _, H, P = x.shape
    W_e = _d(W_e)
    E, S, _ = W_e.shape
    N = S // (2 * G)
    W_r = _d(W_r, (E, F)) if W_r is not None else None
    dt = _d(dt, (B, L, H)) if dt is not None else None
    A = _d(A, (H,))
    dt_bias = _d(dt_bias, (H,))
    D = _d(D, (H,)) if D is not None else None
    h0 = _d(h0, (B, H, P, N)) if h0 is not None else None
    fi = _i(forced_idx).reshape(B * L, k) if forced_idx is not None else None
    fw = _d(forced_w).reshape(B * L, k) if forced_w is not None else None
    y = np.zeros((B, L, H, P), np.float64)
    hf = np.zeros((B, H, P, N), np.float64)
    idx = np.zeros((B, L, k), np.int32)
    w = np.zeros((B, L, k), np.float64)
    BC = np.zeros((B, L, S), np.float64)
    _check(_load().oracle_swimba_forward(_p(u), _p(x), _p(dt), _p(h0), _p(W_r), _p(W_e), _p(A),
                                         _p(dt_bias), _p(D), B, L, F, H, P, N, G, E, k,
                                         _p(fi), _p(fw), _p(y), _p(hf), _p(idx), _p(w), _p(BC)),
           "oracle_swimba_forward")
    return dict(y=y, h_final=hf, idx=idx, w=w, BC=BC)


def backward_weights(u, x, dt, W_r, W_e, A, dt_bias, dy, k: int, G: int = 1, h0=None, forced_idx=None):
    """Gradients of sum(dy * y) with respect to W_r [E,F] and W_e [E,S,F] (the parameters the paper
    trains), the active sets held fixed: dict(dW_r, dW_e, dBC [B,L,S], dpi [B,L,k])."""
    u = _d(u)
    x = _d(x)
    B, L, F = u.shape
    _, _, H, P = x.shape
    W_e = _d(W_e)
    E, S, _ = W_e.shape
    N = S // (2 * G)
    if k > 64:
        raise ValueError("k <= 64")
    W_r = _d(W_r, (E, F))
    dt = _d(dt, (B, L, H)) if dt is not None else None
    A = _d(A, (H,))
    dt_bias = _d(dt_bias, (H,))
    h0 = _d(h0, (B, H, P, N)) if h0 is not None else None
    dy = _d(dy, (B, L, H, P))
    fi = _i(forced_idx).reshape(B * L, k) if forced_idx is not None else None
    dW_r = np.zeros((E, F), np.float64)
    dW_e = np.zeros((E, S, F), np.float64)
    dBC = np.zeros((B, L, S), np.float64)
    dpi = np.zeros((B, L, k), np.float64)
    _check(_load().oracle_swimba_backward_weights(_p(u), _p(x), _p(dt), _p(h0), _p(W_r), _p(W_e), _p(A),
                                                  _p(dt_bias), _p(dy), B, L, F, H, P, N, G, E, k, _p(fi),
                                                  _p(dW_r), _p(dW_e), _p(dBC), _p(dpi)),
           "oracle_swimba_backward_weights")
    return dict(dW_r=dW_r, dW_e=dW_e, dBC=dBC, dpi=dpi)


def swimba_decode_step(u, x, dt, W_r, W_e, A, dt_bias, D, k: int, state, G: int = 1,
                       forced_idx=None, forced_w=None):
    """One token per sequence; `state`[B,H,P,N] (float64, C-contiguous) is updated in place."""
    u = _d(u)
    x = _d(x)
    B, F = u.shape
    _, H, P = x.shape
    W_e = _d(W_e)
    E, S, _ = W_e.shape
    N = S // (2 * G)
    assert isinstance(state, np.ndarray) and state.dtype == np.float64 and state.flags.c_contiguous
    assert state.shape == (B, H, P, N)
    W_r = _d(W_r, (E, F)) if W_r is not None else None
    dt = _d(dt, (B, H)) if dt is not None else None
    A = _d(A, (H,))
    dt_bias = _d(dt_bias, (H,))
    D = _d(D, (H,)) if D is not None else None
    fi = _i(forced_idx).reshape(B, k) if forced_idx is not None else None
    fw = _d(forced_w).reshape(B, k) if forced_w is not None else None
    y = np.zeros((B, H, P), np.float64)
    idx = np.zeros((B, k), np.int32)
    w = np.zeros((B, k), np.float64)
    _check(_load().oracle_swimba_decode_step(_p(u), _p(x), _p(dt), _p(W_r), _p(W_e), _p(A),
                                             _p(dt_bias), _p(D), B, F, H, P, N, G, E, k,
                                             _p(fi), _p(fw), _p(state), _p(y), _p(idx), _p(w)),
           "oracle_swimba_decode_step")
    return dict(y=y, idx=idx, w=w)


def conv_silu(xin, w, bias=None, state=None):
    """Causal depthwise convolution + SiLU.  xin[B,L,C], w[C,K], bias[C] or None, state[B,K-1,C] or
    None (the K-1 tokens before the call, oldest first) -> (out[B,L,C], state_out[B,K-1,C])."""
    xin = _d(xin)
    B, L, C = xin.shape
    w = _d(w)
    K = w.shape[1]
    assert w.shape == (C, K)
    bias = _d(bias, (C,)) if bias is not None else None
    state = _d(state, (B, K - 1, C)) if state is not None else None
    out = np.zeros((B, L, C), np.float64)
    st = np.zeros((B, K - 1, C), np.float64)
    _check(_load().oracle_conv_silu(_p(xin), _p(w), _p(bias), _p(state), B, L, C, K, _p(out), _p(st)),
           "oracle_conv_silu")
    return out, st


def gated_rmsnorm(y, z, weight, ngroups: int = 1, eps: float = 1e-5):
    """out = rmsnorm_groups(y * silu(z)) * weight.  y, z [T,D], weight [D]."""
    y = _d(y)
    T, D = y.shape
    z = _d(z, (T, D))
    weight = _d(weight, (D,))
    out = np.zeros((T, D), np.float64)
    _check(_load().oracle_gated_rmsnorm(_p(y), _p(z), _p(weight), ctypes.c_long(T), D, ngroups,
                                        ctypes.c_double(eps), _p(out)), "oracle_gated_rmsnorm")
    return out


def linear(x, W):
    """out[T,O] = x[T,F] W[O,F]^T."""
    x = _d(x)
    W = _d(W)
    T, F = x.shape
    O = W.shape[0]
    assert W.shape == (O, F)
    out = np.zeros((T, O), np.float64)
    _check(_load().oracle_linear(_p(x), _p(W), ctypes.c_long(T), F, O, _p(out)), "oracle_linear")
    return out


def block_forward(u, W_in, W_r, W_e, conv_w, conv_b, A, dt_bias, D, norm_w, W_out, H: int, k: int,
                  G: int = 1, eps: float = 1e-5, conv_state=None, h0=None, forced_idx=None,
                  forced_w=None):
    """The whole block around the mixer, step by step (the Mamba-2 block with its B / C projection
    replaced by the routed mixture of expert projections):
      [z | x' | dt] = W_in u                      shared in-projection (D = H*P channels each, H step sizes)
      [B' | C']     = router + top-k + expert projections + parameter-space mix of u
      [x | B | C]   = silu(causal depthwise conv([x' | B' | C']))
      y, h          = the single selective-SSM recurrence on (x, B, C, dt)
      out           = W_out ( rmsnorm(y * silu(z)) * norm_w )
    u[B,L,F] -> dict(out[B,L,F], h_final, conv_state, idx, w, y, BC)."""
    u = _d(u)
    B, L, F = u.shape
    W_in = _d(W_in)
    Dm = (W_in.shape[0] - H) // 2
    P = Dm // H
    T = B * L
    zxdt = linear(u.reshape(T, F), W_in)
    z, xp, dt = zxdt[:, :Dm], zxdt[:, Dm:2 * Dm], zxdt[:, 2 * Dm:]
    E, S, _ = np.asarray(W_e).shape
    if forced_idx is None:
        r = router(u.reshape(T, F), W_r, k)
        idx, wts = r["idx"], r["w"]
    else:
        idx, wts = _i(forced_idx).reshape(T, k), _d(forced_w).reshape(T, k)
    BCp = mix_topk(u.reshape(T, F), W_e, idx, wts)
    xbc, cst = conv_silu(np.concatenate([xp, BCp], -1).reshape(B, L, Dm + S), conv_w, conv_b, conv_state)
    x = np.ascontiguousarray(xbc[..., :Dm]).reshape(B, L, H, P)
    BC = np.ascontiguousarray(xbc[..., Dm:])
    y, hf = ssm_recurrence(x, BC, dt.reshape(B, L, H), A, dt_bias, D, h0, G=G)
    g = gated_rmsnorm(y.reshape(T, Dm), z, norm_w, ngroups=G, eps=eps)
    out = linear(g, W_out).reshape(B, L, -1)
    return dict(out=out, h_final=hf, conv_state=cst, idx=idx.reshape(B, L, k), w=wts.reshape(B, L, k),
                y=y, BC=BC, x=x, z=z.reshape(B, L, Dm), dt=dt.reshape(B, L, H))
