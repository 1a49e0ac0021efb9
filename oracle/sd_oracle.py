"""TEST INFRASTRUCTURE: ctypes front end of the CPU oracle in ``sd_oracle.c``.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this module.
It compiles ``sd_oracle.c`` with gcc on first use (``build()``), loads it and exposes
``verify_feedback``, ``draw_interval``, ``verify_greedy`` and ``ensemble_feedback``, which take and return numpy arrays.  Nothing here touches CUDA and nothing
here is imported by the product package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sd_oracle.c")
_LIB = os.path.join(_HERE, "libsd_oracle.so")
_lib = None

F32 = 0
BF16 = 1


def build(force: bool = False) -> str:
    """Compile the oracle into a shared object next to its source; returns the path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        P = ctypes.c_void_p
        lib.sd_oracle.restype = ctypes.c_int
        lib.sd_oracle.argtypes = [P, P, ctypes.c_int, P, P, ctypes.c_double, ctypes.c_int,
                                  ctypes.c_int, ctypes.c_int, P, P, P, P, P, P, P, P, P,
                                  ctypes.c_int]
        lib.sd_oracle_draw_interval.restype = ctypes.c_int
        lib.sd_oracle_draw_interval.argtypes = [P, P, ctypes.c_int, ctypes.c_double, ctypes.c_int, ctypes.c_int,
                                                ctypes.c_int, ctypes.c_int, P]
        lib.sd_oracle_hint_error.restype = ctypes.c_int
        lib.sd_oracle_hint_error.argtypes = [P, P, P, ctypes.c_int, ctypes.c_double, ctypes.c_int, ctypes.c_int,
                                             ctypes.c_int, P]
        lib.sd_oracle_lmhead_grad.restype = ctypes.c_int
        lib.sd_oracle_lmhead_grad.argtypes = [P, ctypes.c_int, P, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                              ctypes.c_longlong, P, P, P]
        lib.sd_oracle_greedy.restype = ctypes.c_int
        lib.sd_oracle_greedy.argtypes = [P, ctypes.c_int, P, ctypes.c_int, ctypes.c_int, ctypes.c_int, P, P, P]
        lib.sd_oracle_ensemble.restype = ctypes.c_int
        lib.sd_oracle_ensemble.argtypes = [P, P, ctypes.c_int, ctypes.c_int, ctypes.c_double, ctypes.c_double,
                                           ctypes.c_int, ctypes.c_int, ctypes.c_int, P, P, P, P, P, P,
                                           ctypes.c_int]
        lib.sd_oracle_max_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def max_threads() -> int:
    return int(_load().sd_oracle_max_threads())


@dataclass
class OracleResult:
    accept_len: np.ndarray          # [B] int32
    tokens: np.ndarray              # [B,k+1] int32, -1 padded
    loss: Optional[np.ndarray]      # [B,k] float64  KL(p||q)
    grad: Optional[np.ndarray]      # [B,k,V] float64 (q-p)/tau
    acc_prob: np.ndarray            # [B,k] float64 sum min(p,q)
    ratio: np.ndarray               # [B,k] float64 p(x)/q(x)
    accept_band: np.ndarray         # [B,k] uint8: reached test with |u - p/q| < 1e-6
    cdf_margin: np.ndarray          # [B] float64
    status: np.ndarray              # [B] uint32


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def verify_feedback(target_logits: np.ndarray, draft_logits: np.ndarray, draft_tokens: np.ndarray,
                    uniforms: np.ndarray, temperature: float, *, want_grad: bool = True,
                    want_loss: bool = True, nthreads: int = 1) -> OracleResult:
    """Run the oracle.  Logits are float32 arrays, or uint16 arrays holding bf16 bit patterns."""
    T = np.ascontiguousarray(target_logits)
    D = np.ascontiguousarray(draft_logits)
    if T.dtype == np.float32 and D.dtype == np.float32:
        dtype = F32
    elif T.dtype == np.uint16 and D.dtype == np.uint16:
        dtype = BF16
    else:
        raise TypeError("logits must both be float32 or both be uint16 (bf16 bits)")
    if T.ndim != 3 or D.ndim != 3:
        raise ValueError("logits must be [B,k+1,V] and [B,k,V]")
    B, k1, V = T.shape
    k = k1 - 1
    if D.shape != (B, k, V):
        raise ValueError(f"draft logits {D.shape} do not match target logits {T.shape}")
    x = np.ascontiguousarray(draft_tokens, dtype=np.int32)
    u = np.ascontiguousarray(uniforms, dtype=np.float32)
    if x.shape != (B, k) or u.shape != (B, k + 1):
        raise ValueError("draft_tokens must be [B,k] and uniforms [B,k+1]")
    res = OracleResult(
        accept_len=np.empty(B, np.int32), tokens=np.empty((B, k + 1), np.int32),
        loss=np.empty((B, k), np.float64) if want_loss else None,
        grad=np.empty((B, k, V), np.float64) if want_grad else None,
        acc_prob=np.empty((B, k), np.float64), ratio=np.empty((B, k), np.float64),
        accept_band=np.empty((B, k), np.uint8), cdf_margin=np.empty(B, np.float64),
        status=np.empty(B, np.uint32))
    rc = _load().sd_oracle(_ptr(T), _ptr(D), dtype, _ptr(x), _ptr(u), float(temperature), B, k, V,
                           _ptr(res.accept_len), _ptr(res.tokens), _ptr(res.loss), _ptr(res.grad),
                           _ptr(res.acc_prob), _ptr(res.ratio), _ptr(res.accept_band),
                           _ptr(res.cdf_margin), _ptr(res.status), int(nthreads))
    if rc != 0:
        raise RuntimeError(f"sd_oracle failed with code {rc}")
    return res


def draw_interval(target_logits: np.ndarray, draft_logits: np.ndarray, temperature: float, n: int, y: int):
    """Where token ``y`` sits on the inverse CDF the extra token of ONE sequence ([k+1,V] and [k,V]
    logits) is drawn from when its accept length is ``n``: returns (c_before, c_after, R); the draw
    with uniform u gives ``y`` exactly when c_before <= u*R < c_after."""
    T = np.ascontiguousarray(target_logits)
    D = np.ascontiguousarray(draft_logits)
    if T.dtype == np.float32 and D.dtype == np.float32:
        dtype = F32
    elif T.dtype == np.uint16 and D.dtype == np.uint16:
        dtype = BF16
    else:
        raise TypeError("logits must both be float32 or both be uint16 (bf16 bits)")
    if T.ndim != 2 or D.ndim != 2 or T.shape[0] != D.shape[0] + 1 or T.shape[1] != D.shape[1]:
        raise ValueError("logits of one sequence: [k+1,V] and [k,V]")
    out = np.empty(3, np.float64)
    rc = _load().sd_oracle_draw_interval(_ptr(T), _ptr(D), dtype, float(temperature), D.shape[0], T.shape[1],
                                         int(n), int(y), _ptr(out))
    if rc != 0:
        raise RuntimeError(f"sd_oracle_draw_interval failed with code {rc}")
    return float(out[0]), float(out[1]), float(out[2])


def _code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError("arrays must be float32 or uint16 (bf16 bits)")


def hint_error(target_logits: np.ndarray, draft_logits: np.ndarray, hint: np.ndarray, temperature: float) -> np.ndarray:
    """Squared distance, per position, between the hint of the optimistic update (the last round's
    gradient, Sec. 3.2) and this round's gradient (q - p)/tau with respect to the draft logits:
    [B,k] float64."""
    T = np.ascontiguousarray(target_logits)
    D = np.ascontiguousarray(draft_logits)
    H = np.ascontiguousarray(hint)
    if not (T.dtype == D.dtype == H.dtype):
        raise TypeError("logits and hint must share one dtype")
    B, k1, V = T.shape
    k = k1 - 1
    if D.shape != (B, k, V) or H.shape != (B, k, V):
        raise ValueError("draft logits and hint must be [B,k,V]")
    out = np.empty((B, k), np.float64)
    rc = _load().sd_oracle_hint_error(_ptr(T), _ptr(D), _ptr(H), _code(T), float(temperature), B, k, V, _ptr(out))
    if rc != 0:
        raise RuntimeError(f"sd_oracle_hint_error failed with code {rc}")
    return out


def lmhead_grad(grad_logits: np.ndarray, hidden: np.ndarray, vs=None, js=None) -> np.ndarray:
    """Gradient of the round's loss with respect to the weights of a linear output layer of the draft,
    dW = g^T X for g [R,V] (gradient w.r.t. the draft logits) and X [R,d] (hidden states): all of it
    ([V,d] float64) or only the entries (vs[e], js[e])."""
    g = np.ascontiguousarray(grad_logits)
    X = np.ascontiguousarray(hidden)
    if g.ndim != 2 or X.ndim != 2 or g.shape[0] != X.shape[0]:
        raise ValueError("g must be [R,V] and X [R,d]")
    R, V = g.shape
    d = X.shape[1]
    if vs is None:
        out = np.empty((V, d), np.float64)
        rc = _load().sd_oracle_lmhead_grad(_ptr(g), _code(g), _ptr(X), _code(X), R, V, d, -1, None, None, _ptr(out))
    else:
        vs = np.ascontiguousarray(vs, dtype=np.int32)
        js = np.ascontiguousarray(js, dtype=np.int32)
        out = np.empty(vs.shape[0], np.float64)
        rc = _load().sd_oracle_lmhead_grad(_ptr(g), _code(g), _ptr(X), _code(X), R, V, d, vs.shape[0], _ptr(vs), _ptr(js),
                                           _ptr(out))
    if rc != 0:
        raise RuntimeError(f"sd_oracle_lmhead_grad failed with code {rc}")
    return out


@dataclass
class GreedyResult:
    accept_len: np.ndarray          # [B] int32
    tokens: np.ndarray              # [B,k+1] int32, -1 padded
    argmax: np.ndarray              # [B,k+1] int32: first index of the largest target logit of every row


def verify_greedy(target_logits: np.ndarray, draft_tokens: np.ndarray) -> GreedyResult:
    """Greedy verification (Algorithm 1 in the limit tau -> 0).  Logits as in ``verify_feedback``."""
    T = np.ascontiguousarray(target_logits)
    if T.dtype == np.float32:
        dtype = F32
    elif T.dtype == np.uint16:
        dtype = BF16
    else:
        raise TypeError("logits must be float32 or uint16 (bf16 bits)")
    if T.ndim != 3:
        raise ValueError("logits must be [B,k+1,V]")
    B, k1, V = T.shape
    k = k1 - 1
    x = np.ascontiguousarray(draft_tokens, dtype=np.int32)
    if x.shape != (B, k):
        raise ValueError("draft_tokens must be [B,k]")
    res = GreedyResult(accept_len=np.empty(B, np.int32), tokens=np.empty((B, k + 1), np.int32),
                       argmax=np.empty((B, k + 1), np.int32))
    rc = _load().sd_oracle_greedy(_ptr(T), dtype, _ptr(x), B, k, V, _ptr(res.accept_len), _ptr(res.tokens),
                                  _ptr(res.argmax))
    if rc != 0:
        raise RuntimeError(f"sd_oracle_greedy failed with code {rc}")
    return res


@dataclass
class EnsembleResult:
    loss: np.ndarray                # [N,B,k] float64 KL(p || q^n)
    grad: Optional[list]            # N arrays [B,k,V] float64, or None
    round_loss: np.ndarray          # [N] mean loss of the round
    cum_loss: np.ndarray            # [N] cumulative loss including this round
    weights: np.ndarray             # [N] Hedge weights of the next round


def ensemble_feedback(target_logits: np.ndarray, draft_logits: Sequence[np.ndarray], tau: float, eps: float,
                      cum_loss: Optional[np.ndarray] = None, want_grad: bool = True,
                      nthreads: int = 1) -> EnsembleResult:
    """Feedback for an online ensemble of N draft models (Sec. 3.3) and the Hedge weights."""
    T = np.ascontiguousarray(target_logits)
    if T.dtype == np.float32:
        dtype = F32
    elif T.dtype == np.uint16:
        dtype = BF16
    else:
        raise TypeError("logits must be float32 or uint16 (bf16 bits)")
    B, k1, V = T.shape
    k = k1 - 1
    Ds = [np.ascontiguousarray(d) for d in draft_logits]
    N = len(Ds)
    for d in Ds:
        if d.dtype != T.dtype or d.shape != (B, k, V):
            raise ValueError("every draft logit set must be [B,k,V] of the target's dtype")
    dptr = (ctypes.c_void_p * N)(*[d.ctypes.data for d in Ds])
    grads = [np.empty((B, k, V), np.float64) for _ in range(N)] if want_grad else None
    gptr = (ctypes.c_void_p * N)(*[g.ctypes.data for g in grads]) if want_grad else None
    cum_in = None if cum_loss is None else np.ascontiguousarray(cum_loss, dtype=np.float64)
    res = EnsembleResult(loss=np.empty((N, B, k), np.float64), grad=grads, round_loss=np.empty(N, np.float64),
                         cum_loss=np.empty(N, np.float64), weights=np.empty(N, np.float64))
    rc = _load().sd_oracle_ensemble(_ptr(T), dptr, N, dtype, ctypes.c_double(tau), ctypes.c_double(eps), B, k, V,
                                    _ptr(cum_in) if cum_in is not None else None, _ptr(res.loss), gptr,
                                    _ptr(res.round_loss), _ptr(res.cum_loss), _ptr(res.weights), int(nthreads))
    if rc != 0:
        raise RuntimeError(f"sd_oracle_ensemble failed with code {rc}")
    return res


@dataclass
class ErrorFeedbackResult:
    full: OracleResult              # the whole step (accept lengths, tokens, losses of every position, bands)
    error_grad: np.ndarray          # [B,V] float64: gradient row of the first rejected position, zeros if none


def error_position_feedback(target_logits: np.ndarray, draft_logits: np.ndarray, draft_tokens: np.ndarray,
                            uniforms: np.ndarray, tau: float, nthreads: int = 1) -> ErrorFeedbackResult:
    """The step with the feedback restricted to the error position (what OSD collects, Sec. 3.1):
    verification as in ``verify_feedback``; of the gradient only the row of the first rejected
    position n_b of every sequence, a zero row where every draft token was accepted."""
    full = verify_feedback(target_logits, draft_logits, draft_tokens, uniforms, tau, want_grad=True,
                           nthreads=nthreads)
    B, k, V = full.grad.shape
    eg = np.zeros((B, V), np.float64)
    for b in range(B):
        n = int(full.accept_len[b])
        if n < k:
            eg[b] = full.grad[b, n]
    return ErrorFeedbackResult(full=full, error_grad=eg)
