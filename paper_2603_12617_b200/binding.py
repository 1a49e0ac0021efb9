"""Thin ctypes binding of the C ABI in ``include/sd_verify.h``.

Argument marshalling only: every step of the verify-and-feedback path runs in the CUDA library.
torch is used for device memory, streams and nothing else.  The functions have the names of the
C entry points.  If the shared library is missing or cannot be loaded the import of this module
fails: there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

SD_DTYPE_F32 = 0
SD_DTYPE_BF16 = 1

SD_OPT_L2_PERSIST_MIB = 0
SD_OPT_CLUSTER = 1
SD_OPT_LAG = 2
SD_OPT_L2_BUDGET_MIB = 3
SD_OPT_FORCE_GENERIC = 4
SD_OPT_GREEDY_BLOCKS_PER_SM = 5
SD_OPT_WAIT_POLLS = 6
SD_OPT_PREFETCH = 7

SD_STATUS_BAD_TOKEN = 1
SD_STATUS_BAD_ROW = 2
SD_STATUS_ZERO_RESIDUAL = 4
SD_STATUS_TIMEOUT = 0x80000000

_HERE = os.path.dirname(os.path.abspath(__file__))
# SD_VERIFY_LIBRARY selects another build of the same library (the range-checked one); there is still no fallback.
LIB_PATH = os.environ.get("SD_VERIFY_LIBRARY") or os.path.join(_HERE, "lib", "libsd_verify.so")


class SdVerifyError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        text = _lib.sd_strerror(code).decode()
        detail = _lib.sd_last_cuda_error().decode()
        super().__init__(f"{where} failed with {code}: {text}" + (f" [{detail}]" if detail else ""))


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -c 'import __graft_entry__ as g; g.build()'` "
            "(there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    P, I, F, Z = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    lib.sd_verify_feedback.restype = I
    lib.sd_verify_feedback.argtypes = [P, P, P, P, F, I, I, I, P, P, P, P, P]
    lib.sd_verify_feedback_bf16.restype = I
    lib.sd_verify_feedback_bf16.argtypes = [P, P, P, P, F, I, I, I, P, P, P, P, P]
    lib.sd_verify_feedback_ex.restype = I
    lib.sd_verify_feedback_ex.argtypes = [P, P, P, P, F, I, I, I, I, P, P, P, P, P, P, P, Z, P]
    lib.sd_verify_feedback_static.restype = I
    lib.sd_verify_feedback_static.argtypes = [P, P, P, P, F, I, I, I, I, P, P, P, P, P, P, P]
    lib.sd_verify_greedy.restype = I
    lib.sd_verify_greedy.argtypes = [P, P, I, I, I, I, P, P, P, P, Z, P]
    lib.sd_greedy_workspace_bytes.restype = Z
    lib.sd_greedy_workspace_bytes.argtypes = [I, I]
    lib.sd_verify_error_feedback.restype = I
    lib.sd_verify_error_feedback.argtypes = [P, P, P, P, ctypes.c_float, I, I, I, I, P, P, P, P, P, P, Z, P]
    lib.sd_ensemble_feedback.restype = I
    lib.sd_ensemble_feedback.argtypes = [P, P, I, ctypes.c_float, ctypes.c_float, I, I, I, I, P, P, P, P, P, P, P,
                                         P, Z, P]
    lib.sd_lmhead_grad.restype = I
    lib.sd_lmhead_grad.argtypes = [P, P, I, I, I, P, P, P]
    lib.sd_hint_workspace_bytes.restype = Z
    lib.sd_hint_workspace_bytes.argtypes = [I, I, I, I]
    lib.sd_verify_feedback_hint.restype = I
    lib.sd_verify_feedback_hint.argtypes = [P, P, P, P, F, I, I, I, I, P, P, P, P, P, P, P, P, Z, P]
    lib.sd_vp_workspace_bytes.restype = Z
    lib.sd_vp_workspace_bytes.argtypes = [I, I, I, I]
    lib.sd_vp_partial.restype = I
    lib.sd_vp_partial.argtypes = [P, P, P, F, I, I, I, I, I, I, P, P, Z, P]
    lib.sd_vp_finish.restype = I
    lib.sd_vp_finish.argtypes = [P, P, P, P, F, I, I, I, I, I, I, P, I, I, P, P, P, P, P, P, Z, P]
    lib.sd_vp_draw.restype = I
    lib.sd_vp_draw.argtypes = [P, P, P, P, F, I, I, I, I, I, I, P, P, I, I, P, P, P, Z, P]
    lib.sd_verify_feedback_host.restype = I
    lib.sd_verify_feedback_host.argtypes = [P, P, P, P, F, I, I, I, I, P, P, P, P, P, P]
    lib.sd_workspace_bytes.restype = Z
    lib.sd_workspace_bytes.argtypes = [I, I, I, I]
    lib.sd_set_option.restype = I
    lib.sd_set_option.argtypes = [I, ctypes.c_longlong]
    lib.sd_get_option.restype = ctypes.c_longlong
    lib.sd_get_option.argtypes = [I]
    lib.sd_launch_info.restype = None
    lib.sd_launch_info.argtypes = [P] * 6
    lib.sd_release_cached_buffers.restype = None
    lib.sd_release_cached_buffers.argtypes = []
    lib.sd_strerror.restype = ctypes.c_char_p
    lib.sd_strerror.argtypes = [I]
    lib.sd_last_cuda_error.restype = ctypes.c_char_p
    lib.sd_last_cuda_error.argtypes = []
    lib.sd_version.restype = I
    lib.sd_version.argtypes = []
    lib.sd_bounds_report.restype = I
    lib.sd_bounds_report.argtypes = [P]
    return lib


_lib = _load()


@dataclass
class StepOutputs:
    accept_len: torch.Tensor            # [B] int32
    tokens: torch.Tensor                # [B,k+1] int32, -1 padded
    loss: Optional[torch.Tensor]        # [B,k] float32 KL(p||q)
    grad_draft: Optional[torch.Tensor]  # [B,k,V], dtype of the logits
    acc_prob: Optional[torch.Tensor] = None   # [B,k] float32
    status: Optional[torch.Tensor] = None     # [B] int32 view of the uint32 status words
    hint_err: Optional[torch.Tensor] = None   # [B,k] float32, sd_verify_feedback_hint only


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return SD_DTYPE_F32
    if t.dtype == torch.bfloat16:
        return SD_DTYPE_BF16
    raise TypeError(f"logits must be float32 or bfloat16, got {t.dtype}")


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _shapes(target_logits, draft_logits, draft_tokens, uniforms):
    if target_logits.dim() != 3 or draft_logits.dim() != 3:
        raise ValueError("logits must be [B,k+1,V] and [B,k,V]")
    B, k1, V = target_logits.shape
    k = k1 - 1
    if tuple(draft_logits.shape) != (B, k, V):
        raise ValueError(f"draft logits {tuple(draft_logits.shape)} do not match target {tuple(target_logits.shape)}")
    if tuple(draft_tokens.shape) != (B, k) or draft_tokens.dtype != torch.int32:
        raise ValueError("draft_tokens must be int32 [B,k]")
    if tuple(uniforms.shape) != (B, k + 1) or uniforms.dtype != torch.float32:
        raise ValueError("uniforms must be float32 [B,k+1]")
    if draft_logits.dtype != target_logits.dtype:
        raise TypeError("target and draft logits must have the same dtype")
    for t in (target_logits, draft_logits, draft_tokens, uniforms):
        if not t.is_contiguous():
            raise ValueError("inputs must be contiguous")
    return B, k, V


def _stream_ptr(stream: Optional[torch.cuda.Stream]):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def sd_version() -> int:
    return int(_lib.sd_version())


def sd_bounds_report() -> Optional[dict]:
    """Violations the range-checked build has counted since the last report (None: this build has no checks)."""
    out = (ctypes.c_ulonglong * 4)()
    rc = _lib.sd_bounds_report(out)
    if rc != 0:
        raise SdVerifyError(rc, "sd_bounds_report")
    if out[0] == 2 ** 64 - 1:
        return None
    return {"violations": int(out[0]), "site": int(out[1]), "index": int(out[2]), "limit": int(out[3])}


def sd_workspace_bytes(B: int, k: int, V: int, dtype: int) -> int:
    return int(_lib.sd_workspace_bytes(B, k, V, dtype))


def sd_launch_info() -> dict:
    vals = [ctypes.c_int(0) for _ in range(6)]
    _lib.sd_launch_info(*[ctypes.byref(v) for v in vals])
    keys = ["path", "cluster_size", "threads", "smem_bytes", "blocks", "kernels"]
    return {k: v.value for k, v in zip(keys, vals)}


def sd_set_option(option_id: int, value: int) -> None:
    rc = _lib.sd_set_option(int(option_id), int(value))
    if rc != 0:
        raise SdVerifyError(rc, "sd_set_option")


def sd_get_option(option_id: int) -> int:
    return int(_lib.sd_get_option(int(option_id)))


def sd_release_cached_buffers() -> None:
    _lib.sd_release_cached_buffers()


def sd_verify_feedback(target_logits: torch.Tensor, draft_logits: torch.Tensor,
                       draft_tokens: torch.Tensor, uniforms: torch.Tensor, temperature: float, *,
                       want_loss: bool = True, want_grad: bool = True,
                       out: Optional[StepOutputs] = None,
                       stream: Optional[torch.cuda.Stream] = None) -> StepOutputs:
    """``sd_verify_feedback`` / ``sd_verify_feedback_bf16`` on device tensors (library scratch)."""
    B, k, V = _shapes(target_logits, draft_logits, draft_tokens, uniforms)
    dev = target_logits.device
    if dev.type != "cuda":
        raise ValueError("device tensors required (use sd_verify_feedback_host for host tensors)")
    if out is None:
        out = StepOutputs(
            accept_len=torch.empty(B, dtype=torch.int32, device=dev),
            tokens=torch.empty((B, k + 1), dtype=torch.int32, device=dev),
            loss=torch.empty((B, k), dtype=torch.float32, device=dev) if (want_loss or want_grad) else None,
            grad_draft=torch.empty_like(draft_logits) if want_grad else None)
    fn = _lib.sd_verify_feedback if target_logits.dtype == torch.float32 else _lib.sd_verify_feedback_bf16
    _dtype_code(target_logits)
    with torch.cuda.device(dev):
        rc = fn(_ptr(target_logits), _ptr(draft_logits), _ptr(draft_tokens), _ptr(uniforms),
                float(temperature), B, k, V, _ptr(out.accept_len), _ptr(out.tokens), _ptr(out.loss),
                _ptr(out.grad_draft), _stream_ptr(stream))
    if rc != 0:
        raise SdVerifyError(rc, "sd_verify_feedback")
    return out


def sd_verify_feedback_ex(target_logits: torch.Tensor, draft_logits: torch.Tensor,
                          draft_tokens: torch.Tensor, uniforms: torch.Tensor, temperature: float, *,
                          want_loss: bool = True, want_grad: bool = True, want_acc_prob: bool = True,
                          want_status: bool = True, workspace: Optional[torch.Tensor] = None,
                          out: Optional[StepOutputs] = None,
                          stream: Optional[torch.cuda.Stream] = None) -> StepOutputs:
    """``sd_verify_feedback_ex`` on device tensors with caller-owned scratch."""
    B, k, V = _shapes(target_logits, draft_logits, draft_tokens, uniforms)
    dev = target_logits.device
    code = _dtype_code(target_logits)
    if workspace is None:
        workspace = torch.empty(sd_workspace_bytes(B, k, V, code), dtype=torch.uint8, device=dev)
    if out is None:
        out = StepOutputs(
            accept_len=torch.empty(B, dtype=torch.int32, device=dev),
            tokens=torch.empty((B, k + 1), dtype=torch.int32, device=dev),
            loss=torch.empty((B, k), dtype=torch.float32, device=dev) if (want_loss or want_grad) else None,
            grad_draft=torch.empty_like(draft_logits) if want_grad else None,
            acc_prob=torch.empty((B, k), dtype=torch.float32, device=dev) if want_acc_prob else None,
            status=torch.empty(B, dtype=torch.int32, device=dev) if want_status else None)
    with torch.cuda.device(dev):
        rc = _lib.sd_verify_feedback_ex(
            _ptr(target_logits), _ptr(draft_logits), _ptr(draft_tokens), _ptr(uniforms), float(temperature),
            B, k, V, code, _ptr(out.accept_len), _ptr(out.tokens), _ptr(out.loss), _ptr(out.grad_draft),
            _ptr(out.acc_prob), _ptr(out.status), _ptr(workspace), workspace.numel() * workspace.element_size(),
            _stream_ptr(stream))
    if rc != 0:
        raise SdVerifyError(rc, "sd_verify_feedback_ex")
    return out


def sd_hint_workspace_bytes(B: int, k: int, V: int, dtype: int) -> int:
    return int(_lib.sd_hint_workspace_bytes(B, k, V, dtype))


def sd_verify_feedback_hint(target_logits: torch.Tensor, draft_logits: torch.Tensor, draft_tokens: torch.Tensor,
                            uniforms: torch.Tensor, temperature: float, hint: torch.Tensor, *,
                            grad_out: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
                            stream: Optional[torch.cuda.Stream] = None) -> StepOutputs:
    """``sd_verify_feedback_hint``: the step plus sum_v (hint - gradient)^2 per position.  ``grad_out``
    may be ``hint`` itself (the gradient then replaces the hint in place)."""
    B, k, V = _shapes(target_logits, draft_logits, draft_tokens, uniforms)
    if tuple(hint.shape) != (B, k, V) or hint.dtype != draft_logits.dtype or not hint.is_contiguous():
        raise ValueError("hint must be a contiguous [B,k,V] tensor of the logits' dtype")
    dev = target_logits.device
    code = _dtype_code(target_logits)
    if workspace is None:
        workspace = torch.empty(sd_hint_workspace_bytes(B, k, V, code), dtype=torch.uint8, device=dev)
    out = StepOutputs(
        accept_len=torch.empty(B, dtype=torch.int32, device=dev),
        tokens=torch.empty((B, k + 1), dtype=torch.int32, device=dev),
        loss=torch.empty((B, k), dtype=torch.float32, device=dev),
        grad_draft=grad_out if grad_out is not None else torch.empty_like(draft_logits),
        status=torch.empty(B, dtype=torch.int32, device=dev),
        hint_err=torch.empty((B, k), dtype=torch.float32, device=dev))
    with torch.cuda.device(dev):
        rc = _lib.sd_verify_feedback_hint(
            _ptr(target_logits), _ptr(draft_logits), _ptr(draft_tokens), _ptr(uniforms), float(temperature),
            B, k, V, code, _ptr(hint), _ptr(out.accept_len), _ptr(out.tokens), _ptr(out.loss), _ptr(out.grad_draft),
            _ptr(out.hint_err), _ptr(out.status), _ptr(workspace), workspace.numel() * workspace.element_size(),
            _stream_ptr(stream))
    if rc != 0:
        raise SdVerifyError(rc, "sd_verify_feedback_hint")
    return out


@dataclass
class GreedyOutputs:
    accept_len: torch.Tensor            # [B] int32
    tokens: torch.Tensor                # [B,k+1] int32, -1 padded
    argmax: Optional[torch.Tensor]      # [B,k+1] int32


def sd_greedy_workspace_bytes(B: int, k: int) -> int:
    return int(_lib.sd_greedy_workspace_bytes(B, k))


def sd_verify_greedy(target_logits: torch.Tensor, draft_tokens: torch.Tensor, *, want_argmax: bool = True,
                     workspace: Optional[torch.Tensor] = None, out: Optional[GreedyOutputs] = None,
                     stream: Optional[torch.cuda.Stream] = None) -> GreedyOutputs:
    """``sd_verify_greedy`` on device tensors: accept iff the draft token is the target's argmax."""
    if target_logits.dim() != 3 or not target_logits.is_contiguous():
        raise ValueError("target logits must be contiguous [B,k+1,V]")
    B, k1, V = target_logits.shape
    k = k1 - 1
    if tuple(draft_tokens.shape) != (B, k) or draft_tokens.dtype != torch.int32 or not draft_tokens.is_contiguous():
        raise ValueError("draft_tokens must be contiguous int32 [B,k]")
    dev = target_logits.device
    if dev.type != "cuda":
        raise ValueError("device tensors required")
    code = _dtype_code(target_logits)
    if out is None:
        out = GreedyOutputs(accept_len=torch.empty(B, dtype=torch.int32, device=dev),
                            tokens=torch.empty((B, k + 1), dtype=torch.int32, device=dev),
                            argmax=torch.empty((B, k + 1), dtype=torch.int32, device=dev) if want_argmax else None)
    with torch.cuda.device(dev):
        rc = _lib.sd_verify_greedy(_ptr(target_logits), _ptr(draft_tokens), B, k, V, code, _ptr(out.accept_len),
                                   _ptr(out.tokens), _ptr(out.argmax), _ptr(workspace),
                                   0 if workspace is None else workspace.numel() * workspace.element_size(),
                                   _stream_ptr(stream))
    if rc != 0:
        raise SdVerifyError(rc, "sd_verify_greedy")
    return out


@dataclass
class ErrorFeedbackOutputs:
    accept_len: torch.Tensor            # [B] int32: also the position the gradient row belongs to
    tokens: torch.Tensor                # [B,k+1] int32, -1 padded
    loss: Optional[torch.Tensor]        # [B,k] float32 KL(p||q), every position
    error_grad: Optional[torch.Tensor]  # [B,V] gradient row of the first rejected position (zeros if none)
    status: Optional[torch.Tensor]      # [B] int32 view of the status words


def sd_verify_error_feedback(target_logits: torch.Tensor, draft_logits: torch.Tensor, draft_tokens: torch.Tensor,
                             uniforms: torch.Tensor, temperature: float, *, want_loss: bool = True,
                             want_grad: bool = True, want_status: bool = True,
                             out: Optional[ErrorFeedbackOutputs] = None,
                             stream: Optional[torch.cuda.Stream] = None) -> ErrorFeedbackOutputs:
    """``sd_verify_error_feedback`` on device tensors (library scratch)."""
    B, k, V = _shapes(target_logits, draft_logits, draft_tokens, uniforms)
    dev = target_logits.device
    if dev.type != "cuda":
        raise ValueError("device tensors required")
    code = _dtype_code(target_logits)
    if out is None:
        out = ErrorFeedbackOutputs(
            accept_len=torch.empty(B, dtype=torch.int32, device=dev),
            tokens=torch.empty((B, k + 1), dtype=torch.int32, device=dev),
            loss=torch.empty((B, k), dtype=torch.float32, device=dev) if want_loss else None,
            error_grad=torch.empty((B, V), dtype=target_logits.dtype, device=dev) if want_grad else None,
            status=torch.empty(B, dtype=torch.int32, device=dev) if want_status else None)
    with torch.cuda.device(dev):
        rc = _lib.sd_verify_error_feedback(_ptr(target_logits), _ptr(draft_logits), _ptr(draft_tokens), _ptr(uniforms),
                                           float(temperature), B, k, V, code, _ptr(out.accept_len), _ptr(out.tokens),
                                           _ptr(out.loss), _ptr(out.error_grad), _ptr(out.status), None, 0,
                                           _stream_ptr(stream))
    if rc != 0:
        raise SdVerifyError(rc, "sd_verify_error_feedback")
    return out


@dataclass
class EnsembleOutputs:
    loss: torch.Tensor                  # [N,B,k] float32 KL(p || q^n)
    grad: Optional[list]                # N tensors [B,k,V] in the dtype of the logits, or None
    round_loss: torch.Tensor            # [N] float64 mean loss of the round
    cum_loss: torch.Tensor              # [N] float64 cumulative loss including this round
    weights: torch.Tensor               # [N] float32 Hedge weights of the next round
    status: Optional[torch.Tensor]      # [B] int32 view of the status words


def sd_ensemble_feedback(target_logits: torch.Tensor, draft_logits, temperature: float, epsilon: float, *,
                         cum_loss: Optional[torch.Tensor] = None, want_grad: bool = True,
                         want_status: bool = False, out: Optional[EnsembleOutputs] = None,
                         stream: Optional[torch.cuda.Stream] = None) -> EnsembleOutputs:
    """``sd_ensemble_feedback`` on device tensors: N draft logit sets against one target."""
    if target_logits.dim() != 3 or not target_logits.is_contiguous():
        raise ValueError("target logits must be contiguous [B,k+1,V]")
    B, k1, V = target_logits.shape
    k = k1 - 1
    N = len(draft_logits)
    dev = target_logits.device
    if dev.type != "cuda":
        raise ValueError("device tensors required")
    for d in draft_logits:
        if tuple(d.shape) != (B, k, V) or d.dtype != target_logits.dtype or not d.is_contiguous() or d.device != dev:
            raise ValueError("every draft logit set must be contiguous [B,k,V] of the target's dtype and device")
    if cum_loss is not None and (cum_loss.dtype != torch.float64 or tuple(cum_loss.shape) != (N,) or cum_loss.device != dev):
        raise ValueError("cum_loss must be float64 [N] on the device")
    code = _dtype_code(target_logits)
    if out is None:
        out = EnsembleOutputs(
            loss=torch.empty((N, B, k), dtype=torch.float32, device=dev),
            grad=[torch.empty((B, k, V), dtype=target_logits.dtype, device=dev) for _ in range(N)] if want_grad else None,
            round_loss=torch.empty(N, dtype=torch.float64, device=dev),
            cum_loss=torch.empty(N, dtype=torch.float64, device=dev),
            weights=torch.empty(N, dtype=torch.float32, device=dev),
            status=torch.empty(B, dtype=torch.int32, device=dev) if want_status else None)
    dptr = (ctypes.c_void_p * N)(*[d.data_ptr() for d in draft_logits])
    gptr = (ctypes.c_void_p * N)(*[g.data_ptr() for g in out.grad]) if out.grad is not None else None
    with torch.cuda.device(dev):
        rc = _lib.sd_ensemble_feedback(_ptr(target_logits), dptr, N, float(temperature), float(epsilon), B, k, V, code,
                                       _ptr(cum_loss), _ptr(out.loss), gptr, _ptr(out.round_loss),
                                       _ptr(out.cum_loss), _ptr(out.weights), _ptr(out.status), None, 0,
                                       _stream_ptr(stream))
    if rc != 0:
        raise SdVerifyError(rc, "sd_ensemble_feedback")
    return out


def sd_lmhead_grad(grad_logits: torch.Tensor, hidden: torch.Tensor, *, out: Optional[torch.Tensor] = None,
                   status: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """``sd_lmhead_grad``: dW = g^T X for g [R,V] (or [B,k,V]) and X [R,d], both bfloat16 on the device;
    returns dW [V,d] float32."""
    if grad_logits.dim() == 3:
        grad_logits = grad_logits.reshape(-1, grad_logits.shape[-1])
    if grad_logits.dim() != 2 or hidden.dim() != 2 or grad_logits.shape[0] != hidden.shape[0]:
        raise ValueError("grad_logits must be [R,V] and hidden [R,d]")
    if grad_logits.dtype != torch.bfloat16 or hidden.dtype != torch.bfloat16:
        raise TypeError("both operands must be bfloat16")
    if not grad_logits.is_contiguous() or not hidden.is_contiguous():
        raise ValueError("operands must be contiguous")
    dev = grad_logits.device
    if dev.type != "cuda" or hidden.device != dev:
        raise ValueError("device tensors on one GPU required")
    R, V = grad_logits.shape
    d = hidden.shape[1]
    if out is None:
        out = torch.empty((V, d), dtype=torch.float32, device=dev)
    with torch.cuda.device(dev):
        rc = _lib.sd_lmhead_grad(_ptr(grad_logits), _ptr(hidden), R, V, d, _ptr(out), _ptr(status), _stream_ptr(stream))
    if rc != 0:
        raise SdVerifyError(rc, "sd_lmhead_grad")
    return out


SD_STATIC_SCRATCH_BYTES = 4 * 1024 * 1024


SD_VP_RECORD_BYTES = 48


def sd_vp_workspace_bytes(B: int, k: int, V_shard: int, dtype: int) -> int:
    return int(_lib.sd_vp_workspace_bytes(B, k, V_shard, dtype))


def _vp_shapes(target_shard, draft_shard, draft_tokens):
    if target_shard.dim() != 3 or draft_shard.dim() != 3:
        raise ValueError("shards must be [B,k+1,V_shard] and [B,k,V_shard]")
    B, k1, Vs = target_shard.shape
    k = k1 - 1
    if tuple(draft_shard.shape) != (B, k, Vs) or tuple(draft_tokens.shape) != (B, k):
        raise ValueError("shape mismatch between the shards and the draft tokens")
    if target_shard.dtype != draft_shard.dtype:
        raise TypeError("target and draft shards must have the same dtype")
    for t in (target_shard, draft_shard, draft_tokens):
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError("device-resident contiguous tensors expected")
    return B, k, Vs


def sd_vp_partial(target_shard: torch.Tensor, draft_shard: torch.Tensor, draft_tokens: torch.Tensor,
                  temperature: float, v_offset: int, V_total: int, workspace: torch.Tensor, *,
                  out_records: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Phase 1 of the vocabulary-parallel step: this shard's record of every row, [B*(k+1), 48] bytes."""
    B, k, Vs = _vp_shapes(target_shard, draft_shard, draft_tokens)
    if out_records is None:
        out_records = torch.empty((B * (k + 1), SD_VP_RECORD_BYTES), dtype=torch.uint8, device=target_shard.device)
    rc = _lib.sd_vp_partial(_ptr(target_shard), _ptr(draft_shard), _ptr(draft_tokens), float(temperature), B, k, Vs,
                            int(v_offset), int(V_total), _dtype_code(target_shard), _ptr(out_records), _ptr(workspace),
                            workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    if rc != 0:
        raise SdVerifyError(rc, "sd_vp_partial")
    return out_records


@dataclass
class VpFinishOutputs:
    accept_len: torch.Tensor            # [B] int32, the same on every rank
    loss: Optional[torch.Tensor]        # [B,k] float32, the same on every rank
    grad_shard: Optional[torch.Tensor]  # [B,k,V_shard]
    local_mass: torch.Tensor            # [B,2] float64
    status: torch.Tensor                # [B] int32 view of the status words


def sd_vp_finish(target_shard: torch.Tensor, draft_shard: torch.Tensor, draft_tokens: torch.Tensor,
                 uniforms: torch.Tensor, temperature: float, v_offset: int, V_total: int, all_records: torch.Tensor,
                 n_ranks: int, rank: int, workspace: torch.Tensor, *, want_loss: bool = True, want_grad: bool = True,
                 stream: Optional[torch.cuda.Stream] = None) -> VpFinishOutputs:
    """Phase 2: ``all_records`` is the rank-ordered gather [n_ranks, B*(k+1), 48] of phase 1's records."""
    B, k, Vs = _vp_shapes(target_shard, draft_shard, draft_tokens)
    if all_records.numel() * all_records.element_size() != n_ranks * B * (k + 1) * SD_VP_RECORD_BYTES:
        raise ValueError("all_records must hold n_ranks * B * (k+1) records")
    dev = target_shard.device
    accept_len = torch.empty((B,), dtype=torch.int32, device=dev)
    loss = torch.empty((B, k), dtype=torch.float32, device=dev) if want_loss else None
    grad = torch.empty_like(draft_shard) if want_grad else None
    mass = torch.empty((B, 2), dtype=torch.float64, device=dev)
    status = torch.empty((B,), dtype=torch.int32, device=dev)
    rc = _lib.sd_vp_finish(_ptr(target_shard), _ptr(draft_shard), _ptr(draft_tokens), _ptr(uniforms), float(temperature),
                           B, k, Vs, int(v_offset), int(V_total), _dtype_code(target_shard), _ptr(all_records),
                           int(n_ranks), int(rank), _ptr(accept_len), _ptr(loss), _ptr(grad), _ptr(mass), _ptr(status),
                           _ptr(workspace), workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    if rc != 0:
        raise SdVerifyError(rc, "sd_vp_finish")
    return VpFinishOutputs(accept_len, loss, grad, mass, status)


def sd_vp_draw(target_shard: torch.Tensor, draft_shard: torch.Tensor, draft_tokens: torch.Tensor,
               uniforms: torch.Tensor, temperature: float, v_offset: int, V_total: int, accept_len: torch.Tensor,
               all_masses: torch.Tensor, n_ranks: int, rank: int, status: torch.Tensor, workspace: torch.Tensor, *,
               stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Phase 3: ``all_masses`` is the rank-ordered gather [n_ranks, B, 2] of phase 2's shares.  Returns
    tokens [B,k+1] with -1 where another rank's shard holds the extra token."""
    B, k, Vs = _vp_shapes(target_shard, draft_shard, draft_tokens)
    if all_masses.dtype != torch.float64 or all_masses.numel() != n_ranks * B * 2:
        raise ValueError("all_masses must be float64 [n_ranks, B, 2]")
    tokens = torch.empty((B, k + 1), dtype=torch.int32, device=target_shard.device)
    rc = _lib.sd_vp_draw(_ptr(target_shard), _ptr(draft_shard), _ptr(draft_tokens), _ptr(uniforms), float(temperature),
                         B, k, Vs, int(v_offset), int(V_total), _dtype_code(target_shard), _ptr(accept_len),
                         _ptr(all_masses), int(n_ranks), int(rank), _ptr(tokens), _ptr(status), _ptr(workspace),
                         workspace.numel() * workspace.element_size(), _stream_ptr(stream))
    if rc != 0:
        raise SdVerifyError(rc, "sd_vp_draw")
    return tokens


def sd_verify_feedback_static(target_logits: torch.Tensor, draft_logits: torch.Tensor,
                              draft_tokens: torch.Tensor, uniforms: torch.Tensor, temperature: float, *,
                              out: StepOutputs, stream: Optional[torch.cuda.Stream] = None) -> StepOutputs:
    """``sd_verify_feedback_static``: the step with the scratch that is built into the library.

    For callers that may not allocate device memory: the C entry point allocates nothing, and
    neither does this wrapper, which is why ``out`` (every output tensor the caller wants, made
    beforehand) is required here instead of being created on the fly.  Shapes that need more than
    ``SD_STATIC_SCRATCH_BYTES`` of scratch raise ``SdVerifyError`` (SD_ERR_WORKSPACE).  Calls that
    overlap on the GPU share the one scratch array and must be serialised by the caller.
    """
    B, k, V = _shapes(target_logits, draft_logits, draft_tokens, uniforms)
    dev = target_logits.device
    if dev.type != "cuda":
        raise ValueError("device tensors required")
    code = _dtype_code(target_logits)
    with torch.cuda.device(dev):
        rc = _lib.sd_verify_feedback_static(
            _ptr(target_logits), _ptr(draft_logits), _ptr(draft_tokens), _ptr(uniforms), float(temperature),
            B, k, V, code, _ptr(out.accept_len), _ptr(out.tokens), _ptr(out.loss), _ptr(out.grad_draft),
            _ptr(out.acc_prob), _ptr(out.status), _stream_ptr(stream))
    if rc != 0:
        raise SdVerifyError(rc, "sd_verify_feedback_static")
    return out


def sd_verify_feedback_host(target_logits: torch.Tensor, draft_logits: torch.Tensor,
                            draft_tokens: torch.Tensor, uniforms: torch.Tensor, temperature: float, *,
                            want_loss: bool = True, want_grad: bool = True, want_acc_prob: bool = False,
                            want_status: bool = False, out: Optional[StepOutputs] = None,
                            pin_outputs: bool = True) -> StepOutputs:
    """``sd_verify_feedback_host``: host tensors in, host tensors out, copies inside the call."""
    B, k, V = _shapes(target_logits, draft_logits, draft_tokens, uniforms)
    if target_logits.device.type != "cpu":
        raise ValueError("host tensors required")
    code = _dtype_code(target_logits)
    pin = pin_outputs and torch.cuda.is_available()
    if out is None:
        out = StepOutputs(
            accept_len=torch.empty(B, dtype=torch.int32, pin_memory=pin),
            tokens=torch.empty((B, k + 1), dtype=torch.int32, pin_memory=pin),
            loss=torch.empty((B, k), dtype=torch.float32, pin_memory=pin) if (want_loss or want_grad) else None,
            grad_draft=torch.empty(draft_logits.shape, dtype=draft_logits.dtype, pin_memory=pin) if want_grad else None,
            acc_prob=torch.empty((B, k), dtype=torch.float32, pin_memory=pin) if want_acc_prob else None,
            status=torch.empty(B, dtype=torch.int32, pin_memory=pin) if want_status else None)
    rc = _lib.sd_verify_feedback_host(
        _ptr(target_logits), _ptr(draft_logits), _ptr(draft_tokens), _ptr(uniforms), float(temperature),
        B, k, V, code, _ptr(out.accept_len), _ptr(out.tokens), _ptr(out.loss), _ptr(out.grad_draft),
        _ptr(out.acc_prob), _ptr(out.status))
    if rc != 0:
        raise SdVerifyError(rc, "sd_verify_feedback_host")
    return out
