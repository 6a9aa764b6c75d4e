"""ctypes binding of liba3po.so: same names as the C ABI, argument marshalling only.

Tensors are torch tensors used as typed device (or, for the host entry, pinned host) buffers;
torch does none of the arithmetic.  Every function raises if the compiled library is missing or
a call returns an error code: there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import c_char_p, c_float, c_int, c_int32, c_int64, c_size_t, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "lib", "liba3po.so")

A3PO_F32 = 0
A3PO_BF16 = 1
STATUS_TARGET_OUT_OF_RANGE = 1
STATUS_WAIT_TIMEOUT = 2
STATUS_KEPT_RANGE = 4


class A3poStats(ctypes.Structure):
    _fields_ = [("n_valid", c_int64), ("n_clipped", c_int64), ("iw_max", c_float), ("iw_min", c_float)]


class A3poError(RuntimeError):
    def __init__(self, fn, code, text):
        super().__init__(f"{fn} failed: {text} (code {code})")
        self.code = code


_SIGNATURES = {
    "a3po_status_string": (c_char_p, [c_int]),
    "a3po_version": (c_int, []),
    "a3po_kernel_launch_count": (c_int64, []),
    "a3po_kernel_name": (c_char_p, [c_int]),
    "a3po_profile_enable": (c_int, [c_int]),
    "a3po_profile_read": (c_int, [c_int, c_void_p, c_void_p, c_void_p]),
    "a3po_token_logprobs_workspace_bytes": (c_size_t, [c_int64, c_int, c_int, c_int, c_int]),
    "a3po_token_logprobs_min_workspace_bytes": (c_size_t, [c_int64, c_int, c_int, c_int, c_int]),
    "a3po_loss_workspace_bytes": (c_size_t, [c_int64]),
    "a3po_train_step_stage_bytes": (c_size_t, [c_int64, c_int, c_int]),
    "a3po_host_to_device_bytes": (c_int64, []),
    "a3po_train_step_workspace_bytes": (c_size_t, [c_int64, c_int, c_int, c_int]),
    "a3po_token_logprobs_fwd": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_int, c_int, c_int, c_float,
                                        c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p, c_void_p]),
    "a3po_token_logprobs_bwd": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_int, c_int, c_int,
                                        c_float, c_void_p, c_void_p, c_int, c_void_p, c_size_t, c_void_p, c_void_p]),
    "a3po_loss_fwd": (c_int, [c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_int, c_int32, c_void_p, c_void_p,
                              c_int64, c_float, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]),
    "a3po_loss_fwd_static": (c_int, [c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_int, c_int32, c_void_p, c_void_p,
                                     c_int64, c_float, c_void_p, c_void_p, c_void_p]),
    "a3po_loss_bwd": (c_int, [c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_int, c_int32, c_void_p, c_void_p,
                              c_int64, c_float, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]),
    "a3po_loss_fwd_bwd": (c_int, [c_void_p, c_void_p, c_void_p, c_int, c_void_p, c_int, c_int32, c_void_p, c_void_p,
                                  c_int64, c_float, c_int, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t,
                                  c_void_p]),
    "a3po_decoupled_loss_fwd_bwd": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_float, c_void_p,
                                            c_void_p, c_void_p, c_void_p, c_size_t, c_void_p]),
    "a3po_grpo_workspace_bytes": (c_size_t, [c_int]),
    "a3po_grpo_advantages": (c_int, [c_void_p, c_int, c_int, c_void_p, c_int64, c_float, c_void_p, c_void_p, c_size_t,
                                     c_void_p]),
    "a3po_selftest_wait_timeout": (c_int, [c_void_p, ctypes.c_uint, c_void_p]),
    "a3po_kept_bytes": (c_size_t, [c_int64, c_int]),
    "a3po_token_logprobs_fwd_keep_workspace_bytes": (c_size_t, [c_int64, c_int, c_int]),
    "a3po_token_logprobs_bwd_kept_workspace_bytes": (c_size_t, [c_int64, c_int, c_int]),
    "a3po_token_logprobs_fwd_keep": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_int, c_int, c_float,
                                             c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p, c_size_t,
                                             c_void_p, c_void_p]),
    "a3po_token_logprobs_bwd_kept": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t,
                                             c_int64, c_int, c_int, c_float, c_void_p, c_void_p, c_int, c_void_p,
                                             c_size_t, c_void_p, c_void_p]),
    "a3po_train_step_min_workspace_bytes": (c_size_t, [c_int64, c_int, c_int, c_int]),
    "a3po_train_step": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_int, c_int, c_int,
                                c_int32, c_float, c_float, c_void_p, c_void_p, c_int, c_void_p, c_void_p, c_void_p,
                                c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_size_t, c_void_p,
                                c_void_p]),
    "a3po_mask_count_workspace_bytes": (c_size_t, []),
    "a3po_mask_count": (c_int, [c_void_p, c_int64, c_void_p, c_void_p, c_size_t, c_void_p]),
    "a3po_dp_loss_scale": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "a3po_train_step_host": (c_int, [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int64, c_int, c_int,
                                     c_int, c_int32, c_float, c_float, c_void_p, c_void_p, c_int, c_void_p, c_void_p,
                                     c_size_t, c_void_p, c_size_t, c_void_p, c_void_p, c_void_p, c_void_p]),
}

_lib = None


def exported_symbols():
    """Names every build of the library must export (those declared in include/a3po.h)."""
    return sorted(_SIGNATURES)


def load_library(path: str | None = None):
    """Load liba3po.so once and attach argument types.  Raises if it has not been built."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise RuntimeError(
            f"{p} not found: build it with `python -m paper_2512_06547_b200.build` "
            "(there is no fallback implementation)")
    lib = ctypes.CDLL(p)
    for name, (res, args) in _SIGNATURES.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    if path is None:
        _lib = lib
    return lib


def _check(fn, code):
    if code != 0:
        raise A3poError(fn, code, load_library().a3po_status_string(code).decode())


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return c_void_p(s.cuda_stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return A3PO_F32
    if t.dtype == torch.bfloat16:
        return A3PO_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _want(t, dtype, name, device_type="cuda"):
    if t is None:
        return
    if t.dtype != dtype or not t.is_contiguous() or t.device.type != device_type:
        raise TypeError(f"{name}: expected contiguous {dtype} tensor on {device_type}, got {t.dtype} on {t.device}")


# ------------------------------------------------------------------------------ sizes
def a3po_version() -> int:
    return load_library().a3po_version()


def a3po_kernel_launch_count() -> int:
    return load_library().a3po_kernel_launch_count()


def a3po_profile_enable(on: bool) -> None:
    _check("a3po_profile_enable", load_library().a3po_profile_enable(int(bool(on))))


def a3po_profile_read(max_entries: int = 1 << 16):
    """Returns [(kernel name, milliseconds), ...] for the launches recorded since the last read."""
    lib = load_library()
    ids = (c_int * max_entries)()
    ms = (c_float * max_entries)()
    count = c_int(0)
    _check("a3po_profile_read", lib.a3po_profile_read(max_entries, ids, ms, ctypes.byref(count)))
    return [(lib.a3po_kernel_name(ids[i]).decode(), float(ms[i])) for i in range(count.value)]


def a3po_token_logprobs_workspace_bytes(N, H, V, dt, is_bwd) -> int:
    return load_library().a3po_token_logprobs_workspace_bytes(N, H, V, dt, int(is_bwd))


def a3po_token_logprobs_min_workspace_bytes(N, H, V, dt, is_bwd) -> int:
    return load_library().a3po_token_logprobs_min_workspace_bytes(N, H, V, dt, int(is_bwd))


def a3po_loss_workspace_bytes(N) -> int:
    return load_library().a3po_loss_workspace_bytes(N)


def a3po_train_step_stage_bytes(N, H, dt) -> int:
    return load_library().a3po_train_step_stage_bytes(N, H, dt)


def a3po_host_to_device_bytes() -> int:
    return int(load_library().a3po_host_to_device_bytes())


def a3po_train_step_workspace_bytes(N, H, V, dt) -> int:
    return load_library().a3po_train_step_workspace_bytes(N, H, V, dt)


def new_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """A byte buffer usable as `ws` (torch's CUDA allocations are at least 256-byte aligned)."""
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


# ------------------------------------------------------------------------------ LM head
def a3po_token_logprobs_fwd(hidden, w, targets, logp, lse, ws, *, row_mask=None, entropy=None,
                            inv_temperature=1.0, status=None, stream=None):
    dt = _dtype_code(hidden)
    _want(hidden, hidden.dtype, "hidden"); _want(w, hidden.dtype, "w")
    _want(targets, torch.int32, "targets"); _want(row_mask, torch.uint8, "row_mask")
    _want(logp, torch.float32, "logp"); _want(lse, torch.float32, "lse"); _want(entropy, torch.float32, "entropy")
    _want(status, torch.int32, "status"); _want(ws, torch.uint8, "ws")
    n, h = hidden.shape
    v = w.shape[0]
    if w.shape[1] != h or targets.numel() != n or logp.numel() != n or lse.numel() != n:
        raise ValueError("shape mismatch")
    rc = load_library().a3po_token_logprobs_fwd(_ptr(hidden), _ptr(w), _ptr(targets), _ptr(row_mask), n, h, v, dt,
                                                float(inv_temperature), _ptr(logp), _ptr(lse), _ptr(entropy),
                                                _ptr(ws), ws.numel(), _ptr(status), _stream(stream))
    _check("a3po_token_logprobs_fwd", rc)


def a3po_token_logprobs_bwd(hidden, w, targets, lse, grad_logp, grad_hidden, grad_w, ws, *, accumulate_grad_w=False,
                            inv_temperature=1.0, status=None, stream=None):
    dt = _dtype_code(hidden)
    _want(hidden, hidden.dtype, "hidden"); _want(w, hidden.dtype, "w"); _want(grad_hidden, hidden.dtype, "grad_hidden")
    _want(targets, torch.int32, "targets"); _want(lse, torch.float32, "lse"); _want(grad_logp, torch.float32, "grad_logp")
    _want(grad_w, torch.float32, "grad_w"); _want(status, torch.int32, "status"); _want(ws, torch.uint8, "ws")
    n, h = hidden.shape
    v = w.shape[0]
    if w.shape[1] != h or grad_hidden.shape != hidden.shape or grad_w.shape != w.shape or grad_logp.numel() != n:
        raise ValueError("shape mismatch")
    rc = load_library().a3po_token_logprobs_bwd(_ptr(hidden), _ptr(w), _ptr(targets), _ptr(lse), _ptr(grad_logp), n, h,
                                                v, dt, float(inv_temperature), _ptr(grad_hidden), _ptr(grad_w),
                                                int(bool(accumulate_grad_w)), _ptr(ws), ws.numel(), _ptr(status),
                                                _stream(stream))
    _check("a3po_token_logprobs_bwd", rc)


def a3po_kept_bytes(N, V) -> int:
    return load_library().a3po_kept_bytes(N, V)


def a3po_token_logprobs_fwd_keep_workspace_bytes(N, H, V) -> int:
    return load_library().a3po_token_logprobs_fwd_keep_workspace_bytes(N, H, V)


def a3po_token_logprobs_bwd_kept_workspace_bytes(N, H, V) -> int:
    return load_library().a3po_token_logprobs_bwd_kept_workspace_bytes(N, H, V)


def a3po_token_logprobs_fwd_keep(hidden, w, targets, logp, lse, kept, ws, *, row_mask=None, entropy=None,
                                 inv_temperature=1.0, status=None, stream=None):
    """Forward that also fills `kept` (uint8 buffer of a3po_kept_bytes) for a3po_token_logprobs_bwd_kept."""
    _want(hidden, torch.bfloat16, "hidden"); _want(w, torch.bfloat16, "w")
    _want(targets, torch.int32, "targets"); _want(row_mask, torch.uint8, "row_mask")
    _want(logp, torch.float32, "logp"); _want(lse, torch.float32, "lse"); _want(entropy, torch.float32, "entropy")
    _want(kept, torch.uint8, "kept"); _want(ws, torch.uint8, "ws"); _want(status, torch.int32, "status")
    n, h = hidden.shape
    v = w.shape[0]
    if w.shape[1] != h or targets.numel() != n or logp.numel() != n or lse.numel() != n:
        raise ValueError("shape mismatch")
    rc = load_library().a3po_token_logprobs_fwd_keep(_ptr(hidden), _ptr(w), _ptr(targets), _ptr(row_mask), n, h, v,
                                                     float(inv_temperature), _ptr(logp), _ptr(lse), _ptr(entropy),
                                                     _ptr(kept), kept.numel(), _ptr(ws), ws.numel(), _ptr(status),
                                                     _stream(stream))
    _check("a3po_token_logprobs_fwd_keep", rc)


def a3po_token_logprobs_bwd_kept(hidden, w, targets, lse, grad_logp, kept, grad_hidden, grad_w, ws, *,
                                 accumulate_grad_w=False, inv_temperature=1.0, status=None, stream=None):
    """Backward from what a3po_token_logprobs_fwd_keep kept (no recomputation of the LM head)."""
    _want(hidden, torch.bfloat16, "hidden"); _want(w, torch.bfloat16, "w")
    _want(grad_hidden, torch.bfloat16, "grad_hidden"); _want(targets, torch.int32, "targets")
    _want(lse, torch.float32, "lse"); _want(grad_logp, torch.float32, "grad_logp")
    _want(grad_w, torch.float32, "grad_w"); _want(kept, torch.uint8, "kept"); _want(ws, torch.uint8, "ws")
    _want(status, torch.int32, "status")
    n, h = hidden.shape
    v = w.shape[0]
    if w.shape[1] != h or grad_hidden.shape != hidden.shape or grad_w.shape != w.shape or grad_logp.numel() != n:
        raise ValueError("shape mismatch")
    rc = load_library().a3po_token_logprobs_bwd_kept(_ptr(hidden), _ptr(w), _ptr(targets), _ptr(lse), _ptr(grad_logp),
                                                     _ptr(kept), kept.numel(), n, h, v, float(inv_temperature),
                                                     _ptr(grad_hidden), _ptr(grad_w), int(bool(accumulate_grad_w)),
                                                     _ptr(ws), ws.numel(), _ptr(status), _stream(stream))
    _check("a3po_token_logprobs_bwd_kept", rc)


# ------------------------------------------------------------------------------ loss
def _loss_common(logp, behav_logp, versions, adv, mask, cu_seqlens):
    _want(logp, torch.float32, "logp"); _want(behav_logp, torch.float32, "behav_logp")
    _want(versions, torch.int32, "versions"); _want(adv, torch.float32, "adv"); _want(mask, torch.uint8, "mask")
    _want(cu_seqlens, torch.int32, "cu_seqlens")
    n = logp.numel()
    if behav_logp.numel() != n or adv.numel() != n or mask.numel() != n:
        raise ValueError("shape mismatch")
    per_seq = cu_seqlens is not None
    b = cu_seqlens.numel() - 1 if per_seq else 0
    if per_seq and versions.numel() != b:
        raise ValueError("versions must have one entry per sequence when cu_seqlens is given")
    if not per_seq and versions.numel() != n:
        raise ValueError("versions must have one entry per token")
    return n, int(per_seq), b


def new_stats(device="cuda") -> torch.Tensor:
    """Device storage for one a3po_stats struct (24 bytes)."""
    return torch.zeros(ctypes.sizeof(A3poStats), dtype=torch.uint8, device=device)


def read_stats(stats: torch.Tensor) -> dict:
    raw = bytes(stats.cpu().numpy().tobytes())
    s = A3poStats.from_buffer_copy(raw)
    return dict(n_valid=s.n_valid, n_clipped=s.n_clipped, iw_max=s.iw_max, iw_min=s.iw_min)


def a3po_loss_fwd(logp, behav_logp, versions, current_version, adv, mask, clip_eps, loss, ws, *, stats=None,
                  cu_seqlens=None, stream=None):
    n, per_seq, b = _loss_common(logp, behav_logp, versions, adv, mask, cu_seqlens)
    _want(loss, torch.float32, "loss"); _want(stats, torch.uint8, "stats"); _want(ws, torch.uint8, "ws")
    rc = load_library().a3po_loss_fwd(_ptr(logp), _ptr(behav_logp), _ptr(versions), per_seq, _ptr(cu_seqlens), b,
                                      int(current_version), _ptr(adv), _ptr(mask), n, float(clip_eps), _ptr(loss),
                                      _ptr(stats), _ptr(ws), ws.numel(), _stream(stream))
    _check("a3po_loss_fwd", rc)


LOSS_FWD_STATIC_MAX_TOKENS = 1 << 20


def a3po_loss_fwd_static(logp, behav_logp, versions, current_version, adv, mask, clip_eps, loss, *, stats=None,
                         cu_seqlens=None, stream=None):
    """a3po_loss_fwd for callers that cannot supply a workspace: the scratch is a fixed array inside the
    library (at most LOSS_FWD_STATIC_MAX_TOKENS tokens; calls on one device must not overlap)."""
    n, per_seq, b = _loss_common(logp, behav_logp, versions, adv, mask, cu_seqlens)
    _want(loss, torch.float32, "loss"); _want(stats, torch.uint8, "stats")
    rc = load_library().a3po_loss_fwd_static(_ptr(logp), _ptr(behav_logp), _ptr(versions), per_seq, _ptr(cu_seqlens),
                                             b, int(current_version), _ptr(adv), _ptr(mask), n, float(clip_eps),
                                             _ptr(loss), _ptr(stats), _stream(stream))
    _check("a3po_loss_fwd_static", rc)


def a3po_loss_bwd(logp, behav_logp, versions, current_version, adv, mask, clip_eps, grad_logp, ws, *,
                  detach_prox=True, grad_loss=None, fwd_stats=None, cu_seqlens=None, stream=None):
    n, per_seq, b = _loss_common(logp, behav_logp, versions, adv, mask, cu_seqlens)
    _want(grad_logp, torch.float32, "grad_logp"); _want(grad_loss, torch.float32, "grad_loss")
    _want(fwd_stats, torch.uint8, "fwd_stats"); _want(ws, torch.uint8, "ws")
    rc = load_library().a3po_loss_bwd(_ptr(logp), _ptr(behav_logp), _ptr(versions), per_seq, _ptr(cu_seqlens), b,
                                      int(current_version), _ptr(adv), _ptr(mask), n, float(clip_eps),
                                      int(bool(detach_prox)), _ptr(grad_loss), _ptr(fwd_stats), _ptr(grad_logp),
                                      _ptr(ws), ws.numel(), _stream(stream))
    _check("a3po_loss_bwd", rc)


def a3po_loss_fwd_bwd(logp, behav_logp, versions, current_version, adv, mask, clip_eps, loss, grad_logp, ws, *,
                      detach_prox=True, stats=None, cu_seqlens=None, stream=None):
    n, per_seq, b = _loss_common(logp, behav_logp, versions, adv, mask, cu_seqlens)
    _want(loss, torch.float32, "loss"); _want(grad_logp, torch.float32, "grad_logp")
    _want(stats, torch.uint8, "stats"); _want(ws, torch.uint8, "ws")
    rc = load_library().a3po_loss_fwd_bwd(_ptr(logp), _ptr(behav_logp), _ptr(versions), per_seq, _ptr(cu_seqlens), b,
                                          int(current_version), _ptr(adv), _ptr(mask), n, float(clip_eps),
                                          int(bool(detach_prox)), _ptr(loss), _ptr(stats), _ptr(grad_logp), _ptr(ws),
                                          ws.numel(), _stream(stream))
    _check("a3po_loss_fwd_bwd", rc)


def a3po_decoupled_loss_fwd_bwd(logp, behav_logp, prox_logp, adv, mask, clip_eps, loss, ws, *, grad_logp=None,
                                stats=None, stream=None):
    """Eq. 2 with an explicit proximal log-prob array (the "recompute" baseline; prox = behav gives Eq. 1)."""
    for t, nm in ((logp, "logp"), (behav_logp, "behav_logp"), (prox_logp, "prox_logp"), (adv, "adv"),
                  (loss, "loss"), (grad_logp, "grad_logp")):
        _want(t, torch.float32, nm)
    _want(mask, torch.uint8, "mask"); _want(stats, torch.uint8, "stats"); _want(ws, torch.uint8, "ws")
    n = logp.numel()
    if not (behav_logp.numel() == prox_logp.numel() == adv.numel() == mask.numel() == n):
        raise ValueError("shape mismatch")
    rc = load_library().a3po_decoupled_loss_fwd_bwd(_ptr(logp), _ptr(behav_logp), _ptr(prox_logp), _ptr(adv),
                                                    _ptr(mask), n, float(clip_eps), _ptr(loss), _ptr(stats),
                                                    _ptr(grad_logp), _ptr(ws), ws.numel(), _stream(stream))
    _check("a3po_decoupled_loss_fwd_bwd", rc)


def a3po_grpo_workspace_bytes(B) -> int:
    return load_library().a3po_grpo_workspace_bytes(B)


def a3po_grpo_advantages(rewards, group_size, cu_seqlens, adv, ws, *, norm_eps=1e-6, stream=None):
    """adv[t] = group-normalised reward of the sequence that owns row t."""
    _want(rewards, torch.float32, "rewards"); _want(cu_seqlens, torch.int32, "cu_seqlens")
    _want(adv, torch.float32, "adv"); _want(ws, torch.uint8, "ws")
    b = rewards.numel()
    if cu_seqlens.numel() != b + 1:
        raise ValueError("cu_seqlens must have B + 1 entries")
    rc = load_library().a3po_grpo_advantages(_ptr(rewards), b, int(group_size), _ptr(cu_seqlens), adv.numel(),
                                             float(norm_eps), _ptr(adv), _ptr(ws), ws.numel(), _stream(stream))
    _check("a3po_grpo_advantages", rc)


def a3po_selftest_wait_timeout(status, timeout_ms=50, stream=None):
    """Runs the bounded-wait self-test kernel; afterwards `status` must hold STATUS_WAIT_TIMEOUT."""
    _want(status, torch.int32, "status")
    _check("a3po_selftest_wait_timeout",
           load_library().a3po_selftest_wait_timeout(_ptr(status), int(timeout_ms), _stream(stream)))


# ------------------------------------------------------------------------------ whole step, device inputs
def a3po_train_step_min_workspace_bytes(N, H, V, dt) -> int:
    return load_library().a3po_train_step_min_workspace_bytes(N, H, V, dt)


def a3po_train_step(hidden, w, targets, behav_logp, versions, current_version, adv, mask, clip_eps, logp, lse,
                    grad_logp, loss, grad_hidden, grad_w, ws, *, stats=None, entropy=None, loss_scale=None,
                    accumulate_grad_w=False, inv_temperature=1.0, status=None, stream=None):
    """token_logprobs_fwd -> loss_fwd_bwd -> token_logprobs_bwd in one call; with the recommended workspace the
    backward reuses the softmax kept by the forward instead of recomputing the logits."""
    dt = _dtype_code(hidden)
    _want(hidden, hidden.dtype, "hidden"); _want(w, hidden.dtype, "w"); _want(grad_hidden, hidden.dtype, "grad_hidden")
    _want(targets, torch.int32, "targets"); _want(versions, torch.int32, "versions"); _want(mask, torch.uint8, "mask")
    for t, nm in ((behav_logp, "behav_logp"), (adv, "adv"), (logp, "logp"), (lse, "lse"), (grad_logp, "grad_logp"),
                  (loss, "loss"), (grad_w, "grad_w")):
        _want(t, torch.float32, nm)
    _want(stats, torch.uint8, "stats"); _want(status, torch.int32, "status"); _want(ws, torch.uint8, "ws")
    _want(entropy, torch.float32, "entropy"); _want(loss_scale, torch.float32, "loss_scale")
    n, h = hidden.shape
    v = w.shape[0]
    if w.shape[1] != h or grad_w.shape != w.shape or grad_hidden.shape != hidden.shape:
        raise ValueError("shape mismatch")
    for t in (targets, behav_logp, versions, adv, mask, logp, lse, grad_logp) + ((entropy,) if entropy is not None
                                                                                  else ()):
        if t.numel() != n:
            raise ValueError("per-token arrays must have N entries")
    rc = load_library().a3po_train_step(
        _ptr(hidden), _ptr(targets), _ptr(behav_logp), _ptr(versions), _ptr(adv), _ptr(mask), n, h, v, dt,
        int(current_version), float(clip_eps), float(inv_temperature), _ptr(w), _ptr(grad_w),
        int(bool(accumulate_grad_w)), _ptr(grad_hidden), _ptr(logp), _ptr(lse), _ptr(entropy), _ptr(grad_logp),
        _ptr(loss), _ptr(stats), _ptr(loss_scale), _ptr(ws), ws.numel(), _ptr(status), _stream(stream))
    _check("a3po_train_step", rc)


# ------------------------------------------------------------------------------ data-parallel helpers
def a3po_mask_count_workspace_bytes() -> int:
    return load_library().a3po_mask_count_workspace_bytes()


def a3po_mask_count(mask, count, ws, *, stream=None):
    """count (int64 device tensor, 1 element) = number of non-zero mask bytes."""
    _want(mask, torch.uint8, "mask"); _want(count, torch.int64, "count"); _want(ws, torch.uint8, "ws")
    _check("a3po_mask_count", load_library().a3po_mask_count(_ptr(mask), mask.numel(), _ptr(count), _ptr(ws),
                                                             ws.numel(), _stream(stream)))


def a3po_dp_loss_scale(m_local, m_global, scale, *, loss_local=None, weighted_loss=None, stream=None):
    """scale = M_local / M_global; with loss_local also weighted_loss = scale * loss_local (device scalars)."""
    _want(m_local, torch.int64, "m_local"); _want(m_global, torch.int64, "m_global")
    _want(scale, torch.float32, "scale"); _want(loss_local, torch.float32, "loss_local")
    _want(weighted_loss, torch.float32, "weighted_loss")
    _check("a3po_dp_loss_scale", load_library().a3po_dp_loss_scale(_ptr(m_local), _ptr(m_global), _ptr(loss_local),
                                                                   _ptr(scale), _ptr(weighted_loss), _stream(stream)))


# ------------------------------------------------------------------------------ whole step, host inputs
def a3po_train_step_host(h_hidden, h_targets, h_behav_logp, h_versions, h_adv, h_mask, current_version, clip_eps,
                         d_w, d_grad_w, d_grad_hidden, d_stage, d_ws, h_loss, *, h_stats=None, accumulate_grad_w=False,
                         inv_temperature=1.0, d_status=None, stream=None):
    dt = _dtype_code(h_hidden)
    for t, ty, nm in ((h_hidden, h_hidden.dtype, "h_hidden"), (h_targets, torch.int32, "h_targets"),
                      (h_behav_logp, torch.float32, "h_behav_logp"), (h_versions, torch.int32, "h_versions"),
                      (h_adv, torch.float32, "h_adv"), (h_mask, torch.uint8, "h_mask"),
                      (h_loss, torch.float32, "h_loss"), (h_stats, torch.uint8, "h_stats")):
        _want(t, ty, nm, device_type="cpu")
    _want(d_w, h_hidden.dtype, "d_w"); _want(d_grad_w, torch.float32, "d_grad_w")
    _want(d_grad_hidden, h_hidden.dtype, "d_grad_hidden"); _want(d_stage, torch.uint8, "d_stage")
    _want(d_ws, torch.uint8, "d_ws"); _want(d_status, torch.int32, "d_status")
    n, h = h_hidden.shape
    v = d_w.shape[0]
    rc = load_library().a3po_train_step_host(
        _ptr(h_hidden), _ptr(h_targets), _ptr(h_behav_logp), _ptr(h_versions), _ptr(h_adv), _ptr(h_mask), n, h, v, dt,
        int(current_version), float(clip_eps), float(inv_temperature), _ptr(d_w), _ptr(d_grad_w),
        int(bool(accumulate_grad_w)), _ptr(d_grad_hidden), _ptr(d_stage), d_stage.numel(), _ptr(d_ws), d_ws.numel(),
        _ptr(h_loss), _ptr(h_stats), _ptr(d_status), _stream(stream))
    _check("a3po_train_step_host", rc)
