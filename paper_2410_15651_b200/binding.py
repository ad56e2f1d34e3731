"""ctypes binding of librlhf_ppo.so: argument marshalling only.

Every function has the name and meaning of the C entry point it calls (include/rlhf_ppo.h);
torch supplies device memory and the current stream, nothing else.  There is no fallback: if
the library is missing or a call returns an error status, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "librlhf_ppo.so")

_i64 = ctypes.c_longlong
_int = ctypes.c_int
_f32 = ctypes.c_float
_vp = ctypes.c_void_p
_sz = ctypes.c_size_t

# name -> (restype, argtypes); mirrors include/rlhf_ppo.h
SIGNATURES = {
    "rlhf_status_string": (ctypes.c_char_p, [_int]),
    "rlhf_last_cuda_error": (ctypes.c_char_p, []),
    "rlhf_pad_share": (_int, [_i64, _i64, _int, _int, _vp, _vp]),
    "rlhf_workspace_bytes": (_sz, [_int, _int]),
    "rlhf_workspace_init": (_int, [_vp, _sz, _vp]),
    "rlhf_poll_status": (_int, [_vp, _vp]),
    "rlhf_selftest_bounded_wait": (_int, [_vp, _sz, ctypes.c_ulonglong, _vp]),
    "rlhf_gather_logprobs": (_int, [_vp, _i64, _i64, _vp, _i64, _vp, _int, _int, _int, _vp, _vp, _sz, _vp]),
    "rlhf_gather_logprobs_ex": (_int, [_vp, _int, _i64, _i64, _vp, _i64, _vp, _int, _int, _int, _vp, _vp, _vp, _sz, _vp]),
    "rlhf_experience_ex": (_int, [_vp, _i64, _i64, _vp, _i64, _i64, _int, _vp, _i64, _vp, _vp, _vp, _vp,
                                  _int, _int, _int, _f32, _f32, _f32, _f32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "rlhf_ppo_loss_fwd_bwd_ex": (_int, [_vp, _int, _i64, _i64, _vp, _i64, _vp, _vp, _vp, _vp, _vp, _vp,
                                        _int, _int, _int, _f32, _f32, _f32, _vp, _vp,
                                        _vp, _i64, _i64, _vp, _vp, _vp, _sz, _vp]),
    "rlhf_kl_reward": (_int, [_vp, _vp, _vp, _vp, _int, _int, _f32, _f32, _vp, _vp]),
    "rlhf_gae": (_int, [_vp, _vp, _vp, _int, _int, _f32, _f32, _vp, _vp, _vp]),
    "rlhf_whiten_advantages": (_int, [_vp, _vp, _int, _int, _f32, _vp, _vp, _sz, _vp]),
    "rlhf_ppo_stats": (_int, [_vp, _vp, _vp, _vp, _int, _int, _f32, _vp, _vp, _sz, _vp]),
    "rlhf_experience": (_int, [_vp, _i64, _i64, _vp, _i64, _i64, _vp, _i64, _vp, _vp, _vp, _vp,
                               _int, _int, _int, _f32, _f32, _f32, _f32, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]),
    "rlhf_ppo_loss_fwd_bwd": (_int, [_vp, _i64, _i64, _vp, _i64, _vp, _vp, _vp, _vp, _vp, _vp,
                                     _int, _int, _int, _f32, _f32, _f32, _vp, _vp,
                                     _vp, _i64, _i64, _vp, _vp, _vp, _sz, _vp]),
    "rlhf_ppo_loss_fwd_bwd_noalloc": (_int, [_vp, _i64, _i64, _vp, _i64, _vp, _vp, _vp, _vp, _vp, _vp,
                                             _int, _int, _int, _f32, _f32, _f32, _vp, _vp,
                                             _vp, _i64, _i64, _vp, _vp, _vp, _vp]),
}

NOALLOC_MAX_TOKENS = 65536

_lib = None


class RlhfError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        name = lib().rlhf_status_string(status).decode()
        detail = lib().rlhf_last_cuda_error().decode() if status == 7 else ""
        super().__init__(f"{where}: {name}" + (f" ({detail})" if detail else ""))


def lib() -> ctypes.CDLL:
    """Load the CUDA library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2410_15651_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        handle = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype = res
            fn.argtypes = args
        _lib = handle
    return _lib


def pad_share(n_valid: int, n_padded: int, n_blocks: int, block: int) -> Tuple[int, int]:
    """(start, count) of the padded rows that `block` zero-fills in a loss launch (host-side helper)."""
    start, count = _i64(0), _i64(0)
    _check(lib().rlhf_pad_share(n_valid, n_padded, n_blocks, block, ctypes.byref(start), ctypes.byref(count)),
           "rlhf_pad_share")
    return int(start.value), int(count.value)


def _check(status: int, where: str) -> None:
    if status != 0:
        raise RlhfError(status, where)


def _stream(t: torch.Tensor) -> int:
    return torch.cuda.current_stream(t.device).cuda_stream


def _dev(t: torch.Tensor, dtype, what: str) -> torch.Tensor:
    if not t.is_cuda:
        raise ValueError(f"{what} must be a CUDA tensor (the library has no CPU path)")
    if t.dtype != dtype:
        raise TypeError(f"{what} must be {dtype}, got {t.dtype}")
    return t


def _bt(t: torch.Tensor, B: int, T: int, what: str) -> torch.Tensor:
    _dev(t, torch.float32, what)
    if tuple(t.shape) != (B, T) or not t.is_contiguous():
        raise ValueError(f"{what} must be a contiguous [{B},{T}] tensor")
    return t


DTYPES = {torch.bfloat16: 0, torch.float16: 1}        # rlhf_dtype_t


def _logits(t: torch.Tensor, what: str) -> Tuple[int, int, int, int, int]:
    if not t.is_cuda:
        raise ValueError(f"{what} must be a CUDA tensor (the library has no CPU path)")
    if t.dtype not in DTYPES:
        raise TypeError(f"{what} must be bfloat16 or float16, got {t.dtype}")
    if t.dim() != 3 or (t.shape[2] > 1 and t.stride(2) != 1):
        raise ValueError(f"{what} must be [B,T,V] with a contiguous vocabulary axis")
    return t.shape[0], t.shape[1], t.shape[2], t.stride(0), t.stride(1)


def _ids(t: torch.Tensor, B: int, T: int) -> int:
    _dev(t, torch.int64, "ids")
    if tuple(t.shape) != (B, T) or (T > 1 and t.stride(1) != 1):
        raise ValueError("ids must be [B,T] with a contiguous time axis")
    return t.stride(0)


def _lengths(t: torch.Tensor, B: int) -> torch.Tensor:
    _dev(t, torch.int32, "lengths")
    if tuple(t.shape) != (B,) or not t.is_contiguous():
        raise ValueError("lengths must be a contiguous int32 [B] tensor")
    return t


def workspace_bytes(B: int, T: int) -> int:
    return int(lib().rlhf_workspace_bytes(B, T))


def workspace(B: int, T: int, device) -> torch.Tensor:
    """Allocate (through torch) and initialise a workspace for batches of up to B x T tokens."""
    ws = torch.empty(workspace_bytes(B, T), dtype=torch.uint8, device=device)
    _check(lib().rlhf_workspace_init(ws.data_ptr(), ws.numel(), _stream(ws)), "rlhf_workspace_init")
    return ws


def poll_status(ws: torch.Tensor) -> int:
    """Synchronise and return (then clear) the device-detected status flags."""
    return int(lib().rlhf_poll_status(ws.data_ptr(), _stream(ws)))


def selftest_bounded_wait(ws: torch.Tensor, limit_ns: int) -> None:
    """Launch the kernel whose only wait can never be satisfied; poll_status(ws) then reports the timeout flag."""
    _check(lib().rlhf_selftest_bounded_wait(ws.data_ptr(), ws.numel(), int(limit_ns), _stream(ws)),
           "rlhf_selftest_bounded_wait")


def status_string(status: int) -> str:
    return lib().rlhf_status_string(int(status)).decode()


def gather_logprobs(logits: torch.Tensor, ids: torch.Tensor, lengths: torch.Tensor,
                    ws: torch.Tensor, out: Optional[torch.Tensor] = None,
                    out_entropy: Optional[torch.Tensor] = None) -> torch.Tensor:
    """rlhf_gather_logprobs for bf16 logits without an entropy output, else rlhf_gather_logprobs_ex."""
    B, T, V, sb, st = _logits(logits, "logits")
    isb = _ids(ids, B, T)
    _lengths(lengths, B)
    if out is None:
        out = torch.empty((B, T), dtype=torch.float32, device=logits.device)
    _bt(out, B, T, "out")
    if logits.dtype == torch.bfloat16 and out_entropy is None:
        _check(lib().rlhf_gather_logprobs(logits.data_ptr(), sb, st, ids.data_ptr(), isb, lengths.data_ptr(),
                                          B, T, V, out.data_ptr(), ws.data_ptr(), ws.numel(), _stream(logits)),
               "rlhf_gather_logprobs")
        return out
    ent_ptr = _bt(out_entropy, B, T, "out_entropy").data_ptr() if out_entropy is not None else None
    _check(lib().rlhf_gather_logprobs_ex(logits.data_ptr(), DTYPES[logits.dtype], sb, st, ids.data_ptr(), isb,
                                         lengths.data_ptr(), B, T, V, out.data_ptr(), ent_ptr,
                                         ws.data_ptr(), ws.numel(), _stream(logits)), "rlhf_gather_logprobs_ex")
    return out


def kl_reward(lp_old: torch.Tensor, lp_ref: torch.Tensor, score: torch.Tensor, lengths: torch.Tensor,
              beta_kl: float, reward_clip: float, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    B, T = lp_old.shape
    _bt(lp_old, B, T, "lp_old")
    _bt(lp_ref, B, T, "lp_ref")
    _dev(score, torch.float32, "score")
    if tuple(score.shape) != (B,) or not score.is_contiguous():
        raise ValueError("score must be a contiguous [B] tensor")
    _lengths(lengths, B)
    if out is None:
        out = torch.empty_like(lp_old)
    _bt(out, B, T, "out")
    _check(lib().rlhf_kl_reward(lp_old.data_ptr(), lp_ref.data_ptr(), score.data_ptr(), lengths.data_ptr(),
                                B, T, beta_kl, reward_clip, out.data_ptr(), _stream(lp_old)),
           "rlhf_kl_reward")
    return out


def gae(rewards: torch.Tensor, values_old: torch.Tensor, lengths: torch.Tensor, gamma: float, lam: float,
        out_adv: Optional[torch.Tensor] = None, out_returns: Optional[torch.Tensor] = None):
    B, T = rewards.shape
    _bt(rewards, B, T, "rewards")
    _bt(values_old, B, T, "values_old")
    _lengths(lengths, B)
    if out_adv is None:
        out_adv = torch.empty_like(rewards)
    if out_returns is None:
        out_returns = torch.empty_like(rewards)
    _bt(out_adv, B, T, "out_adv")
    _bt(out_returns, B, T, "out_returns")
    _check(lib().rlhf_gae(rewards.data_ptr(), values_old.data_ptr(), lengths.data_ptr(), B, T, gamma, lam,
                          out_adv.data_ptr(), out_returns.data_ptr(), _stream(rewards)), "rlhf_gae")
    return out_adv, out_returns


def whiten_advantages(adv: torch.Tensor, lengths: torch.Tensor, eps: float, ws: torch.Tensor,
                      out: Optional[torch.Tensor] = None) -> torch.Tensor:
    B, T = adv.shape
    _bt(adv, B, T, "adv")
    _lengths(lengths, B)
    if out is None:
        out = torch.empty_like(adv)
    _bt(out, B, T, "out")
    _check(lib().rlhf_whiten_advantages(adv.data_ptr(), lengths.data_ptr(), B, T, eps, out.data_ptr(),
                                        ws.data_ptr(), ws.numel(), _stream(adv)), "rlhf_whiten_advantages")
    return out


def ppo_stats(lp_new: torch.Tensor, lp_old: torch.Tensor, adv: torch.Tensor, lengths: torch.Tensor,
              clip_eps: float, ws: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """[approx_kl, clip_frac] of the policy step, as a device tensor of two floats."""
    B, T = lp_new.shape
    for name, t in (("lp_new", lp_new), ("lp_old", lp_old), ("adv", adv)):
        _bt(t, B, T, name)
    _lengths(lengths, B)
    if out is None:
        out = torch.empty(2, dtype=torch.float32, device=lp_new.device)
    _dev(out, torch.float32, "out")
    _check(lib().rlhf_ppo_stats(lp_new.data_ptr(), lp_old.data_ptr(), adv.data_ptr(), lengths.data_ptr(), B, T,
                                clip_eps, out.data_ptr(), ws.data_ptr(), ws.numel(), _stream(lp_new)),
           "rlhf_ppo_stats")
    return out


class Experience:
    """Buffers written by experience(); reusable from call to call."""

    def __init__(self, B: int, T: int, device):
        f = lambda: torch.empty((B, T), dtype=torch.float32, device=device)
        self.lp_actor, self.lp_ref, self.rewards, self.adv, self.returns = f(), f(), f(), f(), f()


def experience(actor_logits: torch.Tensor, ref_logits: torch.Tensor, ids: torch.Tensor, lengths: torch.Tensor,
               score: torch.Tensor, values_old: torch.Tensor, beta_kl: float, reward_clip: float,
               gamma: float, lam: float, ws: torch.Tensor, out: Optional[Experience] = None,
               lp_old: Optional[torch.Tensor] = None, out_entropy: Optional[torch.Tensor] = None) -> Experience:
    """rlhf_experience for bf16 logits without an entropy output, else rlhf_experience_ex."""
    B, T, V, asb, ast = _logits(actor_logits, "actor_logits")
    rB, rT, rV, rsb, rst = _logits(ref_logits, "ref_logits")
    if (rB, rT, rV) != (B, T, V):
        raise ValueError("actor and reference logits must have the same shape")
    isb = _ids(ids, B, T)
    _lengths(lengths, B)
    _dev(score, torch.float32, "score")
    if tuple(score.shape) != (B,) or not score.is_contiguous():
        raise ValueError("score must be a contiguous [B] tensor")
    _bt(values_old, B, T, "values_old")
    if out is None:
        out = Experience(B, T, actor_logits.device)
    for name in ("lp_actor", "lp_ref", "rewards", "adv", "returns"):
        _bt(getattr(out, name), B, T, "out." + name)
    lp_old_ptr = _bt(lp_old, B, T, "lp_old").data_ptr() if lp_old is not None else None
    if actor_logits.dtype != ref_logits.dtype:
        raise TypeError("actor and reference logits must have the same element type")
    if actor_logits.dtype != torch.bfloat16 or out_entropy is not None:
        ent_ptr = _bt(out_entropy, B, T, "out_entropy").data_ptr() if out_entropy is not None else None
        _check(lib().rlhf_experience_ex(
            actor_logits.data_ptr(), asb, ast, ref_logits.data_ptr(), rsb, rst, DTYPES[actor_logits.dtype],
            ids.data_ptr(), isb, lengths.data_ptr(), score.data_ptr(), values_old.data_ptr(), lp_old_ptr, B, T, V,
            beta_kl, reward_clip, gamma, lam, out.lp_actor.data_ptr(), out.lp_ref.data_ptr(),
            out.rewards.data_ptr(), out.adv.data_ptr(), out.returns.data_ptr(), ent_ptr,
            ws.data_ptr(), ws.numel(), _stream(actor_logits)), "rlhf_experience_ex")
        return out
    _check(lib().rlhf_experience(
        actor_logits.data_ptr(), asb, ast, ref_logits.data_ptr(), rsb, rst, ids.data_ptr(), isb,
        lengths.data_ptr(), score.data_ptr(), values_old.data_ptr(), lp_old_ptr, B, T, V,
        beta_kl, reward_clip, gamma, lam, out.lp_actor.data_ptr(), out.lp_ref.data_ptr(),
        out.rewards.data_ptr(), out.adv.data_ptr(), out.returns.data_ptr(),
        ws.data_ptr(), ws.numel(), _stream(actor_logits)), "rlhf_experience")
    return out


class PPOOutputs:
    """Buffers written by ppo_loss_fwd_bwd; reusable from call to call."""

    def __init__(self, logits: torch.Tensor, in_place: bool = False, want_lp_new: bool = True):
        B, T = logits.shape[0], logits.shape[1]
        dev = logits.device
        self.loss = torch.empty(2, dtype=torch.float32, device=dev)       # [loss_pg, loss_vf]
        self.dlogits = logits if in_place else torch.empty(logits.shape, dtype=logits.dtype, device=dev)
        self.dvalues = torch.empty((B, T), dtype=torch.float32, device=dev)
        self.lp_new = torch.empty((B, T), dtype=torch.float32, device=dev) if want_lp_new else None


def ppo_loss_fwd_bwd(logits: torch.Tensor, ids: torch.Tensor, lengths: torch.Tensor,
                     lp_old: torch.Tensor, adv: torch.Tensor, values_new: torch.Tensor,
                     values_old: torch.Tensor, returns: torch.Tensor,
                     clip_eps: float, value_clip: float, grad_scale: float,
                     ws: torch.Tensor, out: Optional[PPOOutputs] = None) -> PPOOutputs:
    B, T, V, sb, st = _logits(logits, "logits")
    isb = _ids(ids, B, T)
    _lengths(lengths, B)
    for name, t in (("lp_old", lp_old), ("adv", adv), ("values_new", values_new),
                    ("values_old", values_old), ("returns", returns)):
        _bt(t, B, T, name)
    if out is None:
        out = PPOOutputs(logits)
    dB, dT, dV, dsb, dst = _logits(out.dlogits, "out.dlogits")
    if (dB, dT, dV) != (B, T, V):
        raise ValueError("out.dlogits must have the shape of logits")
    _bt(out.dvalues, B, T, "out.dvalues")
    lp_new_ptr = None
    if out.lp_new is not None:
        lp_new_ptr = _bt(out.lp_new, B, T, "out.lp_new").data_ptr()
    loss = _dev(out.loss, torch.float32, "out.loss")
    if out.dlogits.dtype != logits.dtype:
        raise TypeError("out.dlogits must have the element type of logits")
    if logits.dtype != torch.bfloat16:
        _check(lib().rlhf_ppo_loss_fwd_bwd_ex(
            logits.data_ptr(), DTYPES[logits.dtype], sb, st, ids.data_ptr(), isb, lengths.data_ptr(),
            lp_old.data_ptr(), adv.data_ptr(), values_new.data_ptr(), values_old.data_ptr(), returns.data_ptr(),
            B, T, V, clip_eps, value_clip, grad_scale,
            loss.data_ptr(), loss.data_ptr() + 4,
            out.dlogits.data_ptr(), dsb, dst, out.dvalues.data_ptr(), lp_new_ptr,
            ws.data_ptr(), ws.numel(), _stream(logits)), "rlhf_ppo_loss_fwd_bwd_ex")
        return out
    _check(lib().rlhf_ppo_loss_fwd_bwd(
        logits.data_ptr(), sb, st, ids.data_ptr(), isb, lengths.data_ptr(),
        lp_old.data_ptr(), adv.data_ptr(), values_new.data_ptr(), values_old.data_ptr(), returns.data_ptr(),
        B, T, V, clip_eps, value_clip, grad_scale,
        loss.data_ptr(), loss.data_ptr() + 4,
        out.dlogits.data_ptr(), dsb, dst, out.dvalues.data_ptr(), lp_new_ptr,
        ws.data_ptr(), ws.numel(), _stream(logits)), "rlhf_ppo_loss_fwd_bwd")
    return out


def ppo_loss_fwd_bwd_noalloc(logits: torch.Tensor, ids: torch.Tensor, lengths: torch.Tensor,
                             lp_old: torch.Tensor, adv: torch.Tensor, values_new: torch.Tensor,
                             values_old: torch.Tensor, returns: torch.Tensor,
                             clip_eps: float, value_clip: float, grad_scale: float,
                             out: PPOOutputs, device_status: Optional[torch.Tensor] = None) -> PPOOutputs:
    """rlhf_ppo_loss_fwd_bwd_noalloc: the same computation with no workspace argument, for callers
    that cannot allocate scratch memory (at most NOALLOC_MAX_TOKENS tokens; calls on one device must
    not overlap).  `out` must be given (this wrapper allocates nothing either); `device_status`,
    if given, is an int32 CUDA tensor of one element that receives the device-detected flags."""
    B, T, V, sb, st = _logits(logits, "logits")
    if logits.dtype != torch.bfloat16 or out.dlogits.dtype != torch.bfloat16:
        raise TypeError("rlhf_ppo_loss_fwd_bwd_noalloc takes bf16 logits")
    isb = _ids(ids, B, T)
    _lengths(lengths, B)
    for name, t in (("lp_old", lp_old), ("adv", adv), ("values_new", values_new),
                    ("values_old", values_old), ("returns", returns)):
        _bt(t, B, T, name)
    dB, dT, dV, dsb, dst = _logits(out.dlogits, "out.dlogits")
    if (dB, dT, dV) != (B, T, V):
        raise ValueError("out.dlogits must have the shape of logits")
    _bt(out.dvalues, B, T, "out.dvalues")
    lp_new_ptr = None
    if out.lp_new is not None:
        lp_new_ptr = _bt(out.lp_new, B, T, "out.lp_new").data_ptr()
    loss = _dev(out.loss, torch.float32, "out.loss")
    st_ptr = None
    if device_status is not None:
        st_ptr = _dev(device_status, torch.int32, "device_status").data_ptr()
    _check(lib().rlhf_ppo_loss_fwd_bwd_noalloc(
        logits.data_ptr(), sb, st, ids.data_ptr(), isb, lengths.data_ptr(),
        lp_old.data_ptr(), adv.data_ptr(), values_new.data_ptr(), values_old.data_ptr(), returns.data_ptr(),
        B, T, V, clip_eps, value_clip, grad_scale,
        loss.data_ptr(), loss.data_ptr() + 4,
        out.dlogits.data_ptr(), dsb, dst, out.dvalues.data_ptr(), lp_new_ptr,
        st_ptr, _stream(logits)), "rlhf_ppo_loss_fwd_bwd_noalloc")
    return out
