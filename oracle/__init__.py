"""float64 CPU oracle for the token-level PPO math (test infrastructure only).

This package wraps ``rlhf_oracle.c`` (plain C, float64, OpenMP over rows) with numpy
arguments.  It is what the CUDA library is checked against and what the CPU-baseline leg of the
benchmark times.  It imports nothing from the CUDA package and the CUDA package imports nothing
from here; the product path never calls it.

The paper (Section 2.1) names the quantities -- actor and reference log-probabilities, the
reward kept close to the reference, returns estimated with the critic, the actor trained to
raise reward while limiting policy deviation -- and prints no formula.  The functions are the
textbook definitions; the readings of every open point are listed at the top of
``rlhf_oracle.c``.

Whole-path parity against values printed by the paper: parity unpinned (the paper prints none).
Each function is pinned instead by closed forms, invariants, brute force, finite differences and
float64 library routines in ``tests/test_oracle_*.py``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rlhf_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

_i64 = ctypes.c_longlong
_dbl = ctypes.c_double
_vp = ctypes.c_void_p


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, no fast-math) if the library is missing or stale."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".{os.getpid()}.tmp"
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_set_num_threads.argtypes = [ctypes.c_int]
        lib.oracle_round_bf16.restype = _dbl
        lib.oracle_round_bf16.argtypes = [_dbl]
        lib.oracle_row_lse_f64.restype = _dbl
        lib.oracle_row_lse_f64.argtypes = [_vp, _i64]
        lib.oracle_gather_logprobs.restype = ctypes.c_int
        lib.oracle_gather_logprobs.argtypes = [_vp, ctypes.c_int, _i64, _i64, _vp, _i64, _vp,
                                               ctypes.c_int, ctypes.c_int, _i64, _vp]
        lib.oracle_kl_reward.restype = None
        lib.oracle_kl_reward.argtypes = [_vp, _vp, _vp, _vp, ctypes.c_int, ctypes.c_int,
                                         _dbl, _dbl, _vp]
        lib.oracle_gae.restype = None
        lib.oracle_gae.argtypes = [_vp, _vp, _vp, ctypes.c_int, ctypes.c_int, _dbl, _dbl, _vp, _vp]
        lib.oracle_ppo_loss.restype = None
        lib.oracle_ppo_loss.argtypes = [_vp] * 7 + [ctypes.c_int, ctypes.c_int, _dbl, _dbl, _dbl,
                                                    _vp, _vp, _vp, _vp]
        lib.oracle_f16_to_double.restype = _dbl
        lib.oracle_f16_to_double.argtypes = [ctypes.c_uint16]
        lib.oracle_round_f16.restype = _dbl
        lib.oracle_round_f16.argtypes = [_dbl]
        lib.oracle_token_entropy.restype = None
        lib.oracle_token_entropy.argtypes = [_vp, ctypes.c_int, _i64, _i64, _vp, ctypes.c_int, ctypes.c_int,
                                             _i64, _vp]
        lib.oracle_ppo_stats.restype = None
        lib.oracle_ppo_stats.argtypes = [_vp, _vp, _vp, _vp, ctypes.c_int, ctypes.c_int, _dbl, _vp, _vp]
        lib.oracle_whiten.restype = None
        lib.oracle_whiten.argtypes = [_vp, _vp, ctypes.c_int, ctypes.c_int, _dbl, _vp]
        lib.oracle_dlogits_rows.restype = None
        lib.oracle_dlogits_rows.argtypes = [_vp, ctypes.c_int, _i64, _i64, _vp, _i64, _vp,
                                            ctypes.c_int, ctypes.c_int, _i64, _vp, _vp, _i64, _vp]
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    _load().oracle_set_num_threads(int(n))


def _p(a: np.ndarray):
    return a.ctypes.data_as(_vp)


def _f64(a, shape=None) -> np.ndarray:
    out = np.ascontiguousarray(np.asarray(a, dtype=np.float64))
    if shape is not None:
        assert out.shape == tuple(shape), (out.shape, shape)
    return out


def _logits_view(logits: np.ndarray):
    """Return (element type code, stride_b, stride_t) for a [B,T,V] array whose last axis is contiguous; the
    first two axes may be strided (a view of a longer tensor).  uint16 = bf16 bit patterns (code 1),
    float16 = IEEE binary16 (code 2, its bit patterns are passed), float64 (code 0)."""
    assert logits.ndim == 3
    if logits.dtype == np.uint16:
        is_bf16 = 1
    elif logits.dtype == np.float16:
        is_bf16 = 2
    elif logits.dtype == np.float64:
        is_bf16 = 0
    else:
        raise TypeError("logits must be uint16 (bf16 bit patterns), float16 or float64")
    item = logits.dtype.itemsize
    if logits.shape[2] > 1 and logits.strides[2] != item:
        raise ValueError("vocabulary axis must be contiguous")
    assert logits.strides[0] % item == 0 and logits.strides[1] % item == 0
    return is_bf16, logits.strides[0] // item, logits.strides[1] // item


def _ids_view(ids: np.ndarray):
    assert ids.ndim == 2 and ids.dtype == np.int64
    if ids.shape[1] > 1 and ids.strides[1] != 8:
        raise ValueError("ids time axis must be contiguous")
    return ids.strides[0] // 8


def _lengths(lengths, B) -> np.ndarray:
    out = np.ascontiguousarray(np.asarray(lengths, dtype=np.int32))
    assert out.shape == (B,)
    return out


def round_bf16(x) -> np.ndarray:
    """Round float64 values to the nearest bf16 (ties to even); returned as float64."""
    lib = _load()
    x = np.asarray(x, dtype=np.float64)
    return np.vectorize(lambda v: lib.oracle_round_bf16(float(v)), otypes=[np.float64])(x)


def bf16_ulp(x) -> np.ndarray:
    """Spacing of bf16 numbers at |x|: 2^(floor(log2|x|) - 7), with the subnormal floor 2^-133."""
    x = np.abs(np.asarray(x, dtype=np.float64))
    with np.errstate(divide="ignore"):
        lg = np.floor(np.log2(np.where(x > 0, x, 1.0)))
    lg = np.maximum(lg, -126.0)
    return np.where(x > 0, np.exp2(lg - 7.0), 2.0 ** -133)


def f16_to_double(bits) -> np.ndarray:
    """Exact widening of IEEE binary16 bit patterns (uint16) to float64."""
    lib = _load()
    bits = np.asarray(bits, dtype=np.uint16)
    return np.vectorize(lambda h: lib.oracle_f16_to_double(int(h)), otypes=[np.float64])(bits)


def round_f16(x) -> np.ndarray:
    """Round float64 values to the nearest binary16 (ties to even); returned as float64."""
    lib = _load()
    x = np.asarray(x, dtype=np.float64)
    return np.vectorize(lambda v: lib.oracle_round_f16(float(v)), otypes=[np.float64])(x)


def f16_ulp(x) -> np.ndarray:
    """Spacing of binary16 numbers at |x|: 2^(floor(log2|x|) - 10), with the subnormal floor 2^-24."""
    x = np.abs(np.asarray(x, dtype=np.float64))
    with np.errstate(divide="ignore"):
        lg = np.floor(np.log2(np.where(x > 0, x, 1.0)))
    lg = np.maximum(lg, -14.0)
    return np.where(x > 0, np.exp2(lg - 10.0), 2.0 ** -24)


def row_lse(z) -> float:
    z = _f64(z)
    return float(_load().oracle_row_lse_f64(_p(z), z.shape[0]))


def gather_logprobs(logits: np.ndarray, ids: np.ndarray, lengths) -> np.ndarray:
    """Step 1.  logits [B,T,V] (uint16 bf16 bits, or float64), ids [B,T] int64, lengths [B].
    Returns float64 [B,T]: log-softmax at the generated token for t < len, 0 elsewhere."""
    B, T, V = logits.shape
    is_bf16, sb, st = _logits_view(logits)
    assert ids.shape == (B, T)
    isb = _ids_view(ids)
    lengths = _lengths(lengths, B)
    out = np.empty((B, T), dtype=np.float64)
    bad = _load().oracle_gather_logprobs(_p(logits), is_bf16, sb, st, _p(ids), isb, _p(lengths),
                                         B, T, V, _p(out))
    if bad:
        raise ValueError("token id or length out of range")
    return out


def kl_reward(lp_old, lp_ref, score, lengths, beta: float, reward_clip: float) -> np.ndarray:
    """Step 2.  Per-token reward: -beta*(lp_old - lp_ref), plus the clipped sequence score at the
    last valid token."""
    lp_old = _f64(lp_old)
    B, T = lp_old.shape
    lp_ref = _f64(lp_ref, (B, T))
    score = _f64(score, (B,))
    lengths = _lengths(lengths, B)
    out = np.empty((B, T), dtype=np.float64)
    _load().oracle_kl_reward(_p(lp_old), _p(lp_ref), _p(score), _p(lengths), B, T,
                             float(beta), float(reward_clip), _p(out))
    return out


def gae(rewards, values, lengths, gamma: float, lam: float):
    """Step 3.  Returns (advantages, returns), float64 [B,T]."""
    rewards = _f64(rewards)
    B, T = rewards.shape
    values = _f64(values, (B, T))
    lengths = _lengths(lengths, B)
    adv = np.empty((B, T), dtype=np.float64)
    ret = np.empty((B, T), dtype=np.float64)
    _load().oracle_gae(_p(rewards), _p(values), _p(lengths), B, T, float(gamma), float(lam),
                       _p(adv), _p(ret))
    return adv, ret


@dataclass
class PPOLoss:
    loss_pg: float
    loss_vf: float
    lp_new: np.ndarray      # [B,T] log-prob of the generated token under the current logits
    g: np.ndarray           # [B,T] d(grad_scale*loss_pg)/d lp_new
    dvalues: np.ndarray     # [B,T] d(grad_scale*loss_vf)/d values_new


def ppo_loss_from_logprobs(lp_new, lp_old, adv, values_new, values_old, returns, lengths,
                           clip_eps: float, value_clip: float, grad_scale: float = 1.0) -> PPOLoss:
    """Step 4 without the vocabulary axis: losses and the per-token gradient factors."""
    lp_new = _f64(lp_new)
    B, T = lp_new.shape
    arrs = [_f64(a, (B, T)) for a in (lp_old, adv, values_new, values_old, returns)]
    lengths = _lengths(lengths, B)
    g = np.empty((B, T), dtype=np.float64)
    dv = np.empty((B, T), dtype=np.float64)
    l_pg = _dbl(0.0)
    l_vf = _dbl(0.0)
    _load().oracle_ppo_loss(_p(lp_new), *[_p(a) for a in arrs], _p(lengths), B, T,
                            float(clip_eps), float(value_clip), float(grad_scale),
                            ctypes.byref(l_pg), ctypes.byref(l_vf), _p(g), _p(dv))
    return PPOLoss(l_pg.value, l_vf.value, lp_new, g, dv)


def ppo_loss(logits, ids, lengths, lp_old, adv, values_new, values_old, returns,
             clip_eps: float, value_clip: float, grad_scale: float = 1.0) -> PPOLoss:
    """Step 4: new log-probs from the current logits (as step 1), then the clipped losses."""
    lp_new = gather_logprobs(logits, ids, lengths)
    return ppo_loss_from_logprobs(lp_new, lp_old, adv, values_new, values_old, returns, lengths,
                                  clip_eps, value_clip, grad_scale)


def dlogits_rows(logits, ids, lengths, g, rows) -> np.ndarray:
    """Gradient of grad_scale*loss_pg with respect to the logits of the listed rows (flat index
    b*T+t): g*(onehot(y) - softmax(z)), float64 [len(rows), V]."""
    B, T, V = logits.shape
    is_bf16, sb, st = _logits_view(logits)
    isb = _ids_view(ids)
    lengths = _lengths(lengths, B)
    g = _f64(g, (B, T))
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    assert rows.ndim == 1 and (rows.size == 0 or (rows.min() >= 0 and rows.max() < B * T))
    out = np.empty((rows.size, V), dtype=np.float64)
    _load().oracle_dlogits_rows(_p(logits), is_bf16, sb, st, _p(ids), isb, _p(lengths),
                                B, T, V, _p(g), _p(rows), rows.size, _p(out))
    return out


def token_entropy(logits: np.ndarray, lengths) -> np.ndarray:
    """Entropy (nats) of the softmax of every valid row, float64 [B,T]; 0 at padded positions."""
    B, T, V = logits.shape
    dtype, sb, st = _logits_view(logits)
    lengths = _lengths(lengths, B)
    out = np.empty((B, T), dtype=np.float64)
    _load().oracle_token_entropy(_p(logits), dtype, sb, st, _p(lengths), B, T, V, _p(out))
    return out


def ppo_stats(lp_new, lp_old, adv, lengths, clip_eps: float):
    """(approx_kl, clip_frac) over the valid tokens: mean of rho - 1 - log rho, and the share of tokens
    whose gradient the clip switches off."""
    lp_new = _f64(lp_new)
    B, T = lp_new.shape
    lp_old, adv = _f64(lp_old, (B, T)), _f64(adv, (B, T))
    lengths = _lengths(lengths, B)
    kl, cf = _dbl(0.0), _dbl(0.0)
    _load().oracle_ppo_stats(_p(lp_new), _p(lp_old), _p(adv), _p(lengths), B, T, float(clip_eps),
                             ctypes.byref(kl), ctypes.byref(cf))
    return kl.value, cf.value


def whiten(adv, lengths, eps: float = 1e-8) -> np.ndarray:
    """Advantages whitened over the valid tokens of the batch: (A - mean) / sqrt(var + eps), population
    variance; 0 at padded positions."""
    adv = _f64(adv)
    B, T = adv.shape
    lengths = _lengths(lengths, B)
    out = np.empty((B, T), dtype=np.float64)
    _load().oracle_whiten(_p(adv), _p(lengths), B, T, float(eps), _p(out))
    return out
