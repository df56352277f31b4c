"""CPU oracle of the IMPACT learner loss and circular buffer (test infrastructure only).

Thin ctypes marshalling around `impact_oracle.c`, which holds all the arithmetic.
Nothing in the product path may import this package; only the tests, the smoke check
and the benchmark's CPU-baseline leg do.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "impact_oracle.c")
_LIB = os.path.join(_HERE, "libimpact_oracle.so")
_lib = None

LOSS_TERM_NAMES = ("total", "policy", "value", "entropy", "kl", "clip_frac", "rho_trunc_frac", "mean_ratio")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, no fast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Coef(ctypes.Structure):
    _fields_ = [("vf_coef", ctypes.c_double), ("ent_coef", ctypes.c_double),
                ("kl_coef", ctypes.c_double), ("lam", ctypes.c_double),
                ("rho_tw", ctypes.c_double), ("is_source", ctypes.c_int32),
                ("ratio_mode", ctypes.c_int32), ("objective", ctypes.c_int32)]


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.oracle_ring_create.restype = ctypes.c_void_p
        lib.oracle_ring_create.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_uint64]
        lib.oracle_ring_destroy.argtypes = [ctypes.c_void_p]
        lib.oracle_ring_push.argtypes = [ctypes.c_void_p, ctypes.POINTER(ctypes.c_int32)]
        lib.oracle_ring_sample.argtypes = [ctypes.c_void_p, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32)]
        lib.oracle_ring_live.argtypes = [ctypes.c_void_p]
        lib.oracle_draw_u64.restype = ctypes.c_uint64
        lib.oracle_draw_u64.argtypes = [ctypes.c_uint64, ctypes.c_uint64]
        _lib = lib
    return _lib


def _f32(x):
    return np.ascontiguousarray(x, dtype=np.float32)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _coef(h) -> _Coef:
    return _Coef(float(h.vf_coef), float(h.ent_coef), float(h.kl_coef), float(h.lam),
                 float(h.rho_tw), int(h.is_source), int(h.ratio_mode), int(getattr(h, "objective", 0)))


def loss_categorical(batch: dict, hyper, flip=None) -> dict:
    """Categorical loss terms and gradients (fp64) for a batch dict of fp32 arrays."""
    lib = _load()
    zl = _f32(batch["learner_logits"])
    zt = _f32(batch["target_logits"])
    B, T, A = zl.shape
    wl = _f32(batch["worker_logp"]); act = np.ascontiguousarray(batch["actions"], dtype=np.int32)
    rew = _f32(batch["rewards"]); dis = _f32(batch["discounts"]); val = _f32(batch["values"])
    boot = _f32(batch["bootstrap_values"])
    assert zt.shape == (B, T, A) and wl.shape == (B, T) and act.shape == (B, T)
    assert rew.shape == (B, T) and dis.shape == (B, T) and val.shape == (B, T) and boot.shape == (B,)
    fl = None if flip is None else np.ascontiguousarray(flip, dtype=np.int8)
    out = dict(loss_terms=np.zeros(8), dlogits=np.zeros((B, T, A)), dvalues=np.zeros((B, T)),
               vtarget=np.zeros((B, T)), advantage=np.zeros((B, T)), ratio=np.zeros((B, T)),
               adv_cond=np.zeros((B, T)), pg_weight=np.zeros((B, T)))
    cf = _coef(hyper)
    rc = lib.oracle_impact_loss_categorical(
        _ptr(zl), _ptr(zt), _ptr(wl), _ptr(act), _ptr(rew), _ptr(dis), _ptr(val), _ptr(boot),
        ctypes.c_double(hyper.rho_bar), ctypes.c_double(hyper.c_bar), ctypes.c_double(hyper.clip_eps),
        ctypes.byref(cf), ctypes.c_int64(B), ctypes.c_int64(T), ctypes.c_int64(A), _ptr(fl),
        _ptr(out["loss_terms"]), _ptr(out["dlogits"]), _ptr(out["dvalues"]), _ptr(out["vtarget"]),
        _ptr(out["advantage"]), _ptr(out["ratio"]), _ptr(out["adv_cond"]), _ptr(out["pg_weight"]))
    if rc != 0:
        raise ValueError("oracle rejected its arguments")
    return out


def loss_gaussian(batch: dict, hyper, flip=None) -> dict:
    """Diagonal-Gaussian loss terms and gradients (fp64)."""
    lib = _load()
    mu = _f32(batch["learner_mean"]); ls = _f32(batch["learner_logstd"])
    mut = _f32(batch["target_mean"]); lst = _f32(batch["target_logstd"])
    B, T, D = mu.shape
    wl = _f32(batch["worker_logp"]); act = _f32(batch["actions"])
    rew = _f32(batch["rewards"]); dis = _f32(batch["discounts"]); val = _f32(batch["values"])
    boot = _f32(batch["bootstrap_values"])
    assert ls.shape == mut.shape == lst.shape == act.shape == (B, T, D)
    assert wl.shape == rew.shape == dis.shape == val.shape == (B, T) and boot.shape == (B,)
    fl = None if flip is None else np.ascontiguousarray(flip, dtype=np.int8)
    out = dict(loss_terms=np.zeros(8), dmean=np.zeros((B, T, D)), dlogstd=np.zeros((B, T, D)),
               dvalues=np.zeros((B, T)), vtarget=np.zeros((B, T)), advantage=np.zeros((B, T)),
               ratio=np.zeros((B, T)), adv_cond=np.zeros((B, T)), pg_weight=np.zeros((B, T)))
    cf = _coef(hyper)
    rc = lib.oracle_impact_loss_gaussian(
        _ptr(mu), _ptr(ls), _ptr(mut), _ptr(lst), _ptr(wl), _ptr(act), _ptr(rew), _ptr(dis),
        _ptr(val), _ptr(boot), ctypes.c_double(hyper.rho_bar), ctypes.c_double(hyper.c_bar),
        ctypes.c_double(hyper.clip_eps), ctypes.byref(cf), ctypes.c_int64(B), ctypes.c_int64(T),
        ctypes.c_int64(D), _ptr(fl), _ptr(out["loss_terms"]), _ptr(out["dmean"]), _ptr(out["dlogstd"]),
        _ptr(out["dvalues"]), _ptr(out["vtarget"]), _ptr(out["advantage"]), _ptr(out["ratio"]),
        _ptr(out["adv_cond"]), _ptr(out["pg_weight"]))
    if rc != 0:
        raise ValueError("oracle rejected its arguments")
    return out


class Ring:
    """Metadata of the circular buffer C(N, K); `push`/`sample` return (status, ...)."""

    OK, EMPTY, FULL = 0, 1, 2
    UNIFORM, ROUND_ROBIN = 0, 1

    def __init__(self, N: int, K: int, mode: int = 0, seed: int = 0):
        self._lib = _load()
        self._h = self._lib.oracle_ring_create(N, K, mode, seed)
        if not self._h:
            raise ValueError("bad ring arguments")

    def push(self):
        slot = ctypes.c_int32(-1)
        st = self._lib.oracle_ring_push(self._h, ctypes.byref(slot))
        return st, slot.value

    def sample(self):
        slot = ctypes.c_int32(-1)
        k = ctypes.c_int32(-1)
        st = self._lib.oracle_ring_sample(self._h, ctypes.byref(slot), ctypes.byref(k))
        return st, slot.value, k.value

    def live(self) -> int:
        return self._lib.oracle_ring_live(self._h)

    def __del__(self):
        try:
            self._lib.oracle_ring_destroy(self._h)
        except Exception:
            pass


def draw_u64(seed: int, n: int) -> int:
    return int(_load().oracle_draw_u64(seed, n))
