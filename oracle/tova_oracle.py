"""TEST INFRASTRUCTURE - ctypes front end of the CPU checker in tova_oracle.c.

Only tests, the smoke check and the CPU-baseline leg of the benchmark may use
this module.  It compiles tova_oracle.c with gcc twice (REAL=float, the parity
checker; REAL=double, the reference the float build is itself checked with)
and keeps one bounded multi-state per layer in numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tova_oracle.c")
_LIBS = {}


def build(force: bool = False) -> None:
    """Compile both precisions of the checker next to its source."""
    for tag, real in (("f32", "float"), ("f64", "double")):
        so = os.path.join(_HERE, f"libtova_oracle_{tag}.so")
        if not force and os.path.exists(so) and os.path.getmtime(so) >= os.path.getmtime(_SRC):
            continue
        tmp = so + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", f"-DREAL={real}",
               "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, so)


def _lib(precision: str):
    if precision not in _LIBS:
        build()
        tag = {"f32": "f32", "f64": "f64"}[precision]
        lib = ctypes.CDLL(os.path.join(_HERE, f"libtova_oracle_{tag}.so"))
        lib.tova_oracle_step.restype = ctypes.c_int
        lib.tova_oracle_step_policy.restype = ctypes.c_int
        lib.tova_oracle_step_units.restype = ctypes.c_int
        lib.tova_oracle_step_poscomp.restype = ctypes.c_int
        lib.tova_oracle_compress_gap.restype = ctypes.c_double
        lib.tova_oracle_compress_gap.argtypes = [ctypes.c_int]
        lib.tova_oracle_real_bytes.restype = ctypes.c_int
        lib.tova_oracle_max_threads.restype = ctypes.c_int
        _LIBS[precision] = lib
    return _LIBS[precision]


def compress_gap(g: int) -> float:
    """The checker's gap function of the position compression (double build)."""
    return float(_lib("f64").tova_oracle_compress_gap(int(g)))


def host_threads() -> int:
    """Threads the checker may use: the cores this process is allowed on."""
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:  # pragma: no cover
        return max(1, os.cpu_count() or 1)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


class OracleCache:
    """Bounded multi-state (K, V) of one layer for B independent sequences."""

    def __init__(self, batch: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                 capacity: int, sm_scale: float = 0.0, precision: str = "f32",
                 threads: Optional[int] = None, policy: str = "tova", keep_first: int = 0,
                 rope_base: float = 0.0):
        """rope_base > 0: position compression (Section "Extrapolation with TOVA"): keys are cached without
        rotary embedding, which is applied at every step with the compressed positions."""
        if n_q_heads % n_kv_heads:
            raise ValueError("n_q_heads must be a multiple of n_kv_heads")
        self.B, self.H, self.Hkv, self.D, self.cap = batch, n_q_heads, n_kv_heads, head_dim, capacity
        self.scale = float(sm_scale) if sm_scale else 1.0 / float(np.sqrt(head_dim))
        self.precision = precision
        self.real = np.float32 if precision == "f32" else np.float64
        self.creal = ctypes.c_float if precision == "f32" else ctypes.c_double
        self.lib = _lib(precision)
        assert self.lib.tova_oracle_real_bytes() == np.dtype(self.real).itemsize
        self.threads = threads or host_threads()
        self.policy = {"tova": 0, "window": 1}[policy]   # Section 4 / Section 4.1
        self.keep_first = int(keep_first)                  # "+i": positions 0..i-1 are never dropped
        self.rope_base = float(rope_base)
        self.last_cpos = None                              # compressed positions of the last step's candidates
        self.len = np.zeros(batch, np.int32)
        self.pos = np.full((batch, capacity), -1, np.int32)
        self.K = np.zeros((batch, n_kv_heads, capacity, head_dim), self.real)
        self.V = np.zeros_like(self.K)

    def step(self, q, k_new, v_new, pos_t: int, forced=None, want_mean: bool = False):
        """Feed one token to every sequence.

        Returns (out [B,H,D], evicted_pos [B], victim [B], argmin [B], gap [B],
        mean [B,cap+1] or None).
        `forced` [B] int: candidate index to drop instead of the arg-min
        (-1 = no override)."""
        B, H, Hkv, D, cap = self.B, self.H, self.Hkv, self.D, self.cap
        q = np.ascontiguousarray(q, self.real).reshape(B, H, D)
        k_new = np.ascontiguousarray(k_new, self.real).reshape(B, Hkv, D)
        v_new = np.ascontiguousarray(v_new, self.real).reshape(B, Hkv, D)
        out = np.empty((B, H, D), self.real)
        ev = np.empty(B, np.int32)
        victim = np.empty(B, np.int32)
        argmin = np.empty(B, np.int32)
        gap = np.zeros(B, self.real)
        mean = np.zeros((B, cap + 1), self.real) if want_mean else None
        f = None if forced is None else np.ascontiguousarray(forced, np.int32)
        if self.rope_base > 0.0:
            cpos = np.zeros((B, cap + 1), np.float64)
            rc = self.lib.tova_oracle_step_poscomp(
                ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(Hkv), ctypes.c_int(D),
                ctypes.c_int(cap), self.creal(self.scale), ctypes.c_int(self.policy), ctypes.c_int(self.keep_first),
                ctypes.c_double(self.rope_base),
                _ptr(self.len), _ptr(self.pos), _ptr(self.K), _ptr(self.V),
                _ptr(q), _ptr(k_new), _ptr(v_new), ctypes.c_int(int(pos_t)), _ptr(f),
                _ptr(out), _ptr(ev), _ptr(victim), _ptr(argmin), _ptr(gap), _ptr(mean), _ptr(cpos),
                ctypes.c_int(self.threads))
            if rc != 0:
                raise RuntimeError("tova_oracle_step_poscomp rejected its arguments")
            self.last_cpos = cpos
            return out, ev, victim, argmin, gap, mean
        rc = self.lib.tova_oracle_step_policy(
            ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(Hkv), ctypes.c_int(D),
            ctypes.c_int(cap), self.creal(self.scale), ctypes.c_int(self.policy), ctypes.c_int(self.keep_first),
            _ptr(self.len), _ptr(self.pos), _ptr(self.K), _ptr(self.V),
            _ptr(q), _ptr(k_new), _ptr(v_new), ctypes.c_int(int(pos_t)), _ptr(f),
            _ptr(out), _ptr(ev), _ptr(victim), _ptr(argmin), _ptr(gap), _ptr(mean),
            ctypes.c_int(self.threads))
        if rc != 0:
            raise RuntimeError("tova_oracle_step rejected its arguments")
        return out, ev, victim, argmin, gap, mean


UNIT_POLICIES = {"tova_head": 2, "h2o_layer": 3, "h2o_head": 4}


class OracleUnitsCache:
    """Bounded multi-state under the policies that own rows per unit: TOVA-head
    (Section 4, appendix ablation), H2O layer-wise and head-wise (Section 4.1).
    A unit is the layer (h2o_layer: U = 1) or one KV head (U = n_kv_heads)."""

    def __init__(self, batch: int, n_q_heads: int, n_kv_heads: int, head_dim: int, capacity: int,
                 policy: str, recent: int = 0, sm_scale: float = 0.0, precision: str = "f32",
                 threads: Optional[int] = None):
        if n_q_heads % n_kv_heads:
            raise ValueError("n_q_heads must be a multiple of n_kv_heads")
        self.B, self.H, self.Hkv, self.D, self.cap = batch, n_q_heads, n_kv_heads, head_dim, capacity
        self.scale = float(sm_scale) if sm_scale else 1.0 / float(np.sqrt(head_dim))
        self.real = np.float32 if precision == "f32" else np.float64
        self.creal = ctypes.c_float if precision == "f32" else ctypes.c_double
        self.lib = _lib(precision)
        self.threads = threads or host_threads()
        self.policy = UNIT_POLICIES[policy]
        self.U = 1 if policy == "h2o_layer" else n_kv_heads
        # H2O: the non-window rows are half the multi-state size unless told otherwise (Section 4.1)
        self.recent = int(recent) if recent else capacity - capacity // 2
        self.len = np.zeros(batch, np.int32)
        self.pos = np.full((batch, self.U, capacity), -1, np.int32)
        self.acc = np.zeros((batch, self.U, capacity), self.real)
        self.K = np.zeros((batch, n_kv_heads, capacity, head_dim), self.real)
        self.V = np.zeros_like(self.K)

    def step(self, q, k_new, v_new, pos_t: int, forced=None, want_score: bool = False):
        """Returns (out [B,H,D], evicted_pos [B,U], victim [B,U], argmin [B,U], gap [B,U],
        score [B,U,cap+1] or None)."""
        B, H, Hkv, D, cap, U = self.B, self.H, self.Hkv, self.D, self.cap, self.U
        q = np.ascontiguousarray(q, self.real).reshape(B, H, D)
        k_new = np.ascontiguousarray(k_new, self.real).reshape(B, Hkv, D)
        v_new = np.ascontiguousarray(v_new, self.real).reshape(B, Hkv, D)
        out = np.empty((B, H, D), self.real)
        ev = np.empty((B, U), np.int32)
        victim = np.empty((B, U), np.int32)
        argmin = np.empty((B, U), np.int32)
        gap = np.zeros((B, U), self.real)
        score = np.zeros((B, U, cap + 1), self.real) if want_score else None
        f = None if forced is None else np.ascontiguousarray(forced, np.int32).reshape(B, U)
        rc = self.lib.tova_oracle_step_units(
            ctypes.c_int(B), ctypes.c_int(H), ctypes.c_int(Hkv), ctypes.c_int(D),
            ctypes.c_int(cap), self.creal(self.scale), ctypes.c_int(self.policy), ctypes.c_int(self.recent),
            _ptr(self.len), _ptr(self.pos), _ptr(self.acc), _ptr(self.K), _ptr(self.V),
            _ptr(q), _ptr(k_new), _ptr(v_new), ctypes.c_int(int(pos_t)), _ptr(f),
            _ptr(out), _ptr(ev), _ptr(victim), _ptr(argmin), _ptr(gap), _ptr(score),
            ctypes.c_int(self.threads))
        if rc != 0:
            raise RuntimeError("tova_oracle_step_units rejected its arguments")
        return out, ev, victim, argmin, gap, score
