"""ctypes front-end of the Keyformer CPU oracle (TEST INFRASTRUCTURE).

The arithmetic lives in ``keyformer_oracle.cpp`` (plain double-precision
loops following Algorithm 1 and Eq. 1, 4, 7, 11, 12 of the paper); this file
only marshals numpy arrays.  Nothing here touches the CUDA library, and the
product package never imports this module.

Parity unpinned: the specific kept sets on random data (no worked example is
printed in the paper); see the header of the C++ file for what pins the rest.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading
from dataclasses import dataclass, field

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "keyformer_oracle.cpp")
_LIB = os.path.join(_HERE, "libkeyformer_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle's C++ file with g++ (no GPU involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-O2", "-fopenmp", "-shared", "-fPIC", _SRC, "-o", tmp])
        os.replace(tmp, _LIB)
    return _LIB


class _Params(C.Structure):
    _fields_ = [
        ("head_dim", C.c_int32), ("n_heads", C.c_int32), ("budget_k", C.c_int32),
        ("recent_w", C.c_int32), ("gen_len_T", C.c_int32), ("noise_mode", C.c_int32),
        ("bias_mode", C.c_int32), ("pos_mode", C.c_int32),
        ("tau_init", C.c_double), ("tau_end", C.c_double), ("logit_scale", C.c_double),
        ("noise_const", C.c_double), ("noise_mu", C.c_double), ("noise_sigma", C.c_double),
        ("noise_seed", C.c_uint64), ("alibi_slopes", C.POINTER(C.c_double)), ("n_kv_heads", C.c_int32),
        ("rotary_dims", C.c_int32), ("rotary_base", C.c_double),
    ]


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = C.CDLL(build())
            vp = C.c_void_p
            i32 = C.c_int32
            pp = C.POINTER(_Params)
            lib.ko_half_to_double.restype = C.c_double
            lib.ko_half_to_double.argtypes = [C.c_uint16]
            lib.ko_philox4x32_10.restype = None
            lib.ko_philox4x32_10.argtypes = [vp, vp, vp]
            lib.ko_uniform_from_word.restype = C.c_double
            lib.ko_uniform_from_word.argtypes = [C.c_uint32]
            lib.ko_gumbel_from_word.restype = C.c_double
            lib.ko_gumbel_from_word.argtypes = [C.c_uint32]
            lib.ko_noise.restype = C.c_double
            lib.ko_noise.argtypes = [pp, i32, i32, i32, i32, i32]
            lib.ko_tau.restype = C.c_double
            lib.ko_tau.argtypes = [pp, i32]
            lib.ko_select.restype = None
            lib.ko_select.argtypes = [vp, vp, i32, i32, i32, i32, vp]
            lib.ko_prefill_score_units.restype = None
            lib.ko_prefill_score_units.argtypes = [pp, i32, vp, i32, vp, vp, vp]
            lib.ko_prefill_attend_units.restype = None
            lib.ko_prefill_attend_units.argtypes = [pp, i32, vp, i32, vp, vp, vp, vp]
            lib.ko_prefill_prune_units.restype = None
            lib.ko_prefill_prune_units.argtypes = [pp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp]
            lib.ko_decode_score_units.restype = None
            lib.ko_decode_score_units.argtypes = [pp, i32, vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
            lib.ko_decode_evict_units.restype = None
            lib.ko_decode_evict_units.argtypes = [pp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
            lib.ko_num_threads.restype = i32
            lib.ko_num_threads.argtypes = []
            _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _half_bits(a) -> np.ndarray:
    """float16 array (numpy) -> contiguous uint16 view of its bit patterns."""
    a = np.ascontiguousarray(a)
    assert a.dtype == np.float16, a.dtype
    return a.view(np.uint16)


NOISE_GUMBEL, NOISE_NONE, NOISE_CONST, NOISE_GAUSS = 0, 1, 2, 3


@dataclass
class Params:
    """Inputs of Algorithm 1 plus the readings the paper leaves open."""
    head_dim: int
    n_heads: int
    budget_k: int
    recent_w: int
    gen_len_T: int
    tau_init: float = 1.0
    tau_end: float = 2.0
    noise_seed: int = 0
    noise_mode: int = NOISE_GUMBEL
    bias_mode: int = 0
    alibi_slopes: np.ndarray | None = None
    logit_scale: float = 0.0          # 0 -> 1/sqrt(d)
    noise_const: float = 0.5772
    noise_mu: float = 0.5772
    noise_sigma: float = 1.2825
    pos_mode: int = 0                 # 0 original positions in the bias, 1 places within the reduced cache
    n_kv_heads: int = 0               # key/value heads shared by groups of n_heads / n_kv_heads query heads (0 = none shared)
    rotary_dims: int = 0              # > 0: Q/K come without rotary embedding; it is applied here to their first rotary_dims features
    rotary_base: float = 10000.0
    _keep: list = field(default_factory=list, repr=False)

    @property
    def group(self) -> int:
        """Query heads per key/value head."""
        return self.n_heads // self.n_kv_heads if 0 < self.n_kv_heads < self.n_heads else 1

    def c(self) -> _Params:
        scale = self.logit_scale if self.logit_scale else 1.0 / float(np.sqrt(np.float64(self.head_dim)))
        p = _Params()
        p.head_dim, p.n_heads, p.budget_k = self.head_dim, self.n_heads, self.budget_k
        p.recent_w, p.gen_len_T, p.noise_mode = self.recent_w, self.gen_len_T, self.noise_mode
        p.bias_mode, p.pos_mode = self.bias_mode, self.pos_mode
        p.tau_init, p.tau_end, p.logit_scale = self.tau_init, self.tau_end, scale
        p.noise_const, p.noise_mu, p.noise_sigma = self.noise_const, self.noise_mu, self.noise_sigma
        p.noise_seed = self.noise_seed & 0xFFFFFFFFFFFFFFFF
        p.n_kv_heads = self.n_kv_heads
        p.rotary_dims, p.rotary_base = self.rotary_dims, self.rotary_base
        if self.alibi_slopes is not None:
            s = np.ascontiguousarray(self.alibi_slopes, dtype=np.float64)
            self._keep.append(s)
            p.alibi_slopes = s.ctypes.data_as(C.POINTER(C.c_double))
        return p


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.ascontiguousarray(ctr, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    _load().ko_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def uniform_from_word(r: int) -> float:
    return _load().ko_uniform_from_word(int(r) & 0xFFFFFFFF)


def gumbel_from_word(r: int) -> float:
    return _load().ko_gumbel_from_word(int(r) & 0xFFFFFFFF)


def half_to_double(bits: int) -> float:
    return _load().ko_half_to_double(int(bits) & 0xFFFF)


def noise(P: Params, b: int, l: int, h: int, i: int, j: int) -> float:
    cp = P.c()
    return _load().ko_noise(C.byref(cp), b, l, h, i, j)


def tau(P: Params, t: int) -> float:
    cp = P.c()
    return _load().ko_tau(C.byref(cp), t)


def select(pos, acc, k: int, w: int, p: int) -> np.ndarray:
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    acc = np.ascontiguousarray(acc, dtype=np.float64)
    keep = np.zeros(pos.shape[0], dtype=np.uint8)
    _load().ko_select(_ptr(pos), _ptr(acc), pos.shape[0], k, w, p, _ptr(keep))
    return keep.astype(bool)


def num_threads() -> int:
    return int(_load().ko_num_threads())


class State:
    """Cache of U independent units: up to k+1 entries (pos, acc, K row, V row) each."""

    def __init__(self, P: Params, lbh):
        self.P = P
        self.lbh = np.ascontiguousarray(lbh, dtype=np.int32).reshape(-1, 3)
        self.U = self.lbh.shape[0]
        cap, d = P.budget_k + 1, P.head_dim
        self.cap = cap
        self.len = np.zeros(self.U, dtype=np.int32)
        self.pos = np.full((self.U, cap), -1, dtype=np.int32)
        self.acc = np.zeros((self.U, cap), dtype=np.float64)
        self.K = np.zeros((self.U, cap, d), dtype=np.uint16)
        self.V = np.zeros((self.U, cap, d), dtype=np.uint16)
        self.n_prompt = 0

    # -- prompt phase -------------------------------------------------------
    def prefill_score(self, Q, K) -> np.ndarray:
        """Accumulated prompt scores f_theta[U][n] before pruning (Algorithm 1, t = 0)."""
        Qb, Kb = _half_bits(Q), _half_bits(K)
        U, n, d = Kb.shape
        assert U == self.U and d == self.P.head_dim and Qb.size == Kb.size * self.P.group    # Q: [U][g][n][d]
        acc = np.zeros((U, n), dtype=np.float64)
        cp = self.P.c()
        _load().ko_prefill_score_units(C.byref(cp), U, _ptr(self.lbh), n, _ptr(Qb), _ptr(Kb), _ptr(acc))
        return acc

    def prefill_attend(self, Q, K, V) -> np.ndarray:
        """Causal attention output of the prompt [U][n][d] ([U][g][n][d] with shared key/value heads)
        (Eq. 1; plain softmax, no adjustment)."""
        Qb, Kb, Vb = _half_bits(Q), _half_bits(K), _half_bits(V)
        U, n, d = Kb.shape
        g = self.P.group
        assert U == self.U and d == self.P.head_dim and Kb.shape == Vb.shape and Qb.size == Kb.size * g
        out = np.zeros((U, n, d) if g == 1 else (U, g, n, d), dtype=np.float64)
        cp = self.P.c()
        _load().ko_prefill_attend_units(C.byref(cp), U, _ptr(self.lbh), n, _ptr(Qb), _ptr(Kb), _ptr(Vb), _ptr(out))
        return out

    def prefill_prune(self, K, V, acc_full, keep_override=None) -> None:
        """Keep w recent + top-(k-w) of the rest (or the imposed set) and store the rows."""
        Kb, Vb = _half_bits(K), _half_bits(V)
        U, n, d = Kb.shape
        acc_full = np.ascontiguousarray(acc_full, dtype=np.float64)
        ko = None if keep_override is None else np.ascontiguousarray(keep_override, dtype=np.uint8)
        cp = self.P.c()
        _load().ko_prefill_prune_units(C.byref(cp), U, n, _ptr(Kb), _ptr(Vb), _ptr(acc_full), _ptr(ko),
                                       _ptr(self.len), _ptr(self.pos), _ptr(self.acc), _ptr(self.K), _ptr(self.V))
        self.n_prompt = n

    # -- generation phase ---------------------------------------------------
    def decode_score(self, step: int, q, knew, vnew):
        """Append the new token, attend, score, accumulate.  Returns (out[U][d] -- [U][g][d] with g query heads
        per key/value head --, z[U][cap] = the score added to f_theta: the group's mean)."""
        qb, kb, vb = _half_bits(q), _half_bits(knew), _half_bits(vnew)
        d, g = self.P.head_dim, self.P.group
        assert qb.size == self.U * g * d and kb.shape == (self.U, d) and vb.shape == (self.U, d)    # q: [U][g][d]
        assert int(self.len.max(initial=0)) < self.cap
        out = np.zeros((self.U, d) if g == 1 else (self.U, g, d), dtype=np.float64)
        z = np.zeros((self.U, self.cap), dtype=np.float64)
        cp = self.P.c()
        _load().ko_decode_score_units(C.byref(cp), self.U, _ptr(self.lbh), step, self.n_prompt,
                                      _ptr(qb), _ptr(kb), _ptr(vb),
                                      _ptr(self.len), _ptr(self.pos), _ptr(self.acc), _ptr(self.K), _ptr(self.V),
                                      _ptr(out), _ptr(z))
        return out, z

    def decode_evict(self, step: int, force_evict_pos=None) -> np.ndarray:
        """Apply the selection (or the imposed eviction).  Returns evicted position per unit (-1: none)."""
        f = None if force_evict_pos is None else np.ascontiguousarray(force_evict_pos, dtype=np.int32)
        ev = np.full(self.U, -1, dtype=np.int32)
        cp = self.P.c()
        _load().ko_decode_evict_units(C.byref(cp), self.U, step, self.n_prompt, _ptr(f),
                                      _ptr(self.len), _ptr(self.pos), _ptr(self.acc), _ptr(self.K), _ptr(self.V),
                                      _ptr(ev))
        return ev
