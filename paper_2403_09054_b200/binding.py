"""Thin ctypes binding of the C ABI declared in ``include/keyformer.h``.

Argument marshalling only: every step of the path runs in the CUDA kernels of
``libkeyformer_b200.so``.  PyTorch supplies device memory and streams.  There is
no fallback: if the library cannot be loaded, importing this module fails.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

from . import build as _build

KF_OK, KF_EINVAL, KF_ENOSPC, KF_ESTATE, KF_ECUDA, KF_ETIMEOUT, KF_EBOUNDS = 0, -1, -2, -3, -4, -5, -6
KF_NOISE_GUMBEL, KF_NOISE_NONE, KF_NOISE_CONST, KF_NOISE_GAUSS = 0, 1, 2, 3
KF_BIAS_NONE, KF_BIAS_ALIBI = 0, 1
KF_PREFILL_TENSOR, KF_PREFILL_SIMT = 0, 1
KF_POS_ORIGINAL, KF_POS_NEW = 0, 1
KF_DECODE_AUTO, KF_DECODE_CUDA_CORES, KF_DECODE_TENSOR = 0, 1, 2

EXPORTS = ("kf_workspace_bytes", "kf_create", "kf_prefill_score_prune", "kf_decode_step",
           "kf_decode_step_host", "kf_view_state", "kf_poll_error", "kf_launch_count",
           "kf_destroy", "kf_strerror", "kf_decode_step_static", "kf_state_bytes", "kf_export_state", "kf_import_state",
           "kf_prefill_attend", "kf_prefill_attend_score_prune", "kf_view_place", "kf_compact_layer", "kf_check_canaries", "kf_describe_decode")


class kf_config(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("batch", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32),
        ("budget_k", C.c_int32), ("recent_w", C.c_int32), ("max_prompt_len", C.c_int32), ("gen_len_T", C.c_int32),
        ("tau_init", C.c_float), ("tau_end", C.c_float), ("noise_seed", C.c_uint64),
        ("noise_mode", C.c_int32), ("bias_mode", C.c_int32), ("h_alibi_slopes", C.POINTER(C.c_float)),
        ("logit_scale", C.c_float), ("noise_const", C.c_float),
        ("decode_splits", C.c_int32), ("prefill_impl", C.c_int32),
        ("noise_mu", C.c_float), ("noise_sigma", C.c_float), ("pos_mode", C.c_int32),
        ("n_kv_heads", C.c_int32), ("rotary_dims", C.c_int32), ("rotary_base", C.c_float), ("decode_impl", C.c_int32), ("debug_canaries", C.c_int32), ("debug_fail_first_wait", C.c_int32),
    ]


class kf_static_step(C.Structure):
    _fields_ = [
        ("batch", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32),
        ("budget_k", C.c_int32), ("recent_w", C.c_int32), ("layer", C.c_int32), ("position", C.c_int32),
        ("noise_mode", C.c_int32), ("bias_mode", C.c_int32), ("reserved", C.c_int32),
        ("tau", C.c_double), ("noise_seed", C.c_uint64), ("logit_scale", C.c_float), ("noise_const", C.c_float),
        ("d_alibi_slopes", C.c_void_p),
    ]


KF_STATIC_SCRATCH_BYTES = 16 << 20


def _load() -> C.CDLL:
    path = _build.LIB
    if not os.path.exists(path):
        path = _build.build()
    lib = C.CDLL(path)
    vp, i32 = C.c_void_p, C.c_int32
    cfgp = C.POINTER(kf_config)
    lib.kf_workspace_bytes.restype = C.c_size_t
    lib.kf_workspace_bytes.argtypes = [cfgp]
    lib.kf_create.restype = C.c_int
    lib.kf_create.argtypes = [cfgp, vp, C.c_size_t, vp, C.POINTER(vp)]
    lib.kf_prefill_score_prune.restype = C.c_int
    lib.kf_prefill_score_prune.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp]
    lib.kf_prefill_attend.restype = C.c_int
    lib.kf_prefill_attend.argtypes = [vp, i32, vp, vp, vp, vp, vp]
    lib.kf_prefill_attend_score_prune.restype = C.c_int
    lib.kf_prefill_attend_score_prune.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp]
    lib.kf_decode_step.restype = C.c_int
    lib.kf_decode_step.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp, vp]
    lib.kf_decode_step_host.restype = C.c_int
    lib.kf_decode_step_host.argtypes = [vp, i32, i32, vp, vp, vp, vp, i32, vp]
    lib.kf_decode_step_static.restype = C.c_int
    lib.kf_decode_step_static.argtypes = [C.POINTER(kf_static_step)] + [vp] * 11
    lib.kf_state_bytes.restype = C.c_size_t
    lib.kf_state_bytes.argtypes = [vp]
    lib.kf_export_state.restype = C.c_int
    lib.kf_export_state.argtypes = [vp, i32, vp, C.c_size_t, C.POINTER(i32), C.POINTER(i32), vp]
    lib.kf_import_state.restype = C.c_int
    lib.kf_import_state.argtypes = [vp, i32, vp, C.c_size_t, i32, i32, vp]
    lib.kf_compact_layer.restype = C.c_int
    lib.kf_compact_layer.argtypes = [vp, i32, vp]
    lib.kf_view_place.restype = C.c_int
    lib.kf_view_place.argtypes = [vp, i32, C.POINTER(vp)]
    lib.kf_view_state.restype = C.c_int
    lib.kf_view_state.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), C.POINTER(vp)]
    lib.kf_poll_error.restype = C.c_int
    lib.kf_poll_error.argtypes = [vp, vp]
    lib.kf_check_canaries.restype = C.c_int
    lib.kf_check_canaries.argtypes = [vp, vp, C.POINTER(i32)]
    lib.kf_describe_decode.restype = C.c_int
    lib.kf_describe_decode.argtypes = [vp, C.c_char_p, C.c_size_t]
    lib.kf_launch_count.restype = C.c_int64
    lib.kf_launch_count.argtypes = [vp]
    lib.kf_destroy.restype = C.c_int
    lib.kf_destroy.argtypes = [vp]
    lib.kf_strerror.restype = C.c_char_p
    lib.kf_strerror.argtypes = [C.c_int]
    return lib


LIB = _load()
LIB_PATH = _build.LIB


class KeyformerError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {LIB.kf_strerror(code).decode()} ({code})")


def _check(code: int, where: str) -> None:
    if code != KF_OK:
        raise KeyformerError(code, where)


def kf_strerror(code: int) -> str:
    return LIB.kf_strerror(code).decode()


def make_config(*, n_layers, batch, n_heads, head_dim, budget_k, recent_w, max_prompt_len, gen_len_T,
                tau_init=1.0, tau_end=2.0, noise_seed=0, noise_mode=KF_NOISE_GUMBEL, bias_mode=KF_BIAS_NONE,
                alibi_slopes=None, logit_scale=0.0, noise_const=0.5772, decode_splits=0,
                prefill_impl=KF_PREFILL_TENSOR, noise_mu=0.5772, noise_sigma=1.2825, pos_mode=KF_POS_ORIGINAL,
                n_kv_heads=0, rotary_dims=0, rotary_base=10000.0, decode_impl=0, debug_canaries=0, debug_fail_first_wait=0):
    """Fill a kf_config; returns (config, keepalive) where keepalive holds the slopes array."""
    cfg = kf_config()
    cfg.n_layers, cfg.batch, cfg.n_heads, cfg.head_dim = n_layers, batch, n_heads, head_dim
    cfg.budget_k, cfg.recent_w, cfg.max_prompt_len, cfg.gen_len_T = budget_k, recent_w, max_prompt_len, gen_len_T
    cfg.tau_init, cfg.tau_end = tau_init, tau_end
    cfg.noise_seed = noise_seed & 0xFFFFFFFFFFFFFFFF
    cfg.noise_mode, cfg.bias_mode = noise_mode, bias_mode
    keep = None
    if alibi_slopes is not None:
        keep = np.ascontiguousarray(alibi_slopes, dtype=np.float32)
        cfg.h_alibi_slopes = keep.ctypes.data_as(C.POINTER(C.c_float))
    cfg.logit_scale, cfg.noise_const = logit_scale, noise_const
    cfg.decode_splits, cfg.prefill_impl = decode_splits, prefill_impl
    cfg.noise_mu, cfg.noise_sigma = noise_mu, noise_sigma
    cfg.pos_mode = pos_mode
    cfg.n_kv_heads, cfg.decode_impl = n_kv_heads, decode_impl
    cfg.rotary_dims, cfg.rotary_base = rotary_dims, rotary_base
    cfg.debug_canaries, cfg.debug_fail_first_wait = debug_canaries, debug_fail_first_wait
    return cfg, keep


def kf_workspace_bytes(cfg: kf_config) -> int:
    return int(LIB.kf_workspace_bytes(C.byref(cfg)))


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _dev_ptr(t, dtype, numel, name):
    if t is None:
        return None
    if not (t.is_cuda and t.is_contiguous() and t.dtype == dtype and t.numel() == numel):
        raise ValueError(f"{name}: expected a contiguous CUDA {dtype} tensor with {numel} elements, "
                         f"got {t.dtype} {tuple(t.shape)} on {t.device}")
    return t.data_ptr()


def kf_decode_step_static(*, batch, n_heads, head_dim, budget_k, recent_w, layer, position, tau,
                          K, V, pos, acc, length, q, knew, vnew, out, score_out=None, noise_seed=0,
                          noise_mode=KF_NOISE_GUMBEL, noise_const=0.5772, bias_mode=KF_BIAS_NONE,
                          alibi_slopes_dev=None, logit_scale=0.0, stream=None) -> int:
    """One generation step on caller-held cache tensors, using the library's built-in scratch block
    (for callers that cannot allocate device memory).  Returns the KF_* status code."""
    a = kf_static_step()
    a.batch, a.n_heads, a.head_dim, a.budget_k, a.recent_w = batch, n_heads, head_dim, budget_k, recent_w
    a.layer, a.position, a.noise_mode, a.bias_mode, a.reserved = layer, position, noise_mode, bias_mode, 0
    a.tau, a.noise_seed, a.logit_scale, a.noise_const = tau, noise_seed & 0xFFFFFFFFFFFFFFFF, logit_scale, noise_const
    a.d_alibi_slopes = None if alibi_slopes_dev is None else alibi_slopes_dev.data_ptr()
    U = batch * n_heads
    return int(LIB.kf_decode_step_static(
        C.byref(a),
        _dev_ptr(K, torch.float16, U * budget_k * head_dim, "K"), _dev_ptr(V, torch.float16, U * budget_k * head_dim, "V"),
        _dev_ptr(pos, torch.int32, U * budget_k, "pos"), _dev_ptr(acc, torch.float32, U * budget_k, "acc"),
        _dev_ptr(length, torch.int32, U, "length"),
        _dev_ptr(q, torch.float16, U * head_dim, "q"), _dev_ptr(knew, torch.float16, U * head_dim, "knew"),
        _dev_ptr(vnew, torch.float16, U * head_dim, "vnew"), _dev_ptr(out, torch.float16, U * head_dim, "out"),
        _dev_ptr(score_out, torch.float32, U * (budget_k + 1), "score_out"), _stream_ptr(stream)))


class Keyformer:
    """A context (kf_create .. kf_destroy) over a torch-allocated workspace."""

    def __init__(self, device="cuda:0", stream=None, **cfg_kwargs):
        if not torch.cuda.is_available():
            raise KeyformerError(KF_ECUDA, "Keyformer(): no CUDA device (the library has no CPU path)")
        self.device = torch.device(device)
        self.cfg, self._keep = make_config(**cfg_kwargs)
        nbytes = kf_workspace_bytes(self.cfg)
        if nbytes == 0:
            raise KeyformerError(KF_EINVAL, "kf_workspace_bytes")
        self.workspace_bytes = nbytes
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            base = self.workspace.data_ptr()
            self._ws_ptr = (base + 255) // 256 * 256
            h = C.c_void_p()
            _check(LIB.kf_create(C.byref(self.cfg), self._ws_ptr, nbytes, _stream_ptr(stream), C.byref(h)), "kf_create")
        self._h = h
        self.kv_heads = self.cfg.n_kv_heads if self.cfg.n_kv_heads > 0 else self.cfg.n_heads
        self.units_q = self.cfg.batch * self.cfg.n_heads       # (batch row, query head) pairs
        self.units = self.cfg.batch * self.kv_heads            # caches per layer: (batch row, key/value head) pairs

    # ---- the C calls, same names ---------------------------------------------------------
    def kf_prefill_score_prune(self, layer, q, k, v, score_out=None, stream=None):
        d = self.cfg.head_dim
        n = q.shape[-2]
        _check(LIB.kf_prefill_score_prune(
            self._h, layer, n,
            _dev_ptr(q, torch.float16, self.units_q * n * d, "q"), _dev_ptr(k, torch.float16, self.units * n * d, "k"),
            _dev_ptr(v, torch.float16, self.units * n * d, "v"),
            _dev_ptr(score_out, torch.float32, self.units * n, "score_out"), _stream_ptr(stream)),
            "kf_prefill_score_prune")

    def kf_prefill_attend(self, q, k, v, out, stream=None):
        d = self.cfg.head_dim
        n = q.shape[-2]
        _check(LIB.kf_prefill_attend(
            self._h, n, _dev_ptr(q, torch.float16, self.units_q * n * d, "q"), _dev_ptr(k, torch.float16, self.units * n * d, "k"),
            _dev_ptr(v, torch.float16, self.units * n * d, "v"), _dev_ptr(out, torch.float16, self.units_q * n * d, "out"),
            _stream_ptr(stream)), "kf_prefill_attend")

    def kf_prefill_attend_score_prune(self, layer, q, k, v, out, score_out=None, stream=None):
        d = self.cfg.head_dim
        n = q.shape[-2]
        _check(LIB.kf_prefill_attend_score_prune(
            self._h, layer, n, _dev_ptr(q, torch.float16, self.units_q * n * d, "q"),
            _dev_ptr(k, torch.float16, self.units * n * d, "k"), _dev_ptr(v, torch.float16, self.units * n * d, "v"),
            _dev_ptr(out, torch.float16, self.units_q * n * d, "out"),
            _dev_ptr(score_out, torch.float32, self.units * n, "score_out"), _stream_ptr(stream)),
            "kf_prefill_attend_score_prune")

    def kf_decode_step(self, layer, step, q, knew, vnew, out, score_out=None, stream=None):
        d = self.cfg.head_dim
        _check(LIB.kf_decode_step(
            self._h, layer, step,
            _dev_ptr(q, torch.float16, self.units_q * d, "q"), _dev_ptr(knew, torch.float16, self.units * d, "knew"),
            _dev_ptr(vnew, torch.float16, self.units * d, "vnew"), _dev_ptr(out, torch.float16, self.units_q * d, "out"),
            _dev_ptr(score_out, torch.float32, self.units * (self.cfg.budget_k + 1), "score_out"),
            _stream_ptr(stream)), "kf_decode_step")

    def kf_decode_step_host(self, layer, step, q, knew, vnew, out, wait=True, stream=None):
        d = self.cfg.head_dim
        for name, t, numel in (("q", q, self.units_q * d), ("knew", knew, self.units * d), ("vnew", vnew, self.units * d),
                               ("out", out, self.units_q * d)):
            if t.is_cuda or not t.is_contiguous() or t.dtype != torch.float16 or t.numel() != numel:
                raise ValueError(f"{name}: expected a contiguous host float16 tensor with {numel} elements")
        _check(LIB.kf_decode_step_host(self._h, layer, step, q.data_ptr(), knew.data_ptr(), vnew.data_ptr(),
                                       out.data_ptr(), 1 if wait else 0, _stream_ptr(stream)), "kf_decode_step_host")

    def kf_view_state(self, layer):
        """Zero-copy torch views (K, V, pos, acc, len) of one layer's cache inside the workspace."""
        ptrs = [C.c_void_p() for _ in range(5)]
        _check(LIB.kf_view_state(self._h, layer, *[C.byref(p) for p in ptrs]), "kf_view_state")
        B, H, k, d = self.cfg.batch, self.kv_heads, self.cfg.budget_k, self.cfg.head_dim   # one cache per key/value head
        base = self.workspace.data_ptr()

        def view(ptr, nbytes, dtype, shape):
            off = ptr.value - base
            return self.workspace[off:off + nbytes].view(dtype).view(shape)
        K = view(ptrs[0], B * H * k * d * 2, torch.float16, (B, H, k, d))
        V = view(ptrs[1], B * H * k * d * 2, torch.float16, (B, H, k, d))
        pos = view(ptrs[2], B * H * k * 4, torch.int32, (B, H, k))
        acc = view(ptrs[3], B * H * k * 4, torch.float32, (B, H, k))
        ln = view(ptrs[4], B * H * 4, torch.int32, (B, H))
        return K, V, pos, acc, ln

    def kf_compact_layer(self, layer, stream=None):
        """Reorder the layer's cache entries into ascending position, in place."""
        _check(LIB.kf_compact_layer(self._h, layer, _stream_ptr(stream)), "kf_compact_layer")

    def kf_view_place(self, layer):
        """Zero-copy torch view of one layer's places (KF_POS_NEW only), int32 [B, H, k]."""
        ptr = C.c_void_p()
        _check(LIB.kf_view_place(self._h, layer, C.byref(ptr)), "kf_view_place")
        B, H, k = self.cfg.batch, self.kv_heads, self.cfg.budget_k
        off = ptr.value - self.workspace.data_ptr()
        return self.workspace[off:off + B * H * k * 4].view(torch.int32).view(B, H, k)

    def kf_state_bytes(self) -> int:
        return int(LIB.kf_state_bytes(self._h))

    def kf_export_state(self, layer, image, stream=None):
        """Copy one layer's cache image into the uint8 CUDA tensor `image`; returns (n_prompt, last_step)."""
        n_prompt, last_step = C.c_int32(), C.c_int32()
        _check(LIB.kf_export_state(self._h, layer, _dev_ptr(image, torch.uint8, image.numel(), "image"), image.numel(),
                                   C.byref(n_prompt), C.byref(last_step), _stream_ptr(stream)), "kf_export_state")
        return n_prompt.value, last_step.value

    def kf_import_state(self, layer, image, n_prompt, last_step, stream=None):
        _check(LIB.kf_import_state(self._h, layer, _dev_ptr(image, torch.uint8, image.numel(), "image"), image.numel(),
                                   n_prompt, last_step, _stream_ptr(stream)), "kf_import_state")

    def kf_poll_error(self, stream=None) -> int:
        return int(LIB.kf_poll_error(self._h, _stream_ptr(stream)))

    def kf_check_canaries(self, stream=None):
        """(status, index of the first sub-buffer whose guard was overwritten or -1); debug layout only."""
        bad = C.c_int32(-1)
        rc = int(LIB.kf_check_canaries(self._h, _stream_ptr(stream), C.byref(bad)))
        return rc, bad.value

    def kf_describe_decode(self) -> str:
        buf = C.create_string_buffer(256)
        _check(min(0, int(LIB.kf_describe_decode(self._h, buf, len(buf)))), "kf_describe_decode")
        return buf.value.decode()

    def kf_launch_count(self) -> int:
        return int(LIB.kf_launch_count(self._h))

    def kf_destroy(self):
        if self._h is not None and self._h.value:
            LIB.kf_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.kf_destroy()
        except Exception:
            pass
