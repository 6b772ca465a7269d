"""ctypes binding of libfaedkv.so: the same names as include/faedkv.h.

Argument marshalling only.  Every step of the path runs in the library's CUDA
kernels; there is no Python or CPU fallback -- if the library is missing or a
call fails, an exception is raised.

Device buffers are torch tensors (PyTorch is used for device memory and
streams only); their ``data_ptr()`` is what crosses the ABI.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# FAEDKV_LIBRARY selects another build of the same library (the checked build, lib/libfaedkv_debug.so)
LIB_PATH = os.environ.get("FAEDKV_LIBRARY") or os.path.join(_HERE, "lib", "libfaedkv.so")

F32, BF16 = 0, 1
PREFILL_AUTO, PREFILL_SIMT, PREFILL_UMMA, PREFILL_FFT = 0, 1, 2, 3
STATE_SUM, STATE_MEAN, STATE_ROTATING = 0, 1, 2
DECODE_AUTO, DECODE_SIMT, DECODE_UMMA, DECODE_FFT, DECODE_FFT_TWO_PASS = 0, 1, 2, 3, 4

EXPORTS = [
    "faedkv_create", "faedkv_destroy", "faedkv_last_error", "faedkv_plan", "faedkv_n_bins",
    "faedkv_get_bins", "faedkv_coef_bytes", "faedkv_mask_lowpass", "faedkv_mask_mixed",
    "faedkv_compress_prefill", "faedkv_append", "faedkv_reconstruct", "faedkv_decode_attn",
    "faedkv_append_decode_attn", "faedkv_chunk_range", "faedkv_ablation_bins", "faedkv_mask_from_scores", "faedkv_ablate",
    "faedkv_convert_state", "faedkv_window_bytes", "faedkv_prefill_windowed", "faedkv_step_windowed",
    "faedkv_reconstruct_windowed",
    "faedkv_device_status", "faedkv_launch_count", "faedkv_decode_attn_static",
    "faedkv_reset_device_status", "faedkv_test_hooks", "faedkv_debug_build", "faedkv_debug_word",
]

STATIC_SCRATCH_BYTES = 8 << 20


class FaedkvError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"faedkv error {code}: {msg}")
        self.code = code


class Config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in (
        "n_layers", "n_kv_heads", "n_q_heads", "head_dim", "n_dft", "max_batch", "kv_dtype",
        "prefill_mode", "twiddle_terms", "decode_mode", "n_sink", "n_recent", "n_defer", "recon_engine")]


_lib = None
_vp = ctypes.c_void_p
_int = ctypes.c_int


def load() -> ctypes.CDLL:
    """Load the library (built by `python -m paper_2507_20030_b200.build`); fails loudly if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2507_20030_b200.build` "
            "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    lib.faedkv_create.argtypes = [ctypes.POINTER(Config), ctypes.POINTER(_vp)]
    lib.faedkv_create.restype = _int
    lib.faedkv_destroy.argtypes = [_vp]
    lib.faedkv_destroy.restype = None
    lib.faedkv_last_error.argtypes = [_vp]
    lib.faedkv_last_error.restype = ctypes.c_char_p
    lib.faedkv_plan.argtypes = [_vp, _int, _vp, ctypes.POINTER(_int)]
    lib.faedkv_plan.restype = _int
    lib.faedkv_n_bins.argtypes = [_vp, _int]
    lib.faedkv_n_bins.restype = _int
    lib.faedkv_get_bins.argtypes = [_vp, _int, _vp]
    lib.faedkv_get_bins.restype = _int
    lib.faedkv_coef_bytes.argtypes = [_vp, _int, _int]
    lib.faedkv_coef_bytes.restype = ctypes.c_size_t
    lib.faedkv_mask_lowpass.argtypes = [_int, _int, _vp]
    lib.faedkv_mask_lowpass.restype = _int
    lib.faedkv_mask_mixed.argtypes = [_int, _int, _int, ctypes.c_uint64, _vp]
    lib.faedkv_mask_mixed.restype = _int
    lib.faedkv_compress_prefill.argtypes = [_vp, _int, _vp, _vp, _int, _int, _vp, _vp, _vp, _vp]
    lib.faedkv_compress_prefill.restype = _int
    lib.faedkv_append.argtypes = [_vp, _int, _vp, _vp, _int, _vp, _vp, _vp, _vp]
    lib.faedkv_append.restype = _int
    lib.faedkv_reconstruct.argtypes = [_vp, _int, _vp, _vp, _vp, _int, _int, _vp, _vp, _vp]
    lib.faedkv_reconstruct.restype = _int
    lib.faedkv_decode_attn.argtypes = [_vp, _int, _vp, _vp, _vp, _vp, _int, ctypes.c_float, _vp, _vp]
    lib.faedkv_decode_attn.restype = _int
    lib.faedkv_append_decode_attn.argtypes = [_vp, _int, _vp, _vp, _vp, _int, _vp, _vp, _vp, ctypes.c_float, _vp, _vp]
    lib.faedkv_append_decode_attn.restype = _int
    lib.faedkv_chunk_range.argtypes = [_int, _int, _int, ctypes.POINTER(_int), ctypes.POINTER(_int)]
    lib.faedkv_chunk_range.restype = _int
    lib.faedkv_ablation_bins.argtypes = [_int, _int, _int, _vp, _vp]
    lib.faedkv_ablation_bins.restype = _int
    lib.faedkv_mask_from_scores.argtypes = [_int, _int, _vp, ctypes.c_double, _vp, ctypes.POINTER(_int)]
    lib.faedkv_mask_from_scores.restype = _int
    lib.faedkv_ablate.argtypes = [_vp, _int, _vp, _vp, _int, _int, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
    lib.faedkv_ablate.restype = _int
    lib.faedkv_convert_state.argtypes = [_vp, _int, _vp, _vp, _int, _int, _int, _vp, _vp]
    lib.faedkv_convert_state.restype = _int
    lib.faedkv_window_bytes.argtypes = [_vp, _int]
    lib.faedkv_window_bytes.restype = ctypes.c_size_t
    lib.faedkv_prefill_windowed.argtypes = [_vp, _int, _vp, _vp, _int, _int, _vp, _vp, _vp, _vp, _vp, _vp]
    lib.faedkv_prefill_windowed.restype = _int
    lib.faedkv_step_windowed.argtypes = [_vp, _int, _vp, _vp, _vp, _int, _vp, _vp, _vp, _vp, _vp, ctypes.c_float, _vp, _vp]
    lib.faedkv_step_windowed.restype = _int
    lib.faedkv_reconstruct_windowed.argtypes = [_vp, _int, _vp, _vp, _vp, _vp, _vp, _int, _int, _vp, _vp, _vp]
    lib.faedkv_reconstruct_windowed.restype = _int
    lib.faedkv_device_status.argtypes = [_vp, _vp]
    lib.faedkv_device_status.restype = _int
    lib.faedkv_decode_attn_static.argtypes = [_int, _int, _int, _int, _vp, _int, _vp, _vp, _vp, _vp, _int,
                                              ctypes.c_float, _vp, _vp, ctypes.c_char_p, ctypes.c_size_t]
    lib.faedkv_decode_attn_static.restype = _int
    lib.faedkv_launch_count.argtypes = [_vp]
    lib.faedkv_launch_count.restype = ctypes.c_ulonglong
    lib.faedkv_reset_device_status.argtypes = [_vp, _vp]
    lib.faedkv_reset_device_status.restype = _int
    lib.faedkv_test_hooks.argtypes = [_vp, ctypes.c_ulonglong, _int]
    lib.faedkv_test_hooks.restype = _int
    lib.faedkv_debug_build.argtypes = []
    lib.faedkv_debug_build.restype = _int
    lib.faedkv_debug_word.argtypes = [_vp, _vp]
    lib.faedkv_debug_word.restype = ctypes.c_longlong
    _lib = lib
    return lib


def mask_lowpass(n_dft: int, n_keep: int) -> np.ndarray:
    out = np.zeros(n_dft // 2 + 1, dtype=np.uint8)
    rc = load().faedkv_mask_lowpass(n_dft, n_keep, out.ctypes.data)
    if rc != 0:
        raise FaedkvError(rc, "faedkv_mask_lowpass rejected its arguments")
    return out


def mask_mixed(n_dft: int, n_keep: int, layer: int, seed: int) -> np.ndarray:
    out = np.zeros(n_dft // 2 + 1, dtype=np.uint8)
    rc = load().faedkv_mask_mixed(n_dft, n_keep, layer, seed, out.ctypes.data)
    if rc != 0:
        raise FaedkvError(rc, "faedkv_mask_mixed rejected its arguments")
    return out


def chunk_range(n_dft: int, n_chunks: int, chunk: int) -> tuple[int, int]:
    lo, hi = _int(0), _int(0)
    rc = load().faedkv_chunk_range(n_dft, n_chunks, chunk, ctypes.byref(lo), ctypes.byref(hi))
    if rc != 0:
        raise FaedkvError(rc, "faedkv_chunk_range rejected its arguments")
    return lo.value, hi.value


def ablation_bins(n_dft: int, lo: int, hi: int) -> tuple[np.ndarray, np.ndarray]:
    mask = np.zeros(n_dft // 2 + 1, dtype=np.uint8)
    gain = np.zeros(n_dft // 2 + 1, dtype=np.float32)
    rc = load().faedkv_ablation_bins(n_dft, lo, hi, mask.ctypes.data, gain.ctypes.data)
    if rc != 0:
        raise FaedkvError(rc, "faedkv_ablation_bins rejected its arguments")
    return mask, gain


def mask_from_scores(n_dft: int, n_chunks: int, delta, ratio: float) -> tuple[np.ndarray, int]:
    d = np.ascontiguousarray(delta, dtype=np.float64)
    if d.shape != (n_chunks,):
        raise ValueError("delta must have one entry per chunk")
    mask = np.zeros(n_dft // 2 + 1, dtype=np.uint8)
    n_keep = _int(0)
    rc = load().faedkv_mask_from_scores(n_dft, n_chunks, d.ctypes.data, float(ratio), mask.ctypes.data, ctypes.byref(n_keep))
    if rc != 0:
        raise FaedkvError(rc, "faedkv_mask_from_scores rejected its arguments")
    return mask, n_keep.value


def decode_attn_static(n_dft: int, n_kv_heads: int, n_q_heads: int, kv_dtype: int, bins, q, coefK, coefV,
                       t_len, out, scale: float = 0.0, stream=None) -> None:
    """faedkv_decode_attn_static: decode attention without a context and without any allocation.

    For callers that cannot allocate device memory where they need attention (inside a stream
    capture, under an external memory pool, in a plugin that only receives tensors).  `bins` is a
    device int32 tensor holding the layer's retained bins.  All intermediates live in a fixed
    array inside the library (STATIC_SCRATCH_BYTES); larger problems raise FaedkvError(-3).
    Calls share that array, so calls that overlap on the GPU must be serialised by the caller."""
    buf = ctypes.create_string_buffer(256)
    rc = load().faedkv_decode_attn_static(
        n_dft, n_kv_heads, n_q_heads, kv_dtype, _ptr(bins), int(bins.numel()), _ptr(q), _ptr(coefK),
        _ptr(coefV), _ptr(t_len), int(q.shape[0]), float(scale), _ptr(out), _stream(stream), buf, 256)
    if rc != 0:
        raise FaedkvError(rc, buf.value.decode())


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_contiguous(), "tensors crossing the ABI must be contiguous"
    return t.data_ptr()


def _stream(stream) -> int | None:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


@dataclass
class Context:
    """Owner of one faedkv_ctx; methods carry the names of the C calls without the prefix."""
    n_layers: int
    n_kv_heads: int
    n_q_heads: int
    n_dft: int
    max_batch: int
    kv_dtype: int = BF16
    head_dim: int = 128
    prefill_mode: int = PREFILL_AUTO
    twiddle_terms: int = 0
    decode_mode: int = DECODE_AUTO
    n_sink: int = 0
    n_recent: int = 0
    n_defer: int = 0
    recon_engine: int = 0

    def __post_init__(self):
        self._lib = load()
        cfg = Config(self.n_layers, self.n_kv_heads, self.n_q_heads, self.head_dim, self.n_dft,
                     self.max_batch, self.kv_dtype, self.prefill_mode, self.twiddle_terms, self.decode_mode,
                     self.n_sink, self.n_recent, self.n_defer, self.recon_engine)
        h = _vp()
        rc = self._lib.faedkv_create(ctypes.byref(cfg), ctypes.byref(h))
        if rc != 0:
            raise FaedkvError(rc, "faedkv_create failed")
        self._h = h

    # -- lifetime
    def close(self):
        if getattr(self, "_h", None):
            self._lib.faedkv_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int):
        if rc != 0:
            raise FaedkvError(rc, self._lib.faedkv_last_error(self._h).decode())

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.kv_dtype == BF16 else torch.float32

    # -- plan
    def plan(self, layer: int, bin_mask: np.ndarray) -> int:
        mask = np.ascontiguousarray(bin_mask, dtype=np.uint8)
        if mask.shape != (self.n_dft // 2 + 1,):
            raise ValueError("bin_mask must have length n_dft // 2 + 1")
        n = _int(0)
        self._check(self._lib.faedkv_plan(self._h, layer, mask.ctypes.data, ctypes.byref(n)))
        return n.value

    def n_bins(self, layer: int) -> int:
        m = self._lib.faedkv_n_bins(self._h, layer)
        if m < 0:
            raise FaedkvError(m, "layer not planned")
        return m

    def get_bins(self, layer: int) -> np.ndarray:
        out = np.zeros(self.n_bins(layer), dtype=np.int32)
        self._check(self._lib.faedkv_get_bins(self._h, layer, out.ctypes.data))
        return out

    def coef_bytes(self, layer: int, batch: int) -> int:
        return int(self._lib.faedkv_coef_bytes(self._h, layer, batch))

    def alloc_coef(self, layer: int, batch: int, device="cuda") -> torch.Tensor:
        """float32 [batch, n_kv_heads, 2, M, head_dim] (uninitialised)."""
        return torch.empty((batch, self.n_kv_heads, 2, self.n_bins(layer), self.head_dim),
                           dtype=torch.float32, device=device)

    # -- the four device calls
    def compress_prefill(self, layer, K, V, coefK, coefV, t_len, stream=None):
        batch, T = K.shape[0], K.shape[2]
        self._check(self._lib.faedkv_compress_prefill(
            self._h, layer, _ptr(K), _ptr(V), batch, T, _ptr(coefK), _ptr(coefV), _ptr(t_len),
            _stream(stream)))

    def append(self, layer, k_new, v_new, coefK, coefV, t_len, stream=None):
        batch = k_new.shape[0]
        self._check(self._lib.faedkv_append(
            self._h, layer, _ptr(k_new), _ptr(v_new), batch, _ptr(coefK), _ptr(coefV), _ptr(t_len),
            _stream(stream)))

    def reconstruct(self, layer, coefK, coefV, t_len, L, K_out, V_out, stream=None):
        batch = t_len.shape[0]
        self._check(self._lib.faedkv_reconstruct(
            self._h, layer, _ptr(coefK), _ptr(coefV), _ptr(t_len), batch, L, _ptr(K_out), _ptr(V_out),
            _stream(stream)))

    def decode_attn(self, layer, q, coefK, coefV, t_len, out, scale: float = 0.0, stream=None):
        batch = q.shape[0]
        self._check(self._lib.faedkv_decode_attn(
            self._h, layer, _ptr(q), _ptr(coefK), _ptr(coefV), _ptr(t_len), batch, float(scale),
            _ptr(out), _stream(stream)))

    def append_decode_attn(self, layer, k_new, v_new, q, coefK, coefV, t_len, out, scale: float = 0.0, stream=None):
        batch = q.shape[0]
        self._check(self._lib.faedkv_append_decode_attn(
            self._h, layer, _ptr(k_new), _ptr(v_new), _ptr(q), batch, _ptr(coefK), _ptr(coefV), _ptr(t_len),
            float(scale), _ptr(out), _stream(stream)))

    def ablate(self, layer, K, V, gain, wsK, wsV, ws_len, K_out, V_out, stream=None):
        batch, T = K.shape[0], K.shape[2]
        self._check(self._lib.faedkv_ablate(
            self._h, layer, _ptr(K), _ptr(V), batch, T, _ptr(gain), _ptr(wsK), _ptr(wsV), _ptr(ws_len),
            _ptr(K_out), _ptr(V_out), _stream(stream)))

    def convert_state(self, layer, coef_in, t_len, from_form, to_form, coef_out=None, stream=None):
        """Stationary sum <-> running mean <-> rotating frame; in place when coef_out is None."""
        coef_out = coef_in if coef_out is None else coef_out
        self._check(self._lib.faedkv_convert_state(
            self._h, layer, _ptr(coef_in), _ptr(t_len), t_len.shape[0], from_form, to_form, _ptr(coef_out),
            _stream(stream)))
        return coef_out

    # -- sink + recent window
    def alloc_window(self, batch: int, device="cuda") -> torch.Tensor:
        """[batch, n_kv_heads, n_sink + ring, head_dim] in the storage type (uninitialised); the ring has
        n_recent slots, or n_recent + n_defer with the block-deferred fold (n_defer >= 2)."""
        ring = self.n_recent + (self.n_defer if self.n_defer > 1 else 0)
        return torch.empty((batch, self.n_kv_heads, self.n_sink + ring, self.head_dim),
                           dtype=self.torch_dtype, device=device)

    def prefill_windowed(self, layer, K, V, coefK, coefV, winK, winV, t_len, stream=None):
        batch, T = K.shape[0], K.shape[2]
        self._check(self._lib.faedkv_prefill_windowed(
            self._h, layer, _ptr(K), _ptr(V), batch, T, _ptr(coefK), _ptr(coefV), _ptr(winK), _ptr(winV),
            _ptr(t_len), _stream(stream)))

    def step_windowed(self, layer, k_new, v_new, q, coefK, coefV, winK, winV, t_len, out, scale: float = 0.0, stream=None):
        batch = q.shape[0]
        self._check(self._lib.faedkv_step_windowed(
            self._h, layer, _ptr(k_new), _ptr(v_new), _ptr(q), batch, _ptr(coefK), _ptr(coefV), _ptr(winK),
            _ptr(winV), _ptr(t_len), float(scale), _ptr(out), _stream(stream)))

    def reconstruct_windowed(self, layer, coefK, coefV, winK, winV, t_len, L: int, K_out=None, V_out=None, stream=None):
        """[sink | reconstructed segment | tokens still in the time domain | zeros] as [batch, n_kv_heads, L, head_dim]."""
        batch = t_len.shape[0]
        shape = (batch, self.n_kv_heads, L, self.head_dim)
        if K_out is None:
            K_out = torch.empty(shape, dtype=self.torch_dtype, device=coefK.device)
        if V_out is None:
            V_out = torch.empty(shape, dtype=self.torch_dtype, device=coefK.device)
        self._check(self._lib.faedkv_reconstruct_windowed(
            self._h, layer, _ptr(coefK), _ptr(coefV), _ptr(winK), _ptr(winV), _ptr(t_len), batch, L, _ptr(K_out),
            _ptr(V_out), _stream(stream)))
        return K_out, V_out

    def launch_count(self) -> int:
        return int(self._lib.faedkv_launch_count(self._h))

    def device_status(self, stream=None) -> int:
        return int(self._lib.faedkv_device_status(self._h, _stream(stream)))

    def debug_word(self, stream=None) -> int:
        """faedkv_debug_word: first failed bounds check of the checked build since the last call (0: none)."""
        return int(self._lib.faedkv_debug_word(self._h, _stream(stream)))

    def reset_device_status(self, stream=None):
        self._check(self._lib.faedkv_reset_device_status(self._h, _stream(stream)))

    def test_hooks(self, wait_limit_ns: int = 0, withhold_step: int = 0):
        """faedkv_test_hooks: wait limit of the tensor-core prefill's bounded waits and the withheld-signal test."""
        self._check(self._lib.faedkv_test_hooks(self._h, int(wait_limit_ns), int(withhold_step)))
