"""ctypes binding of the C ABI in ``include/ssd_b200.h`` -- argument marshalling only.

Every step of the path runs inside the CUDA library.  If the library is missing or cannot be
loaded this module raises; there is no CPU fallback.  torch is used for device memory and the
current stream, nothing else.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

from . import build as _build

SSD_OK = 0
SSD_ERR_INVALID_ARG = -1
SSD_ERR_BAD_STATE = -2
SSD_ERR_OVERFLOW = -3
SSD_ERR_NO_MEM = -4
SSD_ERR_CUDA = -5
SSD_ERR_LIMIT = -6

EXPORTS = [
    "ssd_status_string", "ssd_cache_required_bytes", "ssd_cache_create", "ssd_cache_free",
    "ssd_classify_heads", "ssd_classify_partial", "ssd_set_head_labels", "ssd_compress", "ssd_append",
    "ssd_decode_attn", "ssd_append_decode_layers", "ssd_recompress_layers", "ssd_step_host", "ssd_step_host_layers", "ssd_cache_get_indices", "ssd_cache_max_slots",
    "ssd_cache_get_lengths", "ssd_cache_get_labels", "ssd_cache_tokens", "ssd_cache_rewind",
    "ssd_cache_kv_bytes", "ssd_kernel_launch_count", "ssd_profile_enable", "ssd_profile_collect",
    "ssd_cache_device_status", "ssd_debug_decode_plan", "ssd_decode_attn_static",
    "ssd_cache_set_row_buffer", "ssd_recompress", "ssd_cache_get_scores", "ssd_append_decode",
    "ssd_labels_from_ratio_sums", "ssd_labels_from_sparsity", "ssd_cache_get_compress_scores", "ssd_kv_token_mse",
    "ssd_cache_set_kv_format", "ssd_quantize_rows_e4m3",
]


class SsdConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "n_layers", "n_seqs", "n_heads", "head_dim", "prompt_len", "max_image_tokens", "window",
        "sink_budget", "sink_recent", "cls_window")] + [("tau", C.c_float), ("softmax_scale", C.c_float)]


class SsdError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {status_string(code)} ({code})")


_lib = None


def lib_path() -> str:
    return _build.LIB


def load():
    """Load (building first if the sources are newer) the CUDA library.  Raises if impossible."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    if not os.path.exists(path):
        path = _build.build()
    L = C.CDLL(path)
    vp, i32, u64 = C.c_void_p, C.c_int32, C.c_uint64
    cfgp = C.POINTER(SsdConfig)
    L.ssd_status_string.argtypes = [C.c_int]
    L.ssd_status_string.restype = C.c_char_p
    L.ssd_cache_required_bytes.argtypes = [cfgp, i32]
    L.ssd_cache_required_bytes.restype = C.c_size_t
    L.ssd_cache_create.argtypes = [cfgp, vp, C.c_size_t, C.POINTER(vp)]
    L.ssd_cache_free.argtypes = [vp]
    L.ssd_classify_heads.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp]
    L.ssd_classify_partial.argtypes = [vp, vp, vp, i32, i32, vp, vp]
    L.ssd_set_head_labels.argtypes = [vp, vp]
    L.ssd_compress.argtypes = [vp, i32, vp, vp, vp, i32, i32, vp]
    L.ssd_append.argtypes = [vp, i32, vp, vp, vp]
    L.ssd_decode_attn.argtypes = [vp, i32, vp, vp, vp]
    L.ssd_decode_attn_static.argtypes = [vp, i32, vp, vp, vp]
    L.ssd_append_decode.argtypes = [vp, i32, vp, vp, vp, vp, vp]
    L.ssd_cache_set_row_buffer.argtypes = [vp, i32]
    L.ssd_labels_from_ratio_sums.argtypes = [vp, C.c_int64, i32, i32, C.c_float, vp, vp]
    L.ssd_labels_from_sparsity.argtypes = [vp, C.c_int64, C.c_float, vp]
    L.ssd_recompress.argtypes = [vp, i32, vp]
    L.ssd_cache_get_scores.argtypes = [vp, i32, vp]
    L.ssd_cache_get_compress_scores.argtypes = [vp, i32, vp]
    L.ssd_kv_token_mse.argtypes = [vp, vp, vp, vp, C.c_int64, vp, vp]
    L.ssd_cache_set_kv_format.argtypes = [vp, i32]
    L.ssd_quantize_rows_e4m3.argtypes = [vp, C.c_int64, vp, vp, vp]
    L.ssd_step_host.argtypes = [vp, i32, vp, vp, vp, vp, vp]
    L.ssd_append_decode_layers.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp]
    L.ssd_recompress_layers.argtypes = [vp, i32, i32, vp]
    L.ssd_step_host_layers.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp]
    L.ssd_cache_get_indices.argtypes = [vp, i32, vp]
    L.ssd_cache_max_slots.argtypes = [vp]
    L.ssd_cache_max_slots.restype = i32
    L.ssd_cache_get_lengths.argtypes = [vp, i32, vp]
    L.ssd_cache_get_labels.argtypes = [vp, vp]
    L.ssd_cache_tokens.argtypes = [vp, i32]
    L.ssd_cache_tokens.restype = i32
    L.ssd_cache_rewind.argtypes = [vp, i32, i32]
    L.ssd_cache_kv_bytes.argtypes = [vp, C.POINTER(C.c_size_t)]
    L.ssd_profile_enable.argtypes = [vp, i32]
    L.ssd_profile_collect.argtypes = [vp, vp, C.POINTER(i32)]
    L.ssd_cache_device_status.argtypes = [vp, C.POINTER(C.c_uint32)]
    L.ssd_debug_decode_plan.argtypes = [i32, vp, i32, i32, i32, i32, i32, i32, i32, vp, C.c_int64]
    L.ssd_debug_decode_plan.restype = C.c_int64
    L.ssd_kernel_launch_count.argtypes = []
    L.ssd_kernel_launch_count.restype = u64
    for n in EXPORTS:
        f = getattr(L, n)
        if f.restype is C.c_int and n not in ("ssd_cache_max_slots", "ssd_cache_tokens"):
            f.restype = C.c_int
    _lib = L
    return L


def status_string(code: int) -> str:
    return load().ssd_status_string(int(code)).decode()


def kernel_launch_count() -> int:
    return int(load().ssd_kernel_launch_count())


def make_config(n_layers, n_seqs, n_heads, prompt_len, max_image_tokens, window, sink_budget,
                sink_recent, cls_window=32, tau=0.45, softmax_scale=0.0, head_dim=128) -> SsdConfig:
    return SsdConfig(n_layers, n_seqs, n_heads, head_dim, prompt_len, max_image_tokens, window,
                     sink_budget, sink_recent, cls_window, tau, softmax_scale)


def config_from_workload(w, n_layers: Optional[int] = None, n_seqs: Optional[int] = None) -> SsdConfig:
    return make_config(n_layers or w.n_layers, n_seqs or w.n_seqs, w.n_heads, w.prompt_len, w.n_img,
                       w.window, w.sink_budget, w.sink_recent, w.cls_window, w.tau)


def labels_from_ratio_sums(total_sums, n_cal_total: int, n_img: int, tau: float):
    """(s float32, labels uint8), both shaped like total_sums: the library's threshold rule (Sec. 3.3)."""
    sums = np.ascontiguousarray(total_sums, np.float64)
    s = np.empty(sums.shape, np.float32)
    lab = np.empty(sums.shape, np.uint8)
    rc = load().ssd_labels_from_ratio_sums(sums.ctypes.data, sums.size, int(n_cal_total), int(n_img), float(tau),
                                           s.ctypes.data, lab.ctypes.data)
    if rc != SSD_OK:
        raise SsdError(rc, "ssd_labels_from_ratio_sums")
    return s, lab


def labels_from_sparsity(s, tau: float):
    """labels uint8 shaped like s: semantic iff s > tau, decided by the library in float32."""
    s32 = np.ascontiguousarray(s, np.float32)
    lab = np.empty(s32.shape, np.uint8)
    rc = load().ssd_labels_from_sparsity(s32.ctypes.data, s32.size, float(tau), lab.ctypes.data)
    if rc != SSD_OK:
        raise SsdError(rc, "ssd_labels_from_sparsity")
    return lab


def kv_token_mse(k_a: torch.Tensor, v_a: torch.Tensor, k_b: torch.Tensor, v_b: torch.Tensor,
                 out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Per-token divergence of two KV caches (Sec. 3.2): tensors [..., 128] bf16 on one CUDA device, all
    of one shape; returns float32 [...] on that device."""
    shape = tuple(k_a.shape)
    for t in (k_a, v_a, k_b, v_b):
        if not (t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous() and tuple(t.shape) == shape and shape[-1] == 128):
            raise ValueError("kv_token_mse: want four contiguous CUDA bf16 tensors [..., 128] of one shape")
    if out is None:
        out = torch.empty(shape[:-1], dtype=torch.float32, device=k_a.device)
    n_rows = k_a.numel() // 128
    assert out.is_cuda and out.dtype == torch.float32 and out.is_contiguous() and out.numel() == n_rows
    with torch.cuda.device(k_a.device):
        rc = load().ssd_kv_token_mse(k_a.data_ptr(), v_a.data_ptr(), k_b.data_ptr(), v_b.data_ptr(), n_rows,
                                     out.data_ptr(), _stream())
    if rc != SSD_OK:
        raise SsdError(rc, "ssd_kv_token_mse")
    return out


def quantize_rows_e4m3(rows: torch.Tensor):
    """The library's 8-bit row quantiser: rows [..., 128] bf16 on a CUDA device -> (codes uint8 [..., 128],
    scales float32 [...])."""
    if not (rows.is_cuda and rows.dtype == torch.bfloat16 and rows.is_contiguous() and rows.shape[-1] == 128):
        raise ValueError("quantize_rows_e4m3: want a contiguous CUDA bf16 tensor [..., 128]")
    codes = torch.empty(rows.shape, dtype=torch.uint8, device=rows.device)
    scales = torch.empty(rows.shape[:-1], dtype=torch.float32, device=rows.device)
    with torch.cuda.device(rows.device):
        rc = load().ssd_quantize_rows_e4m3(rows.data_ptr(), rows.numel() // 128, codes.data_ptr(), scales.data_ptr(), _stream())
    if rc != SSD_OK:
        raise SsdError(rc, "ssd_quantize_rows_e4m3")
    return codes, scales


def required_bytes(cfg: SsdConfig, n_sink_heads_total: int = -1) -> int:
    return int(load().ssd_cache_required_bytes(C.byref(cfg), int(n_sink_heads_total)))


def _stream() -> int:
    return int(torch.cuda.current_stream().cuda_stream)


def _dev(t: torch.Tensor, shape, what: str) -> int:
    if not (t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous() and tuple(t.shape) == tuple(shape)):
        raise ValueError(f"{what}: want contiguous CUDA bf16 {tuple(shape)}, got {t.dtype} {tuple(t.shape)} on {t.device}")
    return t.data_ptr()


class SsdCache:
    """Python handle of an ``ssd_cache`` (one GPU, one stream at a time)."""

    def __init__(self, cfg: SsdConfig, n_sink_heads_total: int = -1, device="cuda:0"):
        self._h = None
        self.lib = load()
        self.cfg = cfg
        nbytes = required_bytes(cfg, n_sink_heads_total)
        if nbytes == 0:
            raise SsdError(SSD_ERR_INVALID_ARG, "ssd_cache_required_bytes")
        if not torch.cuda.is_available():
            raise RuntimeError("ssd_b200 needs a CUDA device; there is no CPU path")
        self.device = torch.device(device)
        self.mem = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = (self.mem.data_ptr() + 255) // 256 * 256
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            rc = self.lib.ssd_cache_create(C.byref(cfg), base, nbytes, C.byref(h))
        if rc != SSD_OK:
            raise SsdError(rc, "ssd_cache_create")
        self._h = h
        self.nbytes = nbytes

    # -- lifetime
    def close(self):
        if self._h is not None:
            self.lib.ssd_cache_free(self._h)
            self._h = None
            self.mem = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc, what):
        if rc != SSD_OK:
            raise SsdError(rc, what)

    # -- labels
    def set_head_labels(self, labels):
        lab = np.ascontiguousarray(labels, np.uint8).reshape(-1)
        assert lab.size == self.cfg.n_layers * self.cfg.n_heads
        self._check(self.lib.ssd_set_head_labels(self._h, lab.ctypes.data), "ssd_set_head_labels")

    def classify_heads(self, q_cal: torch.Tensor, k_cal: torch.Tensor):
        c = self.cfg
        P, n_img = q_cal.shape[1], q_cal.shape[3]
        qp = _dev(q_cal, (c.n_layers, P, c.n_heads, n_img, c.head_dim), "q_cal")
        kp = _dev(k_cal, (c.n_layers, P, c.n_heads, c.prompt_len + n_img, c.head_dim), "k_cal")
        s = np.empty(c.n_layers * c.n_heads, np.float32)
        lab = np.empty(c.n_layers * c.n_heads, np.uint8)
        self._check(self.lib.ssd_classify_heads(self._h, qp, kp, P, n_img, s.ctypes.data, lab.ctypes.data,
                                                _stream()), "ssd_classify_heads")
        return s.reshape(c.n_layers, c.n_heads), lab.reshape(c.n_layers, c.n_heads)

    def classify_partial(self, q_cal: torch.Tensor, k_cal: torch.Tensor):
        c = self.cfg
        P, n_img = q_cal.shape[1], q_cal.shape[3]
        qp = _dev(q_cal, (c.n_layers, P, c.n_heads, n_img, c.head_dim), "q_cal")
        kp = _dev(k_cal, (c.n_layers, P, c.n_heads, c.prompt_len + n_img, c.head_dim), "k_cal")
        sums = np.empty(c.n_layers * c.n_heads, np.float64)
        self._check(self.lib.ssd_classify_partial(self._h, qp, kp, P, n_img, sums.ctypes.data, _stream()),
                    "ssd_classify_partial")
        return sums.reshape(c.n_layers, c.n_heads)

    # -- hot path
    def compress(self, layer: int, q_obs: Optional[torch.Tensor], k_full: torch.Tensor, v_full: torch.Tensor,
                 n0: int, n_obs: Optional[int] = None):
        c = self.cfg
        n_obs = (0 if q_obs is None else q_obs.shape[2]) if n_obs is None else n_obs
        qp = None if q_obs is None else _dev(q_obs, (c.n_seqs, c.n_heads, n_obs, c.head_dim), "q_obs")
        kp = _dev(k_full, (c.n_seqs, c.n_heads, c.prompt_len + n0, c.head_dim), "k_full")
        vp = _dev(v_full, (c.n_seqs, c.n_heads, c.prompt_len + n0, c.head_dim), "v_full")
        self._check(self.lib.ssd_compress(self._h, layer, qp, kp, vp, n0, n_obs, _stream()), "ssd_compress")

    def append(self, layer: int, k_new: torch.Tensor, v_new: torch.Tensor):
        c = self.cfg
        shp = (c.n_seqs, c.n_heads, c.head_dim)
        self._check(self.lib.ssd_append(self._h, layer, _dev(k_new, shp, "k_new"), _dev(v_new, shp, "v_new"),
                                        _stream()), "ssd_append")

    def decode_attn(self, layer: int, q: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        c = self.cfg
        shp = (c.n_seqs, c.n_heads, c.head_dim)
        if out is None:
            out = torch.empty(shp, dtype=torch.bfloat16, device=q.device)
        self._check(self.lib.ssd_decode_attn(self._h, layer, _dev(q, shp, "q"), _dev(out, shp, "out"), _stream()),
                    "ssd_decode_attn")
        return out

    def append_decode(self, layer: int, k_new: torch.Tensor, v_new: torch.Tensor, q: torch.Tensor,
                      out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """append + decode_attn of one layer in a single launch."""
        c = self.cfg
        shp = (c.n_seqs, c.n_heads, c.head_dim)
        if out is None:
            out = torch.empty(shp, dtype=torch.bfloat16, device=q.device)
        self._check(self.lib.ssd_append_decode(self._h, layer, _dev(k_new, shp, "k_new"), _dev(v_new, shp, "v_new"),
                                               _dev(q, shp, "q"), _dev(out, shp, "out"), _stream()), "ssd_append_decode")
        return out

    def append_decode_layers(self, first_layer: int, k_new: torch.Tensor, v_new: torch.Tensor, q: torch.Tensor,
                             out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """append + decode_attn of q.shape[0] consecutive layers in one launch; tensors
        [n_layers, n_seqs, n_heads, head_dim]."""
        c = self.cfg
        shp = (q.shape[0], c.n_seqs, c.n_heads, c.head_dim)
        if out is None:
            out = torch.empty(shp, dtype=torch.bfloat16, device=q.device)
        self._check(self.lib.ssd_append_decode_layers(self._h, first_layer, shp[0], _dev(k_new, shp, "k_new"),
                                                      _dev(v_new, shp, "v_new"), _dev(q, shp, "q"), _dev(out, shp, "out"),
                                                      _stream()), "ssd_append_decode_layers")
        return out

    def decode_attn_static(self, layer: int, q: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """decode_attn with the kernel's scratch in the library's built-in array (allocates nothing
        inside the library; `out` should be passed by callers that must not allocate at all)."""
        c = self.cfg
        shp = (c.n_seqs, c.n_heads, c.head_dim)
        if out is None:
            out = torch.empty(shp, dtype=torch.bfloat16, device=q.device)
        self._check(self.lib.ssd_decode_attn_static(self._h, layer, _dev(q, shp, "q"), _dev(out, shp, "out"),
                                                    _stream()), "ssd_decode_attn_static")
        return out

    def set_kv_format(self, fmt: int):
        """0: bf16 rows (default); 1: 8-bit rows (E4M3 codes and a float32 scale per row)."""
        self._check(self.lib.ssd_cache_set_kv_format(self._h, int(fmt)), "ssd_cache_set_kv_format")

    # -- Algorithm 2 (row buffer)
    def set_row_buffer(self, enable: bool = True):
        self._check(self.lib.ssd_cache_set_row_buffer(self._h, 1 if enable else 0), "ssd_cache_set_row_buffer")

    def recompress(self, layer: int):
        self._check(self.lib.ssd_recompress(self._h, layer, _stream()), "ssd_recompress")

    def recompress_layers(self, first_layer: int, n_layers: int):
        self._check(self.lib.ssd_recompress_layers(self._h, first_layer, n_layers, _stream()), "ssd_recompress_layers")

    def get_scores(self, layer: int) -> np.ndarray:
        c = self.cfg
        a = np.empty((c.n_seqs, c.n_heads, c.sink_budget + c.sink_recent), np.float32)
        self._check(self.lib.ssd_cache_get_scores(self._h, layer, a.ctypes.data), "ssd_cache_get_scores")
        return a

    def get_compress_scores(self, layer: int, n0: int) -> np.ndarray:
        """Scores of the latest compress call (which must have been on `layer`, at n0 image tokens)."""
        c = self.cfg
        a = np.empty((c.n_seqs, c.n_heads, n0), np.float32)
        self._check(self.lib.ssd_cache_get_compress_scores(self._h, layer, a.ctypes.data), "ssd_cache_get_compress_scores")
        return a

    def step_host(self, layer: int, q_host, k_new_host, v_new_host, out_host):
        """One append + decode of a layer from (pinned) host bf16 tensors; asynchronous."""
        for t in (q_host, k_new_host, v_new_host, out_host):
            assert (not t.is_cuda) and t.dtype == torch.bfloat16 and t.is_contiguous()
        self._check(self.lib.ssd_step_host(self._h, layer, q_host.data_ptr(), k_new_host.data_ptr(),
                                           v_new_host.data_ptr(), out_host.data_ptr(), _stream()), "ssd_step_host")

    def step_host_layers(self, first_layer: int, q_host, k_new_host, v_new_host, out_host):
        """Append + decode of q_host.shape[0] consecutive layers from (pinned) host bf16 tensors
        [n_layers, n_seqs, n_heads, head_dim], copies overlapped with the kernels; asynchronous."""
        n = q_host.shape[0]
        for t in (q_host, k_new_host, v_new_host, out_host):
            assert (not t.is_cuda) and t.dtype == torch.bfloat16 and t.is_contiguous() and t.shape[0] == n
        self._check(self.lib.ssd_step_host_layers(self._h, first_layer, n, q_host.data_ptr(), k_new_host.data_ptr(),
                                                  v_new_host.data_ptr(), out_host.data_ptr(), _stream()),
                    "ssd_step_host_layers")

    # -- inspection
    def max_slots(self) -> int:
        return int(self.lib.ssd_cache_max_slots(self._h))

    def get_indices(self, layer: int) -> np.ndarray:
        c = self.cfg
        idx = np.empty((c.n_seqs, c.n_heads, self.max_slots()), np.int32)
        self._check(self.lib.ssd_cache_get_indices(self._h, layer, idx.ctypes.data), "ssd_cache_get_indices")
        return idx

    def get_lengths(self, layer: int) -> np.ndarray:
        ln = np.empty(self.cfg.n_heads, np.int32)
        self._check(self.lib.ssd_cache_get_lengths(self._h, layer, ln.ctypes.data), "ssd_cache_get_lengths")
        return ln

    def get_labels(self) -> np.ndarray:
        lab = np.empty(self.cfg.n_layers * self.cfg.n_heads, np.uint8)
        self._check(self.lib.ssd_cache_get_labels(self._h, lab.ctypes.data), "ssd_cache_get_labels")
        return lab.reshape(self.cfg.n_layers, self.cfg.n_heads)

    def tokens(self, layer: int) -> int:
        return int(self.lib.ssd_cache_tokens(self._h, layer))

    def rewind(self, layer: int, t: int):
        self._check(self.lib.ssd_cache_rewind(self._h, layer, t), "ssd_cache_rewind")

    def profile_enable(self, max_launches: int):
        self._prof_cap = int(max_launches)
        self._check(self.lib.ssd_profile_enable(self._h, int(max_launches)), "ssd_profile_enable")

    def profile_collect(self) -> np.ndarray:
        ms = np.empty(max(getattr(self, "_prof_cap", 0), 1), np.float32)
        n = C.c_int32(0)
        self._check(self.lib.ssd_profile_collect(self._h, ms.ctypes.data, C.byref(n)), "ssd_profile_collect")
        return ms[: n.value].copy()

    def device_status(self) -> int:
        v = C.c_uint32(0)
        self._check(self.lib.ssd_cache_device_status(self._h, C.byref(v)), "ssd_cache_device_status")
        return int(v.value)

    def kv_bytes_per_seq(self) -> int:
        v = C.c_size_t(0)
        self._check(self.lib.ssd_cache_kv_bytes(self._h, C.byref(v)), "ssd_cache_kv_bytes")
        return int(v.value)


def decode_plan(head_recs, prompt_len, n_seqs, prompt_valid, static_valid, t_img, max_workers, chunk=0):
    """Copies one decode launch would issue (host-side enumeration): int64 [n, 6] rows of
    (worker, chunk, source slot, destination slot, slots, sequence * n_heads + head)."""
    recs = np.ascontiguousarray(head_recs, np.int32).reshape(-1, 4)
    args = (recs.shape[0], recs.ctypes.data, prompt_len, n_seqs, prompt_valid, static_valid, t_img, max_workers, chunk)
    n = int(load().ssd_debug_decode_plan(*args, None, 0))
    if n < 0:
        raise SsdError(n, "ssd_debug_decode_plan")
    out = np.empty((max(n, 1), 6), np.int64)
    n2 = int(load().ssd_debug_decode_plan(*args, out.ctypes.data, n))
    assert n2 == n
    return out[:n]
