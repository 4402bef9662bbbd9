"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
public header declares, the binding's struct mirrors the header's, and the pure-host entry points
(size arithmetic, status strings, argument rejection) behave."""
import ctypes as C
import os
import re

import numpy as np

from paper_2510_18716_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "ssd_b200.h")


def declared_functions():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(ssd_[a-z0-9_]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    lib = B.load()
    names = declared_functions()
    assert len(names) >= 20 and "ssd_decode_attn" in names
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in the header but not exported"
    assert sorted(B.EXPORTS) == names, "binding and header disagree on the entry points"
    for n in ("ssd_cache_create", "ssd_classify_heads", "ssd_compress", "ssd_append", "ssd_decode_attn",
              "ssd_cache_free"):
        assert n in names


def test_config_struct_matches_header():
    src = open(HEADER).read()
    body = re.search(r"typedef struct ssd_config \{(.*?)\} ssd_config;", src, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = re.findall(r"\b(int32_t|float)\s+([a-z_0-9]+)\s*;", body)
    want = [(n, C.c_int32 if t == "int32_t" else C.c_float) for t, n in fields]
    assert [(n, t) for n, t in B.SsdConfig._fields_] == want
    assert C.sizeof(B.SsdConfig) == 4 * len(want)


def test_status_strings():
    assert B.status_string(0) == "SSD_OK"
    codes = {B.SSD_ERR_INVALID_ARG: "SSD_ERR_INVALID_ARG", B.SSD_ERR_BAD_STATE: "SSD_ERR_BAD_STATE",
             B.SSD_ERR_OVERFLOW: "SSD_ERR_OVERFLOW", B.SSD_ERR_NO_MEM: "SSD_ERR_NO_MEM",
             B.SSD_ERR_CUDA: "SSD_ERR_CUDA", B.SSD_ERR_LIMIT: "SSD_ERR_LIMIT"}
    for c, s in codes.items():
        assert B.status_string(c) == s
    assert B.status_string(-99) == "SSD_ERR_UNKNOWN"


def test_required_bytes_arithmetic():
    # slab bytes = sum over heads of (L + slots) * 512 per sequence; the rest is tables and scratch
    mk = lambda **kw: B.make_config(**{**dict(n_layers=3, n_seqs=4, n_heads=8, prompt_len=16, max_image_tokens=64,
                                              window=8, sink_budget=10, sink_recent=4), **kw})
    c = mk()
    all_spatial = B.required_bytes(c, 0)
    all_sink = B.required_bytes(c, 24)
    worst = B.required_bytes(c, -1)
    assert all_sink - all_spatial == 24 * 4 * ((10 + 4) - 8) * 512
    assert worst == max(all_sink, all_spatial)
    one = B.required_bytes(c, 1)
    assert one - all_spatial == 4 * 6 * 512
    assert B.required_bytes(c, 25) == 0                       # more sink heads than heads
    front = all_spatial - 3 * 8 * 4 * (16 + 8) * 512
    assert 0 < front < 64 << 20 and front % 256 == 0
    for bad in (mk(head_dim=64), mk(n_layers=0), mk(window=0), mk(sink_recent=0), mk(sink_budget=-1),
                mk(n_heads=129), mk(prompt_len=-1), mk(max_image_tokens=0), mk(softmax_scale=-1.0),
                mk(tau=float("nan"))):
        assert B.required_bytes(bad) == 0


def test_null_and_bad_arguments_are_rejected_on_the_host():
    lib = B.load()
    cfg = B.make_config(1, 1, 2, 4, 8, 4, 2, 2)
    h = C.c_void_p()
    assert lib.ssd_cache_create(C.byref(cfg), None, 1 << 20, C.byref(h)) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_cache_create(C.byref(cfg), 256, 1 << 20, None) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_cache_create(C.byref(cfg), 257, 1 << 20, C.byref(h)) == B.SSD_ERR_INVALID_ARG   # misaligned
    assert lib.ssd_cache_create(C.byref(cfg), 256, 16, C.byref(h)) == B.SSD_ERR_NO_MEM
    assert h.value is None
    assert lib.ssd_cache_free(None) == B.SSD_OK
    x = np.zeros(4, np.uint8)
    assert lib.ssd_append(None, 0, x.ctypes.data, x.ctypes.data, None) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_decode_attn(None, 0, x.ctypes.data, x.ctypes.data, None) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_compress(None, 0, None, x.ctypes.data, x.ctypes.data, 0, 0, None) == B.SSD_ERR_INVALID_ARG
    p = x.ctypes.data
    assert lib.ssd_append_decode(None, 0, p, p, p, p, None) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_append_decode_layers(None, 0, 1, p, p, p, p, None) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_step_host(None, 0, p, p, p, p, None) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_step_host_layers(None, 0, 1, p, p, p, p, None) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_recompress(None, 0, None) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_recompress_layers(None, 0, 1, None) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_decode_attn_static(None, 0, p, p, None) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_cache_max_slots(None) == -1
    assert lib.ssd_cache_tokens(None, 0) == -1
    assert isinstance(B.kernel_launch_count(), int)


def test_threshold_rule_exports_need_no_gpu():
    """Sec. 3.3: s = ratio sum / (P * N) in float32, semantic iff s > tau (equality is spatial); host arithmetic."""
    lib = B.load()
    P, N = 3, 10
    sums = np.array([0.45 * P * N, 0.46 * P * N, 0.0, float(P * N)], np.float64)
    s, lab = B.labels_from_ratio_sums(sums, P, N, 0.45)
    assert s.dtype == np.float32 and lab.tolist() == [int(np.float32(0.45 * P * N / (P * N)) > np.float32(0.45)), 1, 0, 1]
    assert np.array_equal(s, (sums / (P * N)).astype(np.float32))
    assert B.labels_from_sparsity(np.array([0.45, 0.4500001, 0.2], np.float32), 0.45).tolist() == [0, 1, 0]
    x = np.zeros(4, np.float64)
    out = np.zeros(4, np.uint8)
    assert lib.ssd_labels_from_ratio_sums(None, 4, 1, 1, C.c_float(0.5), None, out.ctypes.data) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_labels_from_ratio_sums(x.ctypes.data, 4, 0, 1, C.c_float(0.5), None, out.ctypes.data) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_labels_from_ratio_sums(x.ctypes.data, 4, 1, 1, C.c_float(float("nan")), None, out.ctypes.data) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_labels_from_sparsity(None, 4, C.c_float(0.5), out.ctypes.data) == B.SSD_ERR_INVALID_ARG
    p = x.ctypes.data
    assert lib.ssd_kv_token_mse(None, p, p, p, 1, p, None) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_quantize_rows_e4m3(None, 1, p, p, None) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_cache_set_kv_format(None, 1) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_cache_get_compress_scores(None, 0, p) == B.SSD_ERR_INVALID_ARG
