"""fp64 CPU oracle for the SSD hot path -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper around ``ssd_oracle.c`` (plain C, double precision, written
from the paper), plus a few functions in plain numpy: the buffered variant of the
method (Algorithm 2), the per-token divergence of two caches (Sec. 3.2) and the
8-bit K/V extension (E4M3 encode / decode from the format's definition, per-row
quantisation, attention over dequantised rows).  Only the tests, the smoke check
and the benchmark's CPU-baseline leg may import this package; the CUDA library
never does, and this package never imports the CUDA library.  bf16 tensors travel
as numpy ``uint16`` bit patterns.

Every function cites the passage of the paper it follows in ``ssd_oracle.c``.
Parity status: all functions are pinned by ``tests/test_oracle_pins.py``
(closed forms, brute force, special cases, a library routine); none is
"parity unpinned".
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ssd_oracle.c")
_LIB = os.path.join(_HERE, "libssd_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP over independent pairs)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _p(a, ty):
    return a.ctypes.data_as(C.POINTER(ty))


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_LIB)
        u16p, f64p, i32p, u8p = (C.POINTER(C.c_uint16), C.POINTER(C.c_double),
                                 C.POINTER(C.c_int32), C.POINTER(C.c_uint8))
        L.ssd_oracle_attention_row.argtypes = [u16p, u16p, C.c_int, C.c_int, C.c_double, f64p]
        L.ssd_oracle_attention_row.restype = None
        L.ssd_oracle_sparsity_sum.argtypes = [u16p, u16p, C.c_int, C.c_int, C.c_int, C.c_int,
                                              C.c_double]
        L.ssd_oracle_sparsity_sum.restype = C.c_double
        L.ssd_oracle_sparsity.argtypes = [u16p, u16p] + [C.c_int] * 7 + [C.c_double, f64p]
        L.ssd_oracle_sparsity.restype = None
        L.ssd_oracle_labels.argtypes = [f64p, C.c_int, C.c_double, u8p]
        L.ssd_oracle_labels.restype = None
        L.ssd_oracle_scores.argtypes = [u16p, u16p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_double,
                                        f64p, f64p]
        L.ssd_oracle_scores.restype = None
        L.ssd_oracle_topm.argtypes = [f64p, C.c_int, C.c_int, i32p]
        L.ssd_oracle_topm.restype = C.c_int
        L.ssd_oracle_retained_set.argtypes = [C.c_int] * 5 + [i32p, C.c_int, i32p]
        L.ssd_oracle_retained_set.restype = C.c_int
        L.ssd_oracle_attend.argtypes = [u16p, u16p, u16p, C.c_int, i32p, C.c_int, C.c_double, f64p,
                                        f64p]
        L.ssd_oracle_attend.restype = None
        L.ssd_oracle_select_batch.argtypes = [u16p, u16p, u8p, C.c_long] + [C.c_int] * 7 + [
            C.c_double, f64p, i32p, i32p]
        L.ssd_oracle_select_batch.restype = None
        L.ssd_oracle_decode_batch.argtypes = [u16p, u16p, u16p, u8p, i32p, i32p, C.c_long] + [
            C.c_int] * 7 + [C.c_double, C.c_int, f64p]
        L.ssd_oracle_decode_batch.restype = None
        L.ssd_oracle_threads.argtypes = []
        L.ssd_oracle_threads.restype = C.c_int
        _lib = L
    return _lib


def threads() -> int:
    return int(lib().ssd_oracle_threads())


def default_scale(D: int) -> float:
    return 1.0 / float(np.sqrt(np.float64(D)))


def attention_row(q, K, scale=None):
    """a = softmax(scale * K q) over all rows of K.  q [D], K [n_ctx, D] (uint16 bf16)."""
    q, K = _u16(q), _u16(K)
    n, D = K.shape
    out = np.empty(n, np.float64)
    lib().ssd_oracle_attention_row(_p(q, C.c_uint16), _p(K, C.c_uint16), n, D,
                                   default_scale(D) if scale is None else scale, _p(out, C.c_double))
    return out


def sparsity(Q_cal, K_cal, L, w, scale=None):
    """s[l,h] of Sec. 3.3.  Q_cal [layers,P,H,N,D], K_cal [layers,P,H,L+N,D] -> [layers,H]."""
    Q_cal, K_cal = _u16(Q_cal), _u16(K_cal)
    nl, P, H, N, D = Q_cal.shape
    assert K_cal.shape == (nl, P, H, L + N, D), (K_cal.shape, (nl, P, H, L + N, D))
    s = np.empty((nl, H), np.float64)
    lib().ssd_oracle_sparsity(_p(Q_cal, C.c_uint16), _p(K_cal, C.c_uint16), nl, P, H, L, N, D, w,
                              default_scale(D) if scale is None else scale, _p(s, C.c_double))
    return s


def sparsity_sum(Q, K, L, w, scale=None):
    """Inner sum over t of the ratio for one (layer, head, prompt).  Q [N,D], K [L+N,D]."""
    Q, K = _u16(Q), _u16(K)
    N, D = Q.shape
    assert K.shape == (L + N, D)
    return float(lib().ssd_oracle_sparsity_sum(_p(Q, C.c_uint16), _p(K, C.c_uint16), L, N, D, w,
                                               default_scale(D) if scale is None else scale))


def labels(s, tau):
    """1 = Semantic iff s > tau (equality is Spatial)."""
    s = np.ascontiguousarray(s, np.float64)
    out = np.empty(s.shape, np.uint8)
    lib().ssd_oracle_labels(_p(s, C.c_double), s.size, float(tau), _p(out, C.c_uint8))
    return out


def scores(Q_obs, K, L, n0, scale=None, return_prompt_mass=False):
    """Accumulated post-softmax score per image token.  Q_obs [n_obs,D], K [L+n0,D] -> [n0]."""
    Q_obs, K = _u16(Q_obs), _u16(K)
    n_obs, D = Q_obs.shape
    assert K.shape[0] >= L + n0 and K.shape[1] == D
    sc = np.empty(n0, np.float64)
    pm = C.c_double(0.0)
    lib().ssd_oracle_scores(_p(Q_obs, C.c_uint16), _p(K, C.c_uint16), L, n0, n_obs, D,
                            default_scale(D) if scale is None else scale, _p(sc, C.c_double),
                            C.byref(pm))
    return (sc, pm.value) if return_prompt_mass else sc


def topm(score, n_cand, M):
    """Indices (ascending) of the min(M, n_cand) largest of score[:n_cand]; ties -> lowest index."""
    score = np.ascontiguousarray(score, np.float64)
    assert score.size >= n_cand
    idx = np.empty(max(M, 1), np.int32)
    c = lib().ssd_oracle_topm(_p(score, C.c_double), int(n_cand), int(M), _p(idx, C.c_int32))
    return idx[:c].copy()


def retained_set(is_semantic, L, t, W, R, top_idx=None):
    """Absolute positions a head holds after image token t-1 was appended (ascending)."""
    top = np.ascontiguousarray(top_idx if top_idx is not None else np.zeros(0), np.int32)
    pos = np.empty(L + t + top.size + 1, np.int32)
    n = lib().ssd_oracle_retained_set(int(bool(is_semantic)), L, t, W, R, _p(top, C.c_int32),
                                      top.size, _p(pos, C.c_int32))
    return pos[:n].copy()


def attend(q, K_hist, V_hist, pos, scale=None, return_weights=False):
    """softmax attention of q over the given positions of the full history -> out [D] fp64."""
    q, K_hist, V_hist = _u16(q), _u16(K_hist), _u16(V_hist)
    pos = np.ascontiguousarray(pos, np.int32)
    D = q.shape[0]
    out = np.empty(D, np.float64)
    wts = np.empty(max(pos.size, 1), np.float64)
    lib().ssd_oracle_attend(_p(q, C.c_uint16), _p(K_hist, C.c_uint16), _p(V_hist, C.c_uint16), D,
                            _p(pos, C.c_int32), pos.size,
                            default_scale(D) if scale is None else scale, _p(out, C.c_double),
                            _p(wts, C.c_double))
    return (out, wts[:pos.size]) if return_weights else out


def select_batch(Q_obs, K, is_semantic, L, n0, M, R, scale=None):
    """Scores and top-M for many pairs.

    Q_obs [..., n_obs, D], K [..., L+n_keys, D] (n_keys >= n0), is_semantic [...] uint8.
    Returns (score [..., n0] fp64, idx [..., M] int32 padded with -1, cnt [...] int32).
    """
    Q_obs, K = _u16(Q_obs), _u16(K)
    lead = Q_obs.shape[:-2]
    n_obs, D = Q_obs.shape[-2:]
    n_keys = K.shape[-2] - L
    assert K.shape[:-2] == lead and n_keys >= n0
    sem = np.ascontiguousarray(np.broadcast_to(is_semantic, lead), np.uint8)
    n_pairs = int(np.prod(lead)) if lead else 1
    sc = np.zeros(lead + (max(n0, 0),), np.float64)
    idx = np.full(lead + (M,), -1, np.int32)
    cnt = np.zeros(lead, np.int32)
    lib().ssd_oracle_select_batch(_p(Q_obs, C.c_uint16), _p(K, C.c_uint16), _p(sem, C.c_uint8),
                                  n_pairs, L, n_keys, n0, n_obs, D, M, R,
                                  default_scale(D) if scale is None else scale, _p(sc, C.c_double),
                                  _p(idx, C.c_int32), _p(cnt, C.c_int32))
    return sc, idx, cnt


def decode_batch(q, K_hist, V_hist, is_semantic, idx, cnt, L, t, W, M, R, scale=None, full=False):
    """Decode attention at image step t for many pairs -> out [..., D] fp64.

    q [..., D]; K_hist, V_hist [..., L+n_keys, D] with n_keys >= t; idx [..., M], cnt [...].
    """
    q, K_hist, V_hist = _u16(q), _u16(K_hist), _u16(V_hist)
    lead = q.shape[:-1]
    D = q.shape[-1]
    n_keys = K_hist.shape[-2] - L
    assert K_hist.shape[:-2] == lead and V_hist.shape == K_hist.shape and n_keys >= t
    sem = np.ascontiguousarray(np.broadcast_to(is_semantic, lead), np.uint8)
    n_pairs = int(np.prod(lead)) if lead else 1
    if idx is None:
        idx = np.full(lead + (M,), -1, np.int32)
        cnt = np.zeros(lead, np.int32)
    idx = np.ascontiguousarray(idx, np.int32)
    cnt = np.ascontiguousarray(cnt, np.int32)
    assert idx.shape == lead + (M,) and cnt.shape == lead
    out = np.empty(lead + (D,), np.float64)
    lib().ssd_oracle_decode_batch(_p(q, C.c_uint16), _p(K_hist, C.c_uint16), _p(V_hist, C.c_uint16),
                                  _p(sem, C.c_uint8), _p(idx, C.c_int32), _p(cnt, C.c_int32), n_pairs,
                                  L, n_keys, t, D, W, M, R,
                                  default_scale(D) if scale is None else scale, int(bool(full)),
                                  _p(out, C.c_double))
    return out


def _widen(a):
    """bf16 bit patterns (uint16) -> float64, exactly."""
    return (_u16(a).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def kv_token_mse(K_a, V_a, K_b, V_b):
    """Per-token divergence of two KV caches (Sec. 3.2, the MSE_token equation):
    out[..., j] = ||K_a[..., j, :] - K_b[..., j, :]||^2 + ||V_a[..., j, :] - V_b[..., j, :]||^2.

    Inputs [..., T, D] uint16 bf16 bit patterns, all of one shape (the paper's two caches are the
    CFG branch and the native branch of one prompt); output [..., T] float64.  The equation has no
    1/D in it although it is called a mean; it is written out as printed."""
    Ka, Va, Kb, Vb = _widen(K_a), _widen(V_a), _widen(K_b), _widen(V_b)
    assert Ka.shape == Va.shape == Kb.shape == Vb.shape
    dk, dv = Ka - Kb, Va - Vb
    return (dk * dk).sum(-1) + (dv * dv).sum(-1)


# ---- 8-bit K/V (an extension the paper only cites as related work, Sec. 2 "KV Cache Compression")
# Format: OCP 8-bit floating point, E4M3 (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; no
# infinities, S.1111.111 is NaN, largest finite magnitude 448, subnormals 2^-6 * m/8).

def e4m3_decode(codes):
    """E4M3 bit patterns (uint8) -> float64, from the format's definition."""
    c = np.asarray(codes, np.uint8).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = c & 0x7
    mag = np.where(e == 0, np.ldexp(m / 8.0, -6), np.ldexp(1.0 + m / 8.0, e - 7))
    mag = np.where((e == 15) & (m == 7), np.nan, mag)
    return sign * mag


def e4m3_encode(x):
    """float32 values -> E4M3 bit patterns: the nearest finite value, ties to the even bit pattern, magnitudes
    beyond 448 to 448 (round to nearest even, saturating).  Written as a search over the table of the 127
    finite magnitudes (the two neighbours of |x|, the nearer one, the even one on a tie), not as bit
    manipulation."""
    x = np.asarray(x, np.float32)
    table = e4m3_decode(np.arange(127, dtype=np.uint8))          # ascending magnitudes, code = index
    a = np.abs(x.astype(np.float64))
    hi = np.minimum(np.searchsorted(table, a, side="left"), 126)  # table[hi-1] < a <= table[hi] (a below 448)
    lo = np.maximum(hi - 1, 0)
    dl, dh = a - table[lo], table[hi] - a
    k = np.where(dh < dl, hi, np.where(dl < dh, lo, np.where(lo % 2 == 0, lo, hi)))   # ties: the even pattern
    k = np.where(a >= table[-1], 126, k).astype(np.uint8)
    return np.where(np.signbit(x), k | 0x80, k).astype(np.uint8)


def kv_quantize_rows(rows_u16):
    """Per-row (one token of one head) 8-bit quantisation of K or V rows [..., D] (uint16 bf16):
    scale = max|x| / 448 and code = E4M3(x / scale), both in float32 arithmetic (the precision in which the
    library decides the codes); a row of zeros gets scale 0 and codes 0.  Returns (codes uint8 [..., D],
    scale float32 [...])."""
    x = (_u16(rows_u16).astype(np.uint32) << 16).view(np.float32)
    amax = np.abs(x).max(axis=-1)
    scale = (amax / np.float32(448.0)).astype(np.float32)
    safe = np.where(scale > 0, scale, np.float32(1.0)).astype(np.float32)
    y = (x / safe[..., None]).astype(np.float32)
    return e4m3_encode(y), scale


def kv_dequantize(codes, scale):
    """codes [..., D] uint8, scale [...] float32 -> float64 values code * scale."""
    return e4m3_decode(codes) * np.asarray(scale, np.float32).astype(np.float64)[..., None]


def attend_values(q, K, V, pos, scale=None):
    """softmax(scale * K[pos] q) V[pos] for a query q [D] (uint16 bf16) over float64 rows K, V [n, D]: the
    attention of Sec. 3.1 over an explicit set of positions, for caches whose rows are not bf16."""
    qv = _widen(q)
    K, V = np.asarray(K, np.float64), np.asarray(V, np.float64)
    pos = np.asarray(pos, np.int64)
    sc = default_scale(qv.shape[-1]) if scale is None else scale
    logits = (K[pos] @ qv) * sc
    w = np.exp(logits - logits.max())
    w = w / w.sum()
    return w @ V[pos]


class RowBufferOverflow(RuntimeError):
    """Algorithm 2: a token was appended to a row buffer that already holds R tokens."""


def rowbuf_semantic(Q, K, V, L, n0, M, R, t_end, compress_when_full=True, scale=None, choose=None):
    """Algorithm 2 (compression with a row buffer) for ONE semantic (sequence, head).

    Q [N,D] image queries, K, V [L+N,D] (uint16 bf16).  State carried from step to step: `static`, at
    most M image tokens; `buf`, the row buffer, at most R tokens newer than every static token; `acc`,
    the accumulated attention score of every held token.  Invariants: static and buf are disjoint and
    each in ascending position; acc[j] = (prefill running sum of Algorithm 1, if j was selected at
    prefill, else 0) + the attention weight j received at every decode step since it was appended.
      prefill (image step n0): static = top-M of the running sums over all n0 tokens; buf empty.
      decode step t: token t-1 joins buf (a full buffer is the overflow error); the step attends over
        prompt + static + buf and every held token's weight is added to its acc; a buffer that now
        holds R tokens triggers the re-selection: static = top-M of static + buf by acc (ties: lowest
        position), buf = empty, acc of dropped tokens forgotten.
    Returns (outs [t_end-n0, D] fp64, history): history[k] = (t, static positions after step t,
    their scores, buffered positions, their scores) for every step.
    `choose(t, candidates, scores, keep)` may replace the kept candidate indices at a compression (a
    parity test uses it to follow another implementation's choice where scores tie within a tolerance);
    by default the oracle's own top-M stands.
    """
    Q, K, V = _u16(Q), _u16(K), _u16(V)
    sc = scores(Q[:n0], K[: L + n0], L, n0, scale) if n0 > 0 else np.zeros(0)
    static = topm(sc, n0, M).tolist()
    acc = {j: float(sc[j]) for j in static}
    buf = []
    outs, hist = [], []
    for t in range(n0 + 1, t_end + 1):
        if len(buf) + 1 > R:
            raise RowBufferOverflow(f"step {t}: row buffer of {R} is full")
        buf.append(t - 1)
        acc[t - 1] = 0.0
        held = static + buf
        pos = np.array(list(range(L)) + [L + j for j in held], np.int32)
        out, wts = attend(Q[t - 1], K, V, pos, scale, return_weights=True)
        for k, j in enumerate(held):
            acc[j] += float(wts[L + k])
        outs.append(out)
        if compress_when_full and len(buf) == R:
            cand = held                                   # ascending positions by construction
            s = np.array([acc[j] for j in cand], np.float64)
            keep = topm(s, len(cand), M)
            if choose is not None:
                keep = np.asarray(choose(t, cand, s, keep), np.int32)
            static = [cand[i] for i in keep]
            acc = {j: acc[j] for j in static}
            buf = []
        hist.append((t, list(static), [acc[j] for j in static], list(buf), [acc[j] for j in buf]))
    return np.array(outs), hist
