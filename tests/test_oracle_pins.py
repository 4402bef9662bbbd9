"""Pins for the fp64 CPU oracle: closed forms, brute force, special cases and a
library routine.  Nothing here touches the CUDA library."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2510_18716_b200 import workloads as wl


def bf16(a):
    return wl.from_f32(np.asarray(a, np.float32))


def widen(u):
    return (u.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def rand_bf16(rng, *shape):
    return bf16(rng.standard_normal(shape))


# ------------------------------------------------------------------ attention rows
def test_attention_row_brute_force_python_loops():
    rng = np.random.default_rng(0)
    for D, n in [(8, 5), (8, 12), (16, 1)]:
        q, K = rand_bf16(rng, D), rand_bf16(rng, n, D)
        qf, Kf = widen(q), widen(K)
        scale = 1.0 / math.sqrt(D)
        x = [scale * sum(float(qf[d]) * float(Kf[i, d]) for d in range(D)) for i in range(n)]
        z = sum(math.exp(v) for v in x)
        want = [math.exp(v) / z for v in x]
        got = oracle.attention_row(q, K)
        assert np.allclose(got, want, rtol=1e-13, atol=0)
        assert abs(got.sum() - 1.0) < 1e-14


def test_attention_row_shift_invariance_and_huge_logits():
    # subtract-max softmax must survive logits far beyond exp's range
    D = 8
    q = bf16(np.full(D, 64.0))
    K = bf16(np.stack([np.full(D, 64.0), np.full(D, 63.0), np.zeros(D)]))
    a = oracle.attention_row(q, K, scale=1.0)
    d = 64.0 * 8 * 1.0
    want = np.array([1.0, math.exp(-d), math.exp(-64.0 * 64.0 * 8)])
    want /= want.sum()
    assert np.allclose(a, want, rtol=1e-12, atol=0)


def _sdpa_fp64(q, K, V, mask):
    """torch's scaled-dot-product attention in float64 with a boolean mask (library routine)."""
    qt = torch.from_numpy(widen(q)).view(1, 1, 1, -1)
    Kt = torch.from_numpy(widen(K)).view(1, 1, *K.shape)
    Vt = torch.from_numpy(widen(V)).view(1, 1, *V.shape)
    m = torch.from_numpy(mask).view(1, 1, 1, -1)
    return torch.nn.functional.scaled_dot_product_attention(qt, Kt, Vt, attn_mask=m).view(-1).numpy()


@pytest.mark.parametrize("D", [8, 128])
def test_attend_matches_library_masked_sdpa(D):
    rng = np.random.default_rng(1)
    for trial in range(6):
        n = int(rng.integers(3, 40))
        q, K, V = rand_bf16(rng, D), rand_bf16(rng, n, D), rand_bf16(rng, n, D)
        mask = rng.random(n) < 0.5
        mask[int(rng.integers(0, n))] = True
        pos = np.nonzero(mask)[0].astype(np.int32)
        got, wts = oracle.attend(q, K, V, pos, return_weights=True)
        assert np.allclose(got, _sdpa_fp64(q, K, V, mask), rtol=1e-11, atol=1e-13)
        assert abs(wts.sum() - 1.0) < 1e-13 and (wts > 0).all()


def test_attend_distinguishes_k_from_v_and_order_of_positions():
    rng = np.random.default_rng(2)
    D, n = 8, 9
    q, K, V = rand_bf16(rng, D), rand_bf16(rng, n, D), rand_bf16(rng, n, D)
    pos = np.array([7, 1, 4], np.int32)
    a = oracle.attend(q, K, V, pos)
    assert np.allclose(a, oracle.attend(q, K, V, np.sort(pos)), rtol=1e-13)  # a set, not a list
    assert not np.allclose(a, oracle.attend(q, V, K, pos))                  # swapped operands differ
    # one position -> that V row exactly
    assert np.array_equal(oracle.attend(q, K, V, np.array([4], np.int32)), widen(V[4]))


# ------------------------------------------------------------------ retained sets
def test_retained_set_enumeration():
    L = 3
    for t in range(1, 15):
        for W in (1, 2, 5, 20):
            got = oracle.retained_set(False, L, t, W, 0)
            want = list(range(L)) + [L + j for j in range(max(0, t - W), t)]
            assert got.tolist() == want
            assert len(got) <= L + W
    top = np.array([0, 2, 3], np.int32)
    for t in range(6, 15):           # compressed at n0 = 5 + R... candidates all < t - R
        for R in (1, 2):
            got = oracle.retained_set(True, L, t, 99, R, top)
            want = list(range(L)) + [L + j for j in top] + [L + j for j in range(t - R, t)]
            assert got.tolist() == want and len(set(want)) == len(want)
            assert len(got) <= L + len(top) + R


def test_everything_retained_equals_full_attention():
    rng = np.random.default_rng(3)
    L, N, D, S, H = 4, 12, 8, 2, 3
    q = rand_bf16(rng, S, H, D)
    K, V = rand_bf16(rng, S, H, L + N, D), rand_bf16(rng, S, H, L + N, D)
    sem = np.array([0, 1, 1], np.uint8)[None, :].repeat(S, 0)
    Qobs = rand_bf16(rng, S, H, 6, D)
    for n0 in (0, 6):
        _, idx, cnt = oracle.select_batch(Qobs[:, :, : max(n0, 0)], K, sem, L, n0, N, N) if n0 else (
            None, np.full((S, H, N), -1, np.int32), np.zeros((S, H), np.int32))
        for t in (max(n0, 1), 9, N):
            full = oracle.decode_batch(q, K, V, sem, None, None, L, t, N, N, N, full=True)
            got = oracle.decode_batch(q, K, V, sem, idx, cnt, L, t, N, N, N)
            assert np.allclose(got, full, rtol=1e-12, atol=1e-14)
            # all-spatial with W >= N, no compression
            got2 = oracle.decode_batch(q, K, V, np.zeros_like(sem), None, None, L, t, N, 0, 1)
            assert np.allclose(got2, full, rtol=1e-12, atol=1e-14)
            # and it is the library's causal attention
            for s in range(S):
                for h in range(H):
                    mask = np.arange(L + N) < L + t
                    assert np.allclose(full[s, h], _sdpa_fp64(q[s, h], K[s, h], V[s, h], mask),
                                       rtol=1e-11, atol=1e-13)


def test_window_really_drops_old_tokens():
    rng = np.random.default_rng(4)
    L, N, D = 2, 10, 8
    q, K, V = rand_bf16(rng, 1, D), rand_bf16(rng, 1, L + N, D), rand_bf16(rng, 1, L + N, D)
    sem = np.zeros(1, np.uint8)
    t, W = 9, 3
    got = oracle.decode_batch(q, K, V, sem, None, None, L, t, W, 0, 1)[0]
    mask = np.zeros(L + N, bool)
    mask[:L] = True
    mask[L + t - W:L + t] = True
    assert np.allclose(got, _sdpa_fp64(q[0], K[0], V[0], mask), rtol=1e-11)
    full = oracle.decode_batch(q, K, V, sem, None, None, L, t, W, 0, 1, full=True)[0]
    assert not np.allclose(got, full)


# ------------------------------------------------------------------ sparsity metric
def harmonic(n):
    return sum(1.0 / k for k in range(1, n + 1))


@pytest.mark.parametrize("N,w,L", [(576, 32, 64), (64, 16, 32), (40, 7, 0)])
def test_sparsity_uniform_attention_closed_form(N, w, L):
    rng = np.random.default_rng(5)
    D = 8
    Q = bf16(np.zeros((1, 1, 1, N, D)))
    K = rand_bf16(rng, 1, 1, 1, L + N, D)
    s = oracle.sparsity(Q, K, L, w)[0, 0]
    want = ((N - w) - w * (harmonic(N) - harmonic(w))) / N
    assert abs(s - want) < 1e-13
    if (N, w) == (576, 32):
        assert abs(want - 0.7847) < 1e-3
    if (N, w) == (64, 16):
        assert abs(want - 0.4092) < 1e-3


def _onehot_keys(N, D, c, L):
    K = np.zeros((L + N, D))
    K[L + np.arange(N), np.arange(N)] = c
    return K


def test_sparsity_extremes_and_window_boundary():
    N, w, L, D, c = 64, 16, 5, 128, 128.0   # logit of the hit = c*c/sqrt(D) >> others (0)
    K = _onehot_keys(N, D, c, L)
    rng = np.random.default_rng(6)
    K[:L] = rng.standard_normal((L, D)) * 0.01

    def s_for(target_of_t):
        Q = np.zeros((N, D))
        for t in range(1, N + 1):
            j = target_of_t(t)
            if j is not None:
                Q[t - 1, j] = c
        return oracle.sparsity(bf16(Q)[None, None, None], bf16(K)[None, None, None], L, w)[0, 0]

    assert s_for(lambda t: t - 1) < 1e-12                                   # all mass on self
    assert abs(s_for(lambda t: 0) - (N - w) / N) < 1e-12                     # all mass on token 0
    # newest token still counted as "far" is index t-1-w; index t-w is already recent
    assert abs(s_for(lambda t: t - 1 - w if t - 1 - w >= 0 else t - 1) - (N - w) / N) < 1e-12
    assert s_for(lambda t: t - w if t - w >= 0 else t - 1) < 1e-12


def test_sparsity_bounds_prompt_independence_and_averaging():
    rng = np.random.default_rng(7)
    nl, P, H, N, D, L, w = 2, 3, 2, 20, 8, 4, 5
    Q, K = rand_bf16(rng, nl, P, H, N, D), rand_bf16(rng, nl, P, H, L + N, D)
    s = oracle.sparsity(Q, K, L, w)
    assert s.shape == (nl, H) and (s >= 0).all() and (s <= (N - w) / N).all()
    K2 = K.copy()
    K2[..., :L, :] = rand_bf16(rng, nl, P, H, L, D)          # prompt mass cancels in the ratio
    assert np.allclose(oracle.sparsity(Q, K2, L, w), s, rtol=1e-11)
    # mean over prompts of per-prompt sums / N; [layers, P, H] indexing
    for l in range(nl):
        for h in range(H):
            tot = sum(oracle.sparsity_sum(Q[l, p, h], K[l, p, h], L, w) for p in range(P))
            assert abs(tot / (P * N) - s[l, h]) < 1e-14
    # brute force of the definition with python loops
    l, p, h = 1, 2, 0
    acc = 0.0
    for t in range(1, N + 1):
        a = oracle.attention_row(Q[l, p, h, t - 1], K[l, p, h, : L + t])
        num = sum(a[L + i] for i in range(0, t - 1 - w + 1))
        den = sum(a[L + i] for i in range(0, t))
        acc += num / den
    assert abs(acc - oracle.sparsity_sum(Q[l, p, h], K[l, p, h], L, w)) < 1e-12


def test_labels_threshold_equality_is_spatial():
    s = np.array([0.44999, 0.45, 0.45001, 0.0, 1.0])
    assert oracle.labels(s, 0.45).tolist() == [0, 0, 1, 0, 1]


@pytest.mark.parametrize("name", ["tiny", "janus7b", "janus1b"])
def test_classifier_recovers_generator_split(name):
    cfg = wl.CONFIGS[name]
    Qc, Kc = wl.gen_calibration(cfg, [0])
    s = oracle.sparsity(wl.to_u16(Qc), wl.to_u16(Kc), cfg.prompt_len, cfg.cls_window)
    lab = oracle.labels(s, cfg.tau)[0]
    assert lab.tolist() == wl.sink_mask(cfg, 0).tolist()
    assert lab.sum() == cfg.n_sink_heads
    assert np.abs(s - cfg.tau).min() > 0.03        # well clear of the threshold


# ------------------------------------------------------------------ scores
def test_scores_rows_sum_to_one_and_uniform_closed_form():
    rng = np.random.default_rng(8)
    L, n0, D = 5, 17, 8
    K = rand_bf16(rng, L + n0, D)
    for n_obs in (n0, 6, 1):
        Q = rand_bf16(rng, n_obs, D)
        sc, pm = oracle.scores(Q, K, L, n0, return_prompt_mass=True)
        assert abs(sc.sum() + pm - n_obs) < 1e-12 and (sc >= 0).all()
        sc0 = oracle.scores(bf16(np.zeros((n_obs, D))), K, L, n0)
        want = [sum(1.0 / (L + t) for t in range(max(j + 1, n0 - n_obs + 1), n0 + 1)) for j in range(n0)]
        assert np.allclose(sc0, want, rtol=1e-13, atol=1e-15)


def test_scores_brute_force_and_causality():
    rng = np.random.default_rng(9)
    L, n0, n_obs, D = 3, 9, 4, 8
    Q, K = rand_bf16(rng, n_obs, D), rand_bf16(rng, L + n0, D)
    want = np.zeros(n0)
    for r in range(n_obs):
        t = n0 - n_obs + 1 + r
        a = oracle.attention_row(Q[r], K[: L + t])
        want[:t] += a[L:L + t]
    got = oracle.scores(Q, K, L, n0)
    assert np.allclose(got, want, rtol=1e-13)
    # the newest token is only seen by the last query
    a_last = oracle.attention_row(Q[-1], K[: L + n0])
    assert abs(got[n0 - 1] - a_last[L + n0 - 1]) < 1e-15
    # one-hot queries: score counts the hits
    N, Dh, c = 12, 128, 128.0
    Kh = _onehot_keys(N, Dh, c, 0)
    Qh = np.zeros((N, Dh))
    Qh[:, 0] = c                                  # every step looks at image token 0
    sc = oracle.scores(bf16(Qh), bf16(Kh), 0, N)
    assert abs(sc[0] - N) < 1e-9 and sc[1:].max() < 1e-9


# ------------------------------------------------------------------ top-M
def test_topm_tie_rule_and_edges():
    assert oracle.topm(np.ones(10), 10, 4).tolist() == [0, 1, 2, 3]
    assert oracle.topm(np.ones(10), 7, 20).tolist() == list(range(7))
    assert oracle.topm(np.ones(10), 0, 4).tolist() == []
    assert oracle.topm(np.ones(10), 5, 0).tolist() == []
    s = np.array([1.0, 3.0, 3.0, 2.0, 3.0, 0.5])
    assert oracle.topm(s, 6, 2).tolist() == [1, 2]
    assert oracle.topm(s, 6, 4).tolist() == [1, 2, 3, 4]
    assert oracle.topm(s, 4, 3).tolist() == [1, 2, 3]          # candidates only [0, 4)


def test_topm_matches_stable_sort():
    rng = np.random.default_rng(10)
    for _ in range(50):
        n = int(rng.integers(1, 60))
        M = int(rng.integers(1, 70))
        s = rng.integers(0, 8, n).astype(np.float64) / 8        # many duplicates
        want = np.sort(np.argsort(-s, kind="stable")[: min(M, n)])
        got = oracle.topm(s, n, M)
        assert got.tolist() == want.tolist()
        assert (np.diff(got) > 0).all()


@pytest.mark.parametrize("name", ["tiny", "janus7b"])
def test_planted_sinks_are_selected(name):
    cfg = wl.CONFIGS[name]
    seqs = [0] if cfg.n_seqs == 1 else [0, 1]
    q, k, v, planted = wl.gen_layer(cfg, 0, seqs)
    L, n0 = cfg.prompt_len, cfg.n0
    sem = wl.sink_mask(cfg, 0)[None, :].repeat(len(seqs), 0)
    sc, idx, cnt = oracle.select_batch(wl.to_u16(q[:, :, :n0]), wl.to_u16(k[:, :, : L + n0]), sem, L, n0,
                                       cfg.sink_budget, cfg.sink_recent)
    n_cand = n0 - cfg.sink_recent
    for s in range(len(seqs)):
        for h in range(cfg.n_heads):
            if not sem[s, h]:
                assert cnt[s, h] == 0 and (idx[s, h] == -1).all()
                continue
            sel = idx[s, h, : cnt[s, h]]
            assert cnt[s, h] == min(cfg.sink_budget, n_cand)
            assert (np.diff(sel) > 0).all() and sel.min() >= 0 and sel.max() < n_cand
            assert set(planted[s, h].tolist()) <= set(sel.tolist())
            # single-pair functions agree with the batch driver
            one = oracle.scores(wl.to_u16(q[s, h, :n0]), wl.to_u16(k[s, h, : L + n0]), L, n0)
            assert np.array_equal(one, sc[s, h])
            assert oracle.topm(one, n_cand, cfg.sink_budget).tolist() == sel.tolist()


def test_decode_batch_agrees_with_single_pair_functions():
    cfg = wl.CONFIGS["tiny"]
    q, k, v, _ = wl.gen_layer(cfg, 0, [0])
    L, n0, W, M, R = cfg.prompt_len, cfg.n0, cfg.window, cfg.sink_budget, cfg.sink_recent
    sem = wl.sink_mask(cfg, 0)[None, :]
    qu, ku, vu = wl.to_u16(q), wl.to_u16(k), wl.to_u16(v)
    _, idx, cnt = oracle.select_batch(qu[:, :, :n0], ku[:, :, : L + n0], sem, L, n0, M, R)
    for t in (n0 + 1, n0 + 9, cfg.n_img):
        out = oracle.decode_batch(qu[:, :, t - 1], ku, vu, sem, idx, cnt, L, t, W, M, R)
        for h in range(cfg.n_heads):
            pos = oracle.retained_set(sem[0, h], L, t, W, R, idx[0, h, : cnt[0, h]])
            assert len(pos) == min(cfg.slots(bool(sem[0, h])), L + t)
            want = oracle.attend(qu[0, h, t - 1], ku[0, h], vu[0, h], pos)
            assert np.array_equal(out[0, h], want)


# ------------------------------------------------------------------ Algorithm 2 (row buffer)
def test_rowbuf_nothing_dropped_is_full_attention_and_running_sum():
    rng = np.random.default_rng(20)
    L, N, D, n0, R = 3, 14, 8, 4, 3
    Q, K, V = rand_bf16(rng, N, D), rand_bf16(rng, L + N, D), rand_bf16(rng, L + N, D)
    outs, hist = oracle.rowbuf_semantic(Q, K, V, L, n0, N, R, N)          # M = N: nothing is ever dropped
    for k, t in enumerate(range(n0 + 1, N + 1)):
        mask = np.arange(L + N) < L + t
        assert np.allclose(outs[k], _sdpa_fp64(Q[t - 1], K, V, mask), rtol=1e-11, atol=1e-13)
    # accumulated scores = Algorithm 1's running sum over all steps so far (already pinned above)
    t, static, acc, buf, bacc = hist[-1]
    held = static + buf
    want = oracle.scores(Q[:N], K, L, N)
    assert held == list(range(N))
    assert np.allclose(np.array(acc + bacc), want, rtol=1e-12, atol=1e-15)


def test_rowbuf_compresses_when_full_and_overflows_otherwise():
    rng = np.random.default_rng(21)
    L, N, D, n0, M, R = 2, 20, 8, 6, 4, 3
    Q, K, V = rand_bf16(rng, N, D), rand_bf16(rng, L + N, D), rand_bf16(rng, L + N, D)
    outs, hist = oracle.rowbuf_semantic(Q, K, V, L, n0, M, R, N)
    for t, static, acc, buf, _ in hist:
        assert len(static) <= M and len(buf) < R and len(static) + len(buf) <= M + R
        assert static == sorted(set(static)) and all(j < t for j in static + buf)
        assert len(buf) == (t - n0) % R                       # emptied every R steps
        assert all(a >= 0 for a in acc)
    with pytest.raises(oracle.RowBufferOverflow):
        oracle.rowbuf_semantic(Q, K, V, L, n0, M, R, n0 + R + 1, compress_when_full=False)
    # brute force of one cycle: scores after R steps and the re-selection
    sc0 = oracle.scores(Q[:n0], K[: L + n0], L, n0)
    static = oracle.topm(sc0, n0, M).tolist()
    acc = {j: sc0[j] for j in static}
    held = list(static)
    for t in range(n0 + 1, n0 + R + 1):
        held.append(t - 1)
        acc[t - 1] = 0.0
        pos = np.array(list(range(L)) + [L + j for j in held], np.int32)
        a = oracle.attention_row(Q[t - 1], K[pos])
        for k, j in enumerate(held):
            acc[j] += a[L + k]
    order = sorted(held, key=lambda j: (-acc[j], j))[:M]
    assert hist[R - 1][1] == sorted(order)
    assert np.allclose(hist[R - 1][2], [acc[j] for j in sorted(order)], rtol=1e-12)


def test_rowbuf_promotes_a_heavily_attended_buffer_token():
    # one-hot keys: every decode query looks at the token appended at step n0+1, which must then
    # displace the least-attended static token at the first compression
    N, D, L, n0, M, R, c = 12, 128, 0, 6, 3, 3, 128.0
    K = _onehot_keys(N, D, c, L)
    Q = np.zeros((N, D))
    Q[:n0, 0] = c                         # prefill steps look at token 0
    Q[n0:, n0] = c                        # decode steps look at token n0 (first buffered token)
    V = np.random.default_rng(22).standard_normal((N, D))
    outs, hist = oracle.rowbuf_semantic(bf16(Q), bf16(K), bf16(V), L, n0, M, R, n0 + R)
    t, static, acc, buf, _ = hist[-1]
    assert n0 in static and 0 in static and buf == []
    assert abs(acc[static.index(n0)] - R) < 1e-9              # R steps of weight ~1 each


# ------------------------------------------------------------------ stored closed-form values
def test_golden_closed_forms():
    """tests/golden/closed_forms.txt holds values fixed by the definitions (Sec. 3.3 metric, Algorithm 1
    running sum) under uniform or one-token attention, evaluated in exact rational arithmetic by the
    script beside it; the oracle must reproduce each of them."""
    import os
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "closed_forms.txt")
    rng = np.random.default_rng(11)
    D, n_checked = 8, 0
    for ln in open(path):
        f = ln.split()
        if not f or f[0].startswith("#"):
            continue
        want = float(f[-1])
        if f[0] in ("sparsity_uniform", "sparsity_token0"):
            N, w = int(f[1]), int(f[2])
            L = 3
            if f[0] == "sparsity_uniform":
                Q = bf16(np.zeros((1, 1, 1, N, D)))
                K = rand_bf16(rng, 1, 1, 1, L + N, D)
            else:
                # every query points at image token 0's key, far more strongly than at any other key
                K = np.zeros((L + N, D))
                K[L, 0] = 64.0
                K[L + 1:, 1] = 1.0
                Q = np.zeros((N, D))
                Q[:, 0] = 64.0
                K, Q = bf16(K[None, None, None]), bf16(Q[None, None, None])
            got = oracle.sparsity(Q, K, L, w)[0, 0]
            assert abs(got - want) < (1e-12 if f[0] == "sparsity_uniform" else 1e-9), (ln, got)
        elif f[0] == "score_uniform":
            L, n0, n_obs, j = (int(x) for x in f[1:5])
            K = rand_bf16(rng, L + n0, D)
            sc = oracle.scores(bf16(np.zeros((n_obs, D))), K, L, n0)
            assert abs(sc[j] - want) < 1e-12, (ln, sc[j])
        else:
            raise AssertionError(f"unknown golden line: {ln}")
        n_checked += 1
    assert n_checked >= 14


def test_rowbuf_of_one_is_the_drop_one_rule_of_algorithm_1():
    """Algorithm 1 taken literally evicts one token per step: after the step's attention the token
    with the lowest accumulated score leaves (among equal scores the newest).  The row-buffer
    function with R = 1 states it as "top-M of M + 1"; the two must retain the same sets, with the
    same scores and outputs, step by step."""
    rng = np.random.default_rng(21)
    L, N, n0, M, D = 3, 40, 12, 6, 8
    Q, K, V = rand_bf16(rng, N, D), rand_bf16(rng, L + N, D), rand_bf16(rng, L + N, D)
    outs, hist = oracle.rowbuf_semantic(Q, K, V, L, n0, M, 1, N)

    qf, kf, vf = widen(Q), widen(K), widen(V)
    scale = 1.0 / math.sqrt(D)
    sc0 = oracle.scores(Q[:n0], K[: L + n0], L, n0)
    kept = sorted(sorted(range(n0), key=lambda j: (-sc0[j], j))[:M])
    score = {j: float(sc0[j]) for j in kept}
    for i, t in enumerate(range(n0 + 1, N + 1)):
        held = kept + [t - 1]
        score[t - 1] = 0.0
        pos = list(range(L)) + [L + j for j in held]
        logit = np.array([scale * float(qf[t - 1] @ kf[p]) for p in pos])
        w = np.exp(logit - logit.max())
        w /= w.sum()
        assert np.allclose(outs[i], w @ vf[pos], rtol=1e-12, atol=1e-13)
        for k, j in enumerate(held):
            score[j] += w[L + k]
        if len(held) > M:
            worst = min(held, key=lambda j: (score[j], -j))      # lowest score; among equals the newest
            held.remove(worst)
            del score[worst]
        kept = sorted(held)
        assert hist[i][0] == t and hist[i][1] == kept and hist[i][3] == []
        assert np.allclose(hist[i][2], [score[j] for j in kept], rtol=1e-12, atol=0)


def test_kv_token_mse_pins():
    """Sec. 3.2, MSE_token: identical caches give 0; one perturbed element gives its squared change at
    that token only; the sum over tokens is the squared Frobenius distance of K plus that of V (library
    norm); a Python-loop restatement on a small case; symmetry in the two caches; K and V both count."""
    g = torch.Generator().manual_seed(11)
    shape = (2, 3, 7, 16)
    Ka, Va, Kb, Vb = (torch.randn(shape, generator=g).to(torch.bfloat16) for _ in range(4))
    ua, uva, ub, uvb = (wl.to_u16(x) for x in (Ka, Va, Kb, Vb))
    assert np.array_equal(oracle.kv_token_mse(ua, uva, ua, uva), np.zeros(shape[:-1]))
    # one element of V changed by a known amount, at (1, 2, 5, 3)
    Vp = Va.clone()
    Vp[1, 2, 5, 3] = Va[1, 2, 5, 3] + 0.5
    delta = float(Vp[1, 2, 5, 3].double() - Va[1, 2, 5, 3].double())      # after bf16 rounding
    got = oracle.kv_token_mse(ua, wl.to_u16(Vp), ua, uva)
    want = np.zeros(shape[:-1])
    want[1, 2, 5] = delta * delta
    assert np.array_equal(got, want) and delta != 0.0
    # the same through K: both tensors count, and separately
    Kp = Ka.clone()
    Kp[0, 0, 0, 15] = Ka[0, 0, 0, 15] * 2
    d2 = float(Kp[0, 0, 0, 15].double() - Ka[0, 0, 0, 15].double())
    got = oracle.kv_token_mse(wl.to_u16(Kp), wl.to_u16(Vp), ua, uva)
    assert got[0, 0, 0] == d2 * d2 and got[1, 2, 5] == delta * delta and got.sum() == d2 * d2 + delta * delta
    # sum over tokens = squared Frobenius distances (numpy's norm), per (i, h)
    m = oracle.kv_token_mse(ua, uva, ub, uvb)
    for i in range(shape[0]):
        for h in range(shape[1]):
            fro = (np.linalg.norm((Ka[i, h].double() - Kb[i, h].double()).numpy()) ** 2 +
                   np.linalg.norm((Va[i, h].double() - Vb[i, h].double()).numpy()) ** 2)
            assert math.isclose(m[i, h].sum(), fro, rel_tol=1e-12)
    # plain loops on one (i, h)
    for j in range(shape[2]):
        acc = 0.0
        for d in range(shape[3]):
            acc += (float(Ka[1, 0, j, d]) - float(Kb[1, 0, j, d])) ** 2 + (float(Va[1, 0, j, d]) - float(Vb[1, 0, j, d])) ** 2
        assert math.isclose(m[1, 0, j], acc, rel_tol=1e-12)
    assert np.array_equal(m, oracle.kv_token_mse(ub, uvb, ua, uva))
    assert (m > 0).all()


def test_e4m3_decode_and_encode_pins():
    """The 8-bit format of the quantised cache: the decode table against the library's float8_e4m3fn and the
    format's closed form; encode against the library cast on in-range values, exact ties to the even bit
    pattern, saturation at 448, every finite code a fixed point, monotonicity."""
    codes = np.arange(256, dtype=np.uint8)
    lib = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).float().numpy().astype(np.float64)
    got = oracle.e4m3_decode(codes)
    assert np.array_equal(np.isnan(got), np.isnan(lib)) and np.isnan(got).sum() == 2
    ok = ~np.isnan(got)
    assert np.array_equal(got[ok], lib[ok])
    assert got[0x7E] == 448.0 and got[0x01] == 2.0 ** -9 and got[0x08] == 2.0 ** -6 and got[0x38] == 1.0 and got[0xB8] == -1.0
    finite = codes[ok]
    assert np.array_equal(oracle.e4m3_encode(got[ok].astype(np.float32)) & 0x7F, finite & 0x7F)     # fixed points (+-0 aside)
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(0, 100, 4000), rng.normal(0, 1, 4000), rng.uniform(-448, 448, 4000),
                        rng.normal(0, 0.01, 2000)]).astype(np.float32)
    x = x[np.abs(x) <= 448]
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(oracle.e4m3_encode(x), want)
    # midpoints of neighbouring magnitudes go to the even bit pattern
    mags = got[:127]
    mid = ((mags[:-1] + mags[1:]) / 2).astype(np.float32)
    assert np.array_equal(mid.astype(np.float64), (mags[:-1] + mags[1:]) / 2)                     # exact in float32
    enc = oracle.e4m3_encode(mid)
    assert np.array_equal(enc, np.where(np.arange(126) % 2 == 0, np.arange(126), np.arange(1, 127)).astype(np.uint8))
    assert np.array_equal(oracle.e4m3_encode(np.array([449, 480, 1e6, -1e9], np.float32)), np.array([0x7E, 0x7E, 0x7E, 0xFE], np.uint8))
    xs = np.sort(x)
    assert (np.diff(oracle.e4m3_decode(oracle.e4m3_encode(xs))) >= 0).all()


def test_kv_quantize_rows_pins():
    """Per-row scale = max|x| / 448: the largest element is reproduced (up to float32 rounding of the scale),
    every element within half a step of its binade (relative error <= 2^-4 for normal codes, absolute
    <= scale * 2^-10 below), zero rows stay zero, and scaling a row by a power of two scales the scale only."""
    g = torch.Generator().manual_seed(3)
    rows = (torch.randn((5, 7, 128), generator=g) * torch.logspace(-3, 2, 7)[None, :, None]).to(torch.bfloat16)
    rows[2, 3] = 0
    u = wl.to_u16(rows)
    codes, scale = oracle.kv_quantize_rows(u)
    assert codes.shape == (5, 7, 128) and scale.shape == (5, 7) and codes.dtype == np.uint8 and scale.dtype == np.float32
    x = rows.double().numpy()
    dq = oracle.kv_dequantize(codes, scale)
    amax = np.abs(x).max(-1)
    assert np.allclose(np.abs(dq).max(-1), amax, rtol=1e-6) and np.array_equal(scale, (amax.astype(np.float32) / np.float32(448)))
    err = np.abs(dq - x)
    assert (err <= np.maximum(np.abs(x) * 2.0 ** -4, scale[..., None].astype(np.float64) * 2.0 ** -10) * (1 + 1e-6)).all()
    assert (codes[2, 3] == 0).all() and scale[2, 3] == 0 and (dq[2, 3] == 0).all()
    c2, s2 = oracle.kv_quantize_rows(wl.to_u16((rows * 4).to(torch.bfloat16)))
    assert np.array_equal(c2, codes) and np.array_equal(s2, scale * np.float32(4))


def test_attend_values_equals_attend_on_bf16_rows():
    """attend_values on exactly widened bf16 rows is the attention the C routine computes (and, through its own
    pin, the library's masked SDPA)."""
    g = torch.Generator().manual_seed(5)
    q, K, V = (torch.randn(s, generator=g).to(torch.bfloat16) for s in ((128,), (40, 128), (40, 128)))
    pos = np.array([0, 1, 2, 7, 9, 30, 39], np.int32)
    a = oracle.attend(wl.to_u16(q), wl.to_u16(K), wl.to_u16(V), pos)
    b = oracle.attend_values(wl.to_u16(q), K.double().numpy(), V.double().numpy(), pos)
    assert np.allclose(a, b, rtol=1e-12, atol=1e-14)
    # the quantised cache changes the result by the quantisation error only: a few percent of |V|
    ck, sk = oracle.kv_quantize_rows(wl.to_u16(K))
    cv, sv = oracle.kv_quantize_rows(wl.to_u16(V))
    c = oracle.attend_values(wl.to_u16(q), oracle.kv_dequantize(ck, sk), oracle.kv_dequantize(cv, sv), pos)
    assert 0 < np.abs(c - a).max() < 0.1
