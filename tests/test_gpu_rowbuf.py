"""GPU parity of the row-buffer mode (Algorithm 2): append into the buffer, attend over prompt +
static set + buffer, accumulate the attention scores of semantic heads, re-select when the buffer is
full -- against the fp64 oracle, step by step, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_18716_b200 import binding as B
from paper_2510_18716_b200 import workloads as wl

from parity_util import BAND, check_outputs

pytestmark = pytest.mark.gpu


def _run(cfg, layer, seqs, t_end, fused=False):
    dev = torch.device("cuda:0")
    L, n0, M, R, W, H, S = cfg.prompt_len, cfg.n0, cfg.sink_budget, cfg.sink_recent, cfg.window, cfg.n_heads, len(seqs)
    labels = wl.sink_mask(cfg, layer)
    cache = B.SsdCache(B.config_from_workload(cfg, n_layers=1, n_seqs=S), device=dev)
    cache.set_row_buffer(True)
    cache.set_head_labels(labels)
    q, k, v, _ = wl.gen_layer(cfg, layer, seqs, device=dev)
    qu, ku, vu = wl.to_u16(q), wl.to_u16(k), wl.to_u16(v)
    cache.compress(0, q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0)

    # the oracle runs each semantic pair on its own, following the GPU's choice inside the tie band
    gpu_sets = {}          # (s, h, t) -> static image indices after the compression at step t
    n_band = [0]

    def chooser(s, h):
        def choose(t, cand, sc, keep):
            got = gpu_sets[(s, h, t)]
            want = [cand[i] for i in keep]
            if got == want:
                return keep
            n_band[0] += 1
            kth = np.sort(sc)[::-1][len(keep) - 1]
            sure_in = {cand[i] for i in np.nonzero(sc > kth * (1 + BAND))[0]}
            band = {cand[i] for i in np.nonzero(np.abs(sc - kth) <= BAND * abs(kth))[0]}
            assert sure_in <= set(got) <= (sure_in | band) and len(got) == len(want)
            return [cand.index(j) for j in got]
        return choose

    # GPU pass first (records outputs, sets and scores), then the oracle replays it
    outs = []
    for t in range(n0 + 1, t_end + 1):
        kt, vt, qt = (x.contiguous() for x in (k[:, :, L + t - 1], v[:, :, L + t - 1], q[:, :, t - 1]))
        if fused == "layers" and t % 3:  # the one-launch form (accumulates the scores itself), and after
            o = cache.append_decode_layers(0, kt[None], vt[None], qt[None])[0]    # every two of them the two calls
        elif fused and t % 3:            # mostly the single launch, now and then the two calls
            o = cache.append_decode(0, kt, vt, qt)
        else:
            cache.append(0, kt, vt)
            o = cache.decode_attn(0, qt)
        outs.append(o.float().cpu().numpy().astype(np.float64))
        if (t - n0) % R == 0:
            if fused == "layers":
                cache.recompress_layers(0, 1)
            else:
                cache.recompress(0)
            gi = cache.get_indices(0)
            for s in range(S):
                for h in range(H):
                    if labels[h]:
                        st = gi[s, h, L:L + M]
                        # tokens that stay keep their slots and the ones that enter take the freed ones, so
                        # the static slots are not ordered by position after a re-selection: compare as sets
                        gpu_sets[(s, h, t)] = sorted((st[st >= 0] - L).tolist())
                        assert len(set(gpu_sets[(s, h, t)])) == len(gpu_sets[(s, h, t)])
                        ring = gi[s, h, L + M:L + M + R]
                        assert (ring == -1).all(), "the buffer is empty after a re-selection"
            assert (cache.get_lengths(0)[labels == 1] == L + min(M, t)).all()
    assert cache.device_status() == 0

    for s in range(S):
        for h in range(H):
            if labels[h]:
                want, hist = oracle.rowbuf_semantic(qu[s, h], ku[s, h], vu[s, h], L, n0, M, R, t_end,
                                                    choose=chooser(s, h))
                for i, t in enumerate(range(n0 + 1, t_end + 1)):
                    err = np.abs(outs[i][s, h] - want[i])
                    assert err.max() <= 2e-2 and err.mean() <= 2e-3, (s, h, t, err.max())
            else:
                for i, t in enumerate(range(n0 + 1, t_end + 1)):
                    pos = oracle.retained_set(False, L, t, W, R)
                    want = oracle.attend(qu[s, h, t - 1], ku[s, h], vu[s, h], pos)
                    err = np.abs(outs[i][s, h] - want)
                    assert err.max() <= 2e-2 and err.mean() <= 2e-3, (s, h, t, err.max())
    cache.close()
    return n_band[0]


@pytest.mark.parametrize("fused", [False, True, "layers"])
def test_rowbuf_tiny_every_step(fused):
    cfg = wl.CONFIGS["tiny"]
    _run(cfg, 0, [0], cfg.n_img, fused)


@pytest.mark.parametrize("fused", [False, True, "layers"])
def test_rowbuf_janus1b_slice(fused):
    cfg = wl.CONFIGS["janus1b"]
    _run(cfg, 3, [0, 1], cfg.n0 + 3 * cfg.sink_recent + 5, fused)


def test_rowbuf_scores_match_oracle_before_reselection():
    cfg = wl.CONFIGS["tiny"]
    dev = torch.device("cuda:0")
    L, n0, M, R, H = cfg.prompt_len, cfg.n0, cfg.sink_budget, cfg.sink_recent, cfg.n_heads
    labels = wl.sink_mask(cfg, 0)
    cache = B.SsdCache(B.config_from_workload(cfg), device=dev)
    cache.set_row_buffer(True)
    cache.set_head_labels(labels)
    q, k, v, _ = wl.gen_layer(cfg, 0, [0], device=dev)
    qu, ku, vu = wl.to_u16(q), wl.to_u16(k), wl.to_u16(v)
    cache.compress(0, q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0)
    for t in range(n0 + 1, n0 + R + 1):
        kt, vt, qt = (x.contiguous() for x in (k[:, :, L + t - 1], v[:, :, L + t - 1], q[:, :, t - 1]))
        if t % 3 == 0:
            cache.append_decode(0, kt, vt, qt)
        elif t % 3 == 1:
            cache.append_decode_layers(0, kt[None], vt[None], qt[None])
        else:
            cache.append(0, kt, vt)
            cache.decode_attn(0, qt)
    acc = cache.get_scores(0)
    gi = cache.get_indices(0)
    for h in range(H):
        if not labels[h]:
            assert (acc[0, h] == -1).all()
            continue
        _, hist = oracle.rowbuf_semantic(qu[0, h], ku[0, h], vu[0, h], L, n0, M, R, n0 + R, compress_when_full=False)
        _, static, sacc, buf, bacc = hist[-1]
        assert (gi[0, h, L:L + M] - L).tolist() == static
        assert (gi[0, h, L + M:L + M + R] - L).tolist() == buf
        assert np.allclose(acc[0, h, :M], sacc, rtol=2e-4, atol=1e-6)
        assert np.allclose(acc[0, h, M:M + R], bacc, rtol=2e-4, atol=1e-6)
    # one more token without a re-selection: the buffer is full
    x = k[:, :, L + n0 + R].contiguous()
    with pytest.raises(B.SsdError) as e:
        cache.append(0, x, x)
    assert e.value.code == B.SSD_ERR_OVERFLOW
    cache.recompress(0)
    cache.append(0, x, x)                      # accepted again
    cache.close()


def test_per_step_eviction_is_a_row_buffer_of_one():
    """Algorithm 1 taken literally re-selects at every step; that is the row buffer with R = 1 and a
    re-selection after each step (the evicted token is dropped after the step's attention)."""
    import dataclasses
    cfg = dataclasses.replace(wl.CONFIGS["tiny"], sink_recent=1, name="tiny_r1")
    _run(cfg, 0, [0], cfg.n0 + 20, fused=True)
    _run(cfg, 0, [0], cfg.n0 + 20, fused="layers")     # one decode launch and one re-selection launch per step


def test_recompress_layers_equals_per_layer_recompress():
    """Three layers with different head layouts, two buffer cycles: the one-launch step with the
    one-launch re-selection against per-layer calls; same static sets and (to rounding) same scores."""
    cfg = wl.CONFIGS["tiny"]
    dev = torch.device("cuda:0")
    L, n0, M, R, H, NL, S = cfg.prompt_len, cfg.n0, cfg.sink_budget, cfg.sink_recent, cfg.n_heads, 3, 2
    rng = np.random.default_rng(9)
    labels = np.stack([wl.sink_mask(cfg, 0), np.ones(H, np.uint8), rng.integers(0, 2, H).astype(np.uint8)])
    data = [wl.gen_layer(cfg, l, [0, 1], device=dev) for l in range(NL)]
    caches = []
    for _ in range(2):
        c = B.SsdCache(B.config_from_workload(cfg, n_layers=NL, n_seqs=S), device=dev)
        c.set_row_buffer(True)
        c.set_head_labels(labels)
        for l, (q, k, v, _) in enumerate(data):
            c.compress(l, q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0)
        caches.append(c)
    a, b = caches
    for t in range(n0 + 1, n0 + 2 * R + 1):
        qs = torch.stack([data[l][0][:, :, t - 1] for l in range(NL)]).contiguous()
        ks = torch.stack([data[l][1][:, :, L + t - 1] for l in range(NL)]).contiguous()
        vs = torch.stack([data[l][2][:, :, L + t - 1] for l in range(NL)]).contiguous()
        want = torch.stack([a.append_decode(l, ks[l], vs[l], qs[l]) for l in range(NL)])
        got = b.append_decode_layers(0, ks, vs, qs)
        d = (got.float() - want.float()).abs()
        assert d.max().item() <= 2e-2 and d.mean().item() <= 5e-4
        if (t - n0) % R == 0:
            for l in range(NL):
                a.recompress(l)
            b.recompress_layers(0, NL)
            for l in range(NL):
                assert np.array_equal(a.get_indices(l), b.get_indices(l)), (t, l)
                sa, sb = a.get_scores(l), b.get_scores(l)
                assert np.array_equal(sa < 0, sb < 0)
                assert np.allclose(sa, sb, rtol=1e-4, atol=1e-6)
    lib = B.load()
    st = torch.cuda.current_stream().cuda_stream
    assert lib.ssd_recompress_layers(b._h, 2, 2, st) == B.SSD_ERR_INVALID_ARG
    b.set_row_buffer(False)
    assert lib.ssd_recompress_layers(b._h, 0, NL, st) == B.SSD_ERR_BAD_STATE
    assert a.device_status() == 0 and b.device_status() == 0
    for c in caches:
        c.close()


def test_rowbuf_more_than_1024_candidates_takes_the_radix_path():
    """Up to 1024 candidates a re-selection counts ranks directly; above, it radix-selects the
    threshold score and breaks ties on positions.  A head with M + R = 1108 exercises the second
    path (and the score row of that length in the one-launch kernel), against the oracle."""
    import dataclasses
    cfg = dataclasses.replace(wl.CONFIGS["tiny"], grid=(35, 40), n0=1200, sink_budget=1100, sink_recent=8,
                              window=24, name="tiny_wide")
    n = _run(cfg, 0, [0], cfg.n0 + 2 * cfg.sink_recent + 3, fused="layers")
    assert n >= 0


@pytest.mark.parametrize("case", ["janus1b_after_prefill", "tiny_from_empty"])
def test_eviction_in_the_launch_equals_reselection_after_the_step(case):
    """With a buffer of one token ssd_append_decode_layers re-selects inside the launch.  Against the
    general path (append, attend, ssd_recompress): same retained sets after every step, same scores to
    rounding, outputs within the usual bar; and ssd_recompress has nothing to do.  Once on a slice of
    janus1b after a prefill (static set full: every step evicts or drops), once on the tiny shape
    from an empty cache (the static set first grows slot by slot, then starts evicting)."""
    import dataclasses
    base = wl.CONFIGS["janus1b" if case == "janus1b_after_prefill" else "tiny"]
    cfg = dataclasses.replace(base, sink_budget=base.sink_budget + base.sink_recent - 1, sink_recent=1, name=base.name + "_r1")
    dev = torch.device("cuda:0")
    prefill = case == "janus1b_after_prefill"
    L, n0, M, H, S, NL = cfg.prompt_len, (cfg.n0 if prefill else 0), cfg.sink_budget, cfg.n_heads, 3, 2
    labels = np.stack([wl.sink_mask(cfg, l) for l in range(NL)])
    data = [wl.gen_layer(cfg, l, list(range(S)), device=dev) for l in range(NL)]
    caches = []
    for _ in range(2):
        c = B.SsdCache(B.config_from_workload(cfg, n_layers=NL, n_seqs=S), device=dev)
        c.set_row_buffer(True)
        c.set_head_labels(labels)
        for l, (q, k, v, _) in enumerate(data):
            if prefill:
                c.compress(l, q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0)
        caches.append(c)
    general, fused = caches
    launches_before = None
    for t in range(n0 + 1, n0 + 41):
        qs = torch.stack([data[l][0][:, :, t - 1] for l in range(NL)]).contiguous()
        ks = torch.stack([data[l][1][:, :, L + t - 1] for l in range(NL)]).contiguous()
        vs = torch.stack([data[l][2][:, :, L + t - 1] for l in range(NL)]).contiguous()
        want = []
        for l in range(NL):
            general.append(l, ks[l], vs[l])
            want.append(general.decode_attn(l, qs[l]))
            general.recompress(l)
        got = fused.append_decode_layers(0, ks, vs, qs)
        launches_before = B.kernel_launch_count()
        fused.recompress_layers(0, NL)                      # the buffer is already empty
        assert B.kernel_launch_count() == launches_before
        d = (got.float() - torch.stack(want).float()).abs()
        assert d.max().item() <= 2e-2 and d.mean().item() <= 5e-4, (t, d.max().item())
        for l in range(NL):
            ga, gb = general.get_indices(l), fused.get_indices(l)
            assert np.array_equal(np.sort(ga[:, :, L:L + M], axis=-1), np.sort(gb[:, :, L:L + M], axis=-1)), (t, l)
            assert (gb[:, :, L + M:] == -1)[:, labels[l] == 1].all()          # semantic heads: buffer empty
            # scores travel with the tokens: compare them by position
            sa, sb = general.get_scores(l), fused.get_scores(l)
            for s in range(S):
                for h in np.nonzero(labels[l])[0]:
                    a = dict(zip(ga[s, h, L:L + M].tolist(), sa[s, h, :M].tolist()))
                    b = dict(zip(gb[s, h, L:L + M].tolist(), sb[s, h, :M].tolist()))
                    assert a.keys() == b.keys()
                    assert all(abs(a[k] - b[k]) <= 1e-4 * max(abs(a[k]), 1e-3) for k in a), (t, l, s, h)
    assert general.device_status() == 0 and fused.device_status() == 0
    for c in caches:
        c.close()


def _run_full_launch_sampled(cfg, n_layers, seqs, sample, n_steps, form, evict=False):
    """The launch sizes the benchmark times (all `seqs` x all heads x `n_layers` layers), row-buffer mode;
    the oracle replays only the sampled (layer, sequence, head) pairs: every step's output, and the static
    set after every re-selection (exact outside the 1e-5 band, following the GPU's choice inside it).
    form: "per_layer" (ssd_append_decode per layer; ssd_recompress_layers when the buffer is full, after
    every step when evict) or "one_launch" (ssd_append_decode_layers; with evict it re-selects itself).
    Returns (re-selections replayed, of which inside the band)."""
    import dataclasses
    if evict:      # Algorithm 1 taken literally: a buffer of one token, same number of slots per head
        cfg = dataclasses.replace(cfg, sink_budget=cfg.sink_budget + cfg.sink_recent - 1, sink_recent=1,
                                  name=cfg.name + "_evict")
    dev = torch.device("cuda:0")
    L, n0, M, R, W, H, S = cfg.prompt_len, cfg.n0, cfg.sink_budget, cfg.sink_recent, cfg.window, cfg.n_heads, len(seqs)
    labels = np.stack([wl.sink_mask(cfg, l) for l in range(n_layers)])
    cache = B.SsdCache(B.config_from_workload(cfg, n_layers=n_layers, n_seqs=S),
                       n_sink_heads_total=int(labels.sum()), device=dev)
    cache.set_row_buffer(True)
    cache.set_head_labels(labels)
    step_in = [torch.empty((n_steps, n_layers, S, H, 128), dtype=torch.bfloat16, device=dev) for _ in range(3)]
    picked = {}
    for layer in range(n_layers):
        q, k, v, _ = wl.gen_layer(cfg, layer, seqs, device=dev)
        cache.compress(layer, q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0)
        step_in[0][:, layer] = q[:, :, n0:n0 + n_steps].permute(2, 0, 1, 3)
        step_in[1][:, layer] = k[:, :, L + n0:L + n0 + n_steps].permute(2, 0, 1, 3)
        step_in[2][:, layer] = v[:, :, L + n0:L + n0 + n_steps].permute(2, 0, 1, 3)
        for (l, s, h) in sample:
            if l == layer:
                picked[(l, s, h)] = (wl.to_u16(q[s, h]), wl.to_u16(k[s, h]), wl.to_u16(v[s, h]))
        del q, k, v
    assert len(picked) == len(sample)
    sample_layers = sorted({l for (l, _, _) in sample})
    outs = {key: [] for key in sample}
    gpu_sets = {}
    out = torch.empty((S, H, 128), dtype=torch.bfloat16, device=dev)
    for i in range(n_steps):
        t = n0 + 1 + i
        if form == "one_launch":
            o = cache.append_decode_layers(0, step_in[1][i], step_in[2][i], step_in[0][i])
            for key in sample:
                outs[key].append(o[key[0], key[1], key[2]].clone())
        else:
            for layer in range(n_layers):
                cache.append_decode(layer, step_in[1][i, layer], step_in[2][i, layer], step_in[0][i, layer], out)
                for key in sample:
                    if key[0] == layer:
                        outs[key].append(out[key[1], key[2]].clone())
        if (t - n0) % R == 0:
            if not (evict and form == "one_launch"):       # that launch has re-selected already
                cache.recompress_layers(0, n_layers)
            for layer in sample_layers:
                gi = cache.get_indices(layer)
                for (l, s, h) in sample:
                    if l == layer and labels[l][h]:
                        st = gi[s, h, L:L + M]
                        gpu_sets[(l, s, h, t)] = sorted((st[st >= 0] - L).tolist())
    assert cache.device_status() == 0
    t_end = n0 + n_steps
    n_resel, n_band = [0], [0]

    def chooser(key):
        def choose(t, cand, sc, keep):
            n_resel[0] += 1
            got, want = gpu_sets[key + (t,)], [cand[i] for i in keep]
            if got == want:
                return keep
            n_band[0] += 1
            kth = np.sort(sc)[::-1][len(keep) - 1]
            sure_in = {cand[i] for i in np.nonzero(sc > kth * (1 + BAND))[0]}
            band = {cand[i] for i in np.nonzero(np.abs(sc - kth) <= BAND * abs(kth))[0]}
            assert sure_in <= set(got) <= (sure_in | band) and len(got) == len(want), key
            return [cand.index(j) for j in got]
        return choose

    for key, (qu, ku, vu) in picked.items():
        l, s, h = key
        got = torch.stack(outs[key]).float().cpu().numpy().astype(np.float64)
        if labels[l][h]:
            want, _ = oracle.rowbuf_semantic(qu, ku, vu, L, n0, M, R, t_end, choose=chooser(key))
        else:
            want = np.stack([oracle.attend(qu[t - 1], ku, vu, oracle.retained_set(False, L, t, W, R))
                             for t in range(n0 + 1, t_end + 1)])
        err = np.abs(got - want)
        assert err.max() <= 2e-2 and err.mean() <= 2e-3, (key, err.max(), err.mean())
    cache.close()
    print(f"{cfg.name} {form}: {n_resel[0]} re-selections replayed, {n_band[0]} of them decided inside the tie band")
    return n_resel[0], n_band[0]


def _sample_of(cfg, layers, n_seqs, n_per_layer, seed):
    rng = np.random.default_rng(seed)
    sample = []
    for layer in layers:
        labels = wl.sink_mask(cfg, layer)
        for i in range(n_per_layer):
            heads = np.nonzero(labels == (1 if i % 3 else 0))[0]     # two semantic heads for every spatial one
            sample.append((layer, int(rng.integers(0, n_seqs)), int(rng.choice(heads))))
    return sorted(set(sample))


@pytest.mark.parametrize("form", ["per_layer", "one_launch"])
def test_rowbuf_janus7b_launch_size_sampled_pairs(form):
    """Algorithm 2 at the sizes the benchmark times: 30 layers x 64 sequences x 32 heads, one full buffer
    cycle and two steps of the next, ten sampled pairs against the oracle."""
    cfg = wl.CONFIGS["janus7b"]
    sample = _sample_of(cfg, (0, 7, 14, 22, 29), cfg.n_seqs, 3, seed=3)
    assert len(sample) >= 8
    n_resel, n_band = _run_full_launch_sampled(cfg, cfg.n_layers, list(range(cfg.n_seqs)), sample,
                                               cfg.sink_recent + 2, form)
    assert n_resel >= 8 and 0 <= n_band <= n_resel


@pytest.mark.parametrize("form", ["per_layer", "one_launch"])
def test_evict_every_step_janus7b_launch_size_sampled_pairs(form):
    """Algorithm 1 taken literally (a re-selection after every step) at the benchmark's sizes, ten steps."""
    cfg = wl.CONFIGS["janus7b"]
    sample = _sample_of(cfg, (0, 11, 19, 29), cfg.n_seqs, 3, seed=4)
    assert len(sample) >= 8
    n_resel, n_band = _run_full_launch_sampled(cfg, cfg.n_layers, list(range(cfg.n_seqs)), sample, 10, form, evict=True)
    assert n_resel >= 60 and 0 <= n_band <= n_resel


@pytest.mark.parametrize("form", ["per_layer", "one_launch"])
def test_rowbuf_hires7b_slice(form):
    """The 4096-token grid (M + R = 320 entries per score row): two layers, four sequences, a full buffer
    cycle of 64 steps and three more; four sampled pairs."""
    cfg = wl.CONFIGS["hires7b"]
    sample = _sample_of(cfg, (0, 1), 4, 2, seed=5)
    n_resel, n_band = _run_full_launch_sampled(cfg, 2, [0, 1, 2, 3], sample, cfg.sink_recent + 3, form)
    assert n_resel >= 2 and 0 <= n_band <= n_resel
