"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_18716_b200 import binding as B
from paper_2510_18716_b200 import workloads as wl

from parity_util import check_outputs, run_workload

pytestmark = pytest.mark.gpu


def test_tiny_every_step():
    cfg = wl.CONFIGS["tiny"]
    r = run_workload(cfg, [0], [0], check_steps=(), full_every_step=True, check_planted=True)
    assert r.steps_checked == cfg.n_img - cfg.n0 and r.n_pairs == 8


def test_tiny_fewer_observation_queries():
    cfg = wl.CONFIGS["tiny"]
    for n_obs in (1, 5, 0):
        run_workload(cfg, [0], [0], check_steps=(cfg.n0 + 1, cfg.n_img), classify=False, n_obs=n_obs)


def test_janus1b_sampled_layers_all_sequences():
    cfg = wl.CONFIGS["janus1b"]
    steps = (cfg.n0 + 1, cfg.n0 + 2, cfg.n0 + 25, cfg.n_img)
    r = run_workload(cfg, [0, 23], list(range(cfg.n_seqs)), steps, check_planted=True)
    assert r.steps_checked == 2 * len(steps)


def test_janus7b_sampled_layers_all_sequences():
    cfg = wl.CONFIGS["janus7b"]
    steps = (cfg.n0 + 1, cfg.n0 + 24, cfg.n_img)
    r = run_workload(cfg, [0, 29], list(range(cfg.n_seqs)), steps, check_planted=True)
    assert r.steps_checked == 2 * len(steps)


def test_hires7b_one_layer_two_sequences():
    cfg = wl.CONFIGS["hires7b"]
    steps = (cfg.n0 + 1, cfg.n0 + 65, cfg.n_img)
    run_workload(cfg, [0], [0, 1], steps, classify=False)


def test_sweep_points():
    for cfg, seqs in ((wl.sweep(32, 5, 0.25), [0, 1, 2, 3]), (wl.sweep(32, 10, 0.75), [0, 1]),
                      (wl.sweep(32, 2, 0.5), [5, 6])):
        run_workload(cfg, [3], seqs, (cfg.n0 + 1, cfg.n0 + 30, cfg.n_img), classify=False)


def _full_cache_case(cfg: wl.Workload, seqs, steps, one_launch=False):
    """Uncompressed baseline: every head spatial with W = N, prompt loaded with n0 = 0."""
    dev = torch.device("cuda:0")
    L, N, H, S = cfg.prompt_len, cfg.n_img, cfg.n_heads, len(seqs)
    c = B.make_config(1, S, H, L, N, N, 0, 1, cfg.cls_window, cfg.tau)
    cache = B.SsdCache(c)
    cache.set_head_labels(np.zeros(H, np.uint8))
    q, k, v, _ = wl.gen_layer(cfg, 0, seqs, device=dev)
    qu, ku, vu = wl.to_u16(q), wl.to_u16(k), wl.to_u16(v)
    cache.compress(0, None, k[:, :, :L].contiguous(), v[:, :, :L].contiguous(), 0, 0)
    sem = np.zeros((S, H), np.uint8)
    for t in range(1, N + 1):
        kt, vt = k[:, :, L + t - 1].contiguous(), v[:, :, L + t - 1].contiguous()
        if t not in steps:
            cache.append(0, kt, vt)
            continue
        if one_launch:
            out = cache.append_decode_layers(0, kt[None], vt[None], q[:, :, t - 1].contiguous()[None])[0]
        else:
            cache.append(0, kt, vt)
            out = cache.decode_attn(0, q[:, :, t - 1].contiguous())
        want = oracle.decode_batch(qu[:, :, t - 1], ku, vu, sem, None, None, L, t, N, 0, 1, full=True)
        check_outputs(out, want, f"full cache step {t}")
        assert (cache.get_lengths(0) == L + t).all()
    cache.close()


def test_full_cache_baseline_matches_full_attention():
    _full_cache_case(wl.CONFIGS["tiny"], [0], steps=range(1, 65))
    _full_cache_case(wl.CONFIGS["janus7b"], [0, 1, 2], steps=(1, 2, 7, 8, 9, 100, 333, 575, 576))
    _full_cache_case(wl.CONFIGS["tiny"], [0], steps=range(1, 65), one_launch=True)
    _full_cache_case(wl.CONFIGS["janus7b"], [0, 1, 2], steps=(1, 2, 7, 8, 9, 100, 333, 575, 576), one_launch=True)


def _small_cfg(seed):
    rng = np.random.default_rng(seed)
    h = int(rng.integers(2, 7))
    w = int(rng.integers(2, 7))
    N = h * w
    H = int(rng.integers(1, 6))
    n0 = int(rng.integers(0, N))
    return wl.Workload(f"rand{seed}", 1, int(rng.integers(1, 4)), H, int(rng.integers(0, 6)), (h, w),
                       int(rng.integers(1, N + 2)), int(rng.integers(0, N + 2)), int(rng.integers(1, 6)),
                       int(rng.integers(0, 8)), int(rng.integers(0, H + 1)), n0, 1, 1.0, seed=seed)


@pytest.mark.parametrize("seed", range(24))
def test_random_small_shapes(seed):
    cfg = _small_cfg(seed)
    if cfg.prompt_len + cfg.n0 == 0:
        pytest.skip("nothing to load")
    run_workload(cfg, [0], list(range(cfg.n_seqs)), (), classify=False, full_every_step=True,
                 n_obs=min(cfg.n0, seed % 5 + (cfg.n0 if seed % 2 else 0)),
                 step_form=("two", "fused", "layers")[seed % 3])      # every form of the step sees odd shapes


def test_decode_before_any_compress_fills_ring_from_zero():
    cfg = wl.CONFIGS["tiny"]
    dev = torch.device("cuda:0")
    L, N, H = cfg.prompt_len, cfg.n_img, cfg.n_heads
    cache = B.SsdCache(B.config_from_workload(cfg))
    labels = wl.sink_mask(cfg, 0)
    cache.set_head_labels(labels)
    q, k, v, _ = wl.gen_layer(cfg, 0, [0], device=dev)
    qu, ku, vu = wl.to_u16(q), wl.to_u16(k), wl.to_u16(v)
    with pytest.raises(B.SsdError) as e:
        cache.decode_attn(0, q[:, :, 0].contiguous())
    assert e.value.code == B.SSD_ERR_BAD_STATE
    sem = labels[None, :]
    for t in range(1, N + 1):
        cache.append(0, k[:, :, L + t - 1].contiguous(), v[:, :, L + t - 1].contiguous())
        out = cache.decode_attn(0, q[:, :, t - 1].contiguous())
        # no prompt, no static set: windows over image tokens only
        want = np.empty((1, H, 128))
        for h in range(H):
            capn = cfg.sink_recent if labels[h] else cfg.window
            pos = np.arange(max(0, t - capn), t, dtype=np.int32) + L
            want[0, h] = oracle.attend(qu[0, h, t - 1], ku[0, h], vu[0, h], pos)
        check_outputs(out, want, f"ring-only step {t}")
    with pytest.raises(B.SsdError) as e:
        cache.append(0, k[:, :, L].contiguous(), v[:, :, L].contiguous())
    assert e.value.code == B.SSD_ERR_OVERFLOW
    cache.close()


def test_hires7b_classifier_one_layer():
    """Head classification at the 4096-token grid (32 blocks of query rows per unit): sparsity values and
    labels of one layer's 32 heads over the configuration's calibration sequences, against the oracle."""
    from parity_util import check_labels
    cfg = wl.CONFIGS["hires7b"]
    dev = torch.device("cuda:0")
    qc, kc = wl.gen_calibration(cfg, [7], device=dev)
    cache = B.SsdCache(B.config_from_workload(cfg, n_layers=1, n_seqs=1))
    s_gpu, lab_gpu = cache.classify_heads(qc, kc)
    s_ora = oracle.sparsity(wl.to_u16(qc), wl.to_u16(kc), cfg.prompt_len, cfg.cls_window)
    labels = check_labels(s_gpu, lab_gpu, s_ora, cfg.tau)
    assert np.array_equal(labels[0], wl.sink_mask(cfg, 7)), "classifier must recover the generator's split"
    assert cache.device_status() == 0
    cache.close()


def test_classifier_scores_match_oracle_on_mixed_heads():
    # sparsity values themselves (not only labels), on data with no planted structure
    cfg = wl.Workload("cls", 2, 2, 5, 7, (6, 9), 8, 8, 4, 11, 0, 20, 3, 1.2, seed=7)
    dev = torch.device("cuda:0")
    qc, kc = wl.gen_calibration(cfg, [0, 1], device=dev)
    cache = B.SsdCache(B.config_from_workload(cfg))
    s_gpu, lab = cache.classify_heads(qc, kc)
    s_ora = oracle.sparsity(wl.to_u16(qc), wl.to_u16(kc), cfg.prompt_len, cfg.cls_window)
    assert np.allclose(s_gpu, s_ora, rtol=2e-4, atol=2e-5)
    sums = cache.classify_partial(qc[:, :2].contiguous(), kc[:, :2].contiguous())
    s2 = oracle.sparsity(wl.to_u16(qc[:, :2]), wl.to_u16(kc[:, :2]), cfg.prompt_len, cfg.cls_window)
    assert np.allclose(sums / (2 * cfg.n_img), s2, rtol=2e-4, atol=2e-5)
    cache.close()


def test_step_host_matches_device_path():
    cfg = wl.CONFIGS["tiny"]
    dev = torch.device("cuda:0")
    L, n0 = cfg.prompt_len, cfg.n0
    q, k, v, _ = wl.gen_layer(cfg, 0, [0], device=dev)
    outs = []
    for mode in ("device", "host"):
        cache = B.SsdCache(B.config_from_workload(cfg))
        cache.set_head_labels(wl.sink_mask(cfg, 0))
        cache.compress(0, q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0)
        res = []
        for t in range(n0 + 1, n0 + 6):
            qt, kt, vt = (x.contiguous() for x in (q[:, :, t - 1], k[:, :, L + t - 1], v[:, :, L + t - 1]))
            if mode == "device":
                cache.append(0, kt, vt)
                res.append(cache.decode_attn(0, qt).cpu())
            else:
                hq, hk, hv = (x.cpu().pin_memory() for x in (qt, kt, vt))
                ho = torch.empty_like(hq).pin_memory()
                cache.step_host(0, hq, hk, hv, ho)
                torch.cuda.synchronize()
                res.append(ho.clone())
        outs.append(res)
        cache.close()
    for a, b in zip(*outs):
        assert torch.equal(a, b)


def test_step_host_layers_matches_device_path():
    """Thirty-four layers (four groups: more than the staging ring holds, the last group short) from
    pinned host arrays in one call, several steps in a row, against per-layer calls on device
    tensors: bit-identical outputs."""
    import dataclasses
    cfg = dataclasses.replace(wl.CONFIGS["tiny"], n_layers=34, n_seqs=2)
    dev = torch.device("cuda:0")
    L, n0, nl, steps = cfg.prompt_len, cfg.n0, cfg.n_layers, 5
    data = [wl.gen_layer(cfg, l, range(cfg.n_seqs), device=dev) for l in range(nl)]
    labels = np.concatenate([wl.sink_mask(cfg, l) for l in range(nl)])
    caches = []
    for _ in range(2):
        cache = B.SsdCache(B.config_from_workload(cfg))
        cache.set_head_labels(labels)
        for l, (q, k, v, _) in enumerate(data):
            cache.compress(l, q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0)
        caches.append(cache)
    dev_cache, host_cache = caches
    for t in range(n0 + 1, n0 + 1 + steps):
        qs = torch.stack([data[l][0][:, :, t - 1] for l in range(nl)]).contiguous()
        ks = torch.stack([data[l][1][:, :, L + t - 1] for l in range(nl)]).contiguous()
        vs = torch.stack([data[l][2][:, :, L + t - 1] for l in range(nl)]).contiguous()
        want = torch.stack([dev_cache.append_decode(l, ks[l], vs[l], qs[l]) for l in range(nl)]).cpu()
        hq, hk, hv = (x.cpu().pin_memory() for x in (qs, ks, vs))
        ho = torch.zeros_like(hq).pin_memory()
        host_cache.step_host_layers(0, hq, hk, hv, ho)
        torch.cuda.synchronize()
        assert torch.equal(ho, want)
    # a sub-range of layers, and the full-layer guard
    hq1, hk1, hv1 = (x[2:4].contiguous().pin_memory() for x in (hq, hk, hv))   # the layers' own step inputs
    ho1 = torch.zeros_like(hq1).pin_memory()
    host_cache.step_host_layers(2, hq1, hk1, hv1, ho1)
    torch.cuda.synchronize()
    assert host_cache.tokens(2) == host_cache.tokens(0) + 1 and host_cache.tokens(4) == host_cache.tokens(0)
    lib = B.load()
    assert lib.ssd_step_host_layers(host_cache._h, 33, 2, hq1.data_ptr(), hk1.data_ptr(), hv1.data_ptr(), ho1.data_ptr(),
                                    None) == B.SSD_ERR_INVALID_ARG
    assert host_cache.device_status() == 0
    for c in caches:
        c.close()


def test_argument_errors_launch_nothing():
    cfg = B.make_config(2, 2, 4, 8, 16, 4, 4, 2)
    cache = B.SsdCache(cfg)
    dev = torch.device("cuda:0")
    x = torch.zeros((2, 4, 128), dtype=torch.bfloat16, device=dev)
    before = B.kernel_launch_count()
    for fn in (lambda: cache.append(0, x, x), lambda: cache.decode_attn(0, x)):
        with pytest.raises(B.SsdError) as e:
            fn()
        assert e.value.code == B.SSD_ERR_BAD_STATE          # no labels yet
    cache.set_head_labels(np.array([0, 1, 0, 1, 1, 1, 0, 0], np.uint8))
    for layer in (-1, 2):
        with pytest.raises(B.SsdError) as e:
            cache.append(layer, x, x)
        assert e.value.code == B.SSD_ERR_INVALID_ARG
    kf = torch.zeros((2, 4, 8 + 17, 128), dtype=torch.bfloat16, device=dev)
    with pytest.raises(B.SsdError) as e:
        cache.compress(0, None, kf, kf, 17, 0)               # n0 beyond max_image_tokens
    assert e.value.code == B.SSD_ERR_INVALID_ARG
    # the tensor-core kernels read their inputs through the TMA unit: misaligned tensors are refused
    lib = B.load()
    kok = torch.zeros((2, 4, 8 + 8, 128), dtype=torch.bfloat16, device=dev)
    pad = torch.zeros(2 * 4 * 16 * 128 + 8, dtype=torch.bfloat16, device=dev)
    off = pad.data_ptr() + 2                                # 2-byte aligned only
    st = torch.cuda.current_stream().cuda_stream
    assert lib.ssd_compress(cache._h, 0, kok.data_ptr(), off, kok.data_ptr(), 8, 8, st) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_compress(cache._h, 0, off, kok.data_ptr(), kok.data_ptr(), 8, 8, st) == B.SSD_ERR_INVALID_ARG
    sums = np.zeros(2 * 4, np.float64)
    assert lib.ssd_classify_partial(cache._h, off, kok.data_ptr(), 1, 8, sums.ctypes.data, st) == B.SSD_ERR_INVALID_ARG
    assert B.kernel_launch_count() == before
    assert cache.kv_bytes_per_seq() == ((8 + 4) * 4 + (8 + 6) * 4) * 512
    cache.close()
    bad = B.make_config(1, 1, 1, 0, 4, 1, 1, 1, head_dim=64)
    assert B.required_bytes(bad) == 0


@pytest.mark.parametrize("kind", ["all_spatial", "all_semantic", "random"])
def test_other_head_partitions(kind):
    """The paper's ablation assigns heads at random with the same policies (Sec. 4.4); all-spatial is a
    sliding-window cache for every head and all-semantic a heavy-hitter cache for every head.  The
    policies do not depend on what the heads' data look like, so parity must hold for any labelling."""
    for name, layers, seqs in (("tiny", [0], [0]), ("janus1b", [5], [0, 1, 2])):
        cfg = wl.CONFIGS[name]
        H = cfg.n_heads
        if kind == "all_spatial":
            lab = np.zeros((len(layers), H), np.uint8)
        elif kind == "all_semantic":
            lab = np.ones((len(layers), H), np.uint8)
        else:
            from paper_2510_18716_b200 import ablation
            lab = ablation.random_partition(np.stack([wl.sink_mask(cfg, l) for l in layers]), seed=123)
        r = run_workload(cfg, layers, seqs, (cfg.n0 + 1, cfg.n0 + 9, cfg.n_img), classify=False, labels_override=lab)
        assert r.steps_checked == 3 * len(layers)


@pytest.mark.parametrize("case", ["tiny_compressed", "tiny_ring_from_zero", "janus7b_slice"])
def test_fused_append_decode_matches_the_two_calls(case):
    """ssd_append_decode must give the bits of ssd_append + ssd_decode_attn at every step, and leave
    the same cache behind (later steps read the token that the fused kernel stored)."""
    dev = torch.device("cuda:0")
    if case == "janus7b_slice":
        cfg, seqs, n_steps = wl.CONFIGS["janus7b"], [0, 1, 2, 3, 4], 30
    else:
        cfg, seqs, n_steps = wl.CONFIGS["tiny"], [0], 32
    L, n0 = cfg.prompt_len, cfg.n0
    q, k, v, _ = wl.gen_layer(cfg, 0, seqs, device=dev)
    caches = []
    for _ in range(2):
        c = B.SsdCache(B.config_from_workload(cfg, n_layers=1, n_seqs=len(seqs)), device=dev)
        c.set_head_labels(wl.sink_mask(cfg, 0))
        if case == "tiny_ring_from_zero":
            t0 = 0                       # no compress: prompt slots unused, rings fill from empty
        else:
            t0 = n0
            c.compress(0, q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0)
        caches.append(c)
    two, fused = caches
    for t in range(t0 + 1, t0 + n_steps + 1):
        kt, vt, qt = (x.contiguous() for x in (k[:, :, L + t - 1], v[:, :, L + t - 1], q[:, :, t - 1]))
        two.append(0, kt, vt)
        want = two.decode_attn(0, qt)
        got = fused.append_decode(0, kt, vt, qt)
        assert torch.equal(got, want), f"step {t}"
        assert fused.tokens(0) == two.tokens(0) == t
    assert np.array_equal(fused.get_indices(0), two.get_indices(0))
    # the fused cache is a full substitute: switch roles for a few more steps
    for t in range(t0 + n_steps + 1, min(t0 + n_steps + 4, cfg.n_img) + 1):
        kt, vt, qt = (x.contiguous() for x in (k[:, :, L + t - 1], v[:, :, L + t - 1], q[:, :, t - 1]))
        fused.append(0, kt, vt)
        a = fused.decode_attn(0, qt)
        b = two.append_decode(0, kt, vt, qt)
        assert torch.equal(a, b), f"step {t} after switching roles"
    assert fused.device_status() == 0 and two.device_status() == 0
    for c in caches:
        c.close()


def _sample_pairs(cfg, layer, n, seed):
    rng = np.random.default_rng(seed)
    labels = wl.sink_mask(cfg, layer)
    sem_heads, spa_heads = np.nonzero(labels)[0], np.nonzero(labels == 0)[0]
    pairs = []
    for i in range(n):
        heads = sem_heads if (i % 2 == 0 and len(sem_heads)) else spa_heads
        pairs.append((int(rng.integers(0, cfg.n_seqs)), int(rng.choice(heads))))
    return pairs


def test_hires7b_full_launch_size_sampled_pairs():
    cfg = wl.CONFIGS["hires7b"]
    from parity_util import run_sampled
    run_sampled(cfg, 7, _sample_pairs(cfg, 7, 6, 1), (cfg.n0 + 1, cfg.n0 + 70))


def test_sweep_batch128_full_launch_size_sampled_pairs():
    cfg = wl.sweep(128, 5, 0.5)
    from parity_util import run_sampled
    run_sampled(cfg, 2, _sample_pairs(cfg, 2, 8, 2), (cfg.n0 + 1, cfg.n0 + 26))


@pytest.mark.parametrize("name,layer,n_seqs", [("janus7b", 11, 64), ("hires7b", 2, 2)])
def test_compress_scores_elementwise(name, layer, n_seqs):
    """Algorithm 1, AttentionScores summed over the observed steps: the score rows ssd_compress selects
    from, element by element against the oracle (not only through the sets they produce)."""
    cfg = wl.CONFIGS[name]
    dev = torch.device("cuda:0")
    L, n0, M, R, H = cfg.prompt_len, cfg.n0, cfg.sink_budget, cfg.sink_recent, cfg.n_heads
    labels = wl.sink_mask(cfg, layer)
    cache = B.SsdCache(B.config_from_workload(cfg, n_layers=1, n_seqs=n_seqs), device=dev)
    cache.set_head_labels(labels)
    with pytest.raises(B.SsdError) as e:
        cache.get_compress_scores(0, n0)                 # nothing compressed yet
    assert e.value.code == B.SSD_ERR_BAD_STATE
    q, k, v, _ = wl.gen_layer(cfg, layer, list(range(n_seqs)), device=dev)
    cache.compress(0, q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0)
    got = cache.get_compress_scores(0, n0)
    assert cache.device_status() == 0
    cache.compress(0, q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0)
    assert np.array_equal(got, cache.get_compress_scores(0, n0)), "scores must be reproducible bit for bit"

    sem = labels[None, :].repeat(n_seqs, 0).astype(np.uint8)
    want, _, _ = oracle.select_batch(wl.to_u16(q[:, :, :n0]), wl.to_u16(k[:, :, : L + n0]), sem, L, n0, M, R)
    for h in range(H):
        if labels[h]:
            assert np.allclose(got[:, h], want[:, h], rtol=2e-4, atol=1e-7), (h, np.abs(got[:, h] - want[:, h]).max())
            assert (got[:, h] >= 0).all()
        else:
            assert (got[:, h] == -1).all()
    cache.close()


def test_compress_scores_with_large_logits():
    """Queries eight times larger (an exact scaling in bf16): row maxima of several hundred in base-2 units, so
    the normalisers the second sweep subtracts are large numbers and most probabilities underflow.  The score rows
    must still match the oracle element by element and contain nothing that is not a finite non-negative number."""
    cfg = wl.CONFIGS["janus1b"]
    dev = torch.device("cuda:0")
    L, n0, M, R, H, layer, n_seqs = cfg.prompt_len, cfg.n0, cfg.sink_budget, cfg.sink_recent, cfg.n_heads, 3, 2
    labels = wl.sink_mask(cfg, layer)
    cache = B.SsdCache(B.config_from_workload(cfg, n_layers=1, n_seqs=n_seqs), device=dev)
    cache.set_head_labels(labels)
    q, k, v, _ = wl.gen_layer(cfg, layer, list(range(n_seqs)), device=dev)
    q = (q.float() * 8.0).to(torch.bfloat16)
    cache.compress(0, q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0)
    got = cache.get_compress_scores(0, n0)
    assert cache.device_status() == 0
    sem = labels[None, :].repeat(n_seqs, 0).astype(np.uint8)
    want, _, _ = oracle.select_batch(wl.to_u16(q[:, :, :n0]), wl.to_u16(k[:, :, : L + n0]), sem, L, n0, M, R)
    for h in range(H):
        if labels[h]:
            assert np.isfinite(got[:, h]).all() and (got[:, h] >= 0).all()
            assert np.allclose(got[:, h], want[:, h], rtol=2e-4, atol=1e-7), (h, np.abs(got[:, h] - want[:, h]).max())
    cache.close()


def test_exact_ties_on_the_radix_path_select_the_lowest_indices():
    """Algorithm 1, IndicesOfTopM with the lowest-index tie rule, where the selection radix-selects the
    threshold (more than 1024 candidates): with no observed step every score is zero, all candidates tie,
    and the M lowest must be kept."""
    cfg = wl.CONFIGS["hires7b"]
    dev = torch.device("cuda:0")
    L, n0, M, R, H = cfg.prompt_len, cfg.n0, cfg.sink_budget, cfg.sink_recent, cfg.n_heads
    assert n0 - R > 1024
    labels = wl.sink_mask(cfg, 0)
    cache = B.SsdCache(B.config_from_workload(cfg, n_layers=1, n_seqs=1), device=dev)
    cache.set_head_labels(labels)
    _, k, v, _ = wl.gen_layer(cfg, 0, [0], device=dev)
    cache.compress(0, None, k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0, 0)
    gi = cache.get_indices(0)
    want = oracle.topm(np.zeros(n0 - R), n0 - R, M)
    assert np.array_equal(want, np.arange(M))
    for h in range(H):
        if labels[h]:
            assert np.array_equal(gi[0, h, L:L + M] - L, want), h
    assert cache.device_status() == 0
    cache.close()


@pytest.mark.parametrize("frac", [0.25, 0.75])
def test_sweep_point_through_the_classifier(frac):
    """A point of the large-batch sweep with a quarter / three quarters of the heads semantic: the
    classifier has to recover that split (and everything after it is checked as usual)."""
    cfg = wl.sweep(32, 5, frac)
    assert cfg.n_sink_heads == round(frac * cfg.n_heads)
    r = run_workload(cfg, [3, 17], [0, 1], (cfg.n0 + 1, cfg.n_img), classify=True)
    assert r.steps_checked == 4


def test_append_refuses_misaligned_rows_before_any_launch():
    cfg = wl.CONFIGS["tiny"]
    dev = torch.device("cuda:0")
    cache = B.SsdCache(B.config_from_workload(cfg), device=dev)
    cache.set_head_labels(wl.sink_mask(cfg, 0))
    x = torch.zeros((cfg.n_seqs * cfg.n_heads * 128 + 8,), dtype=torch.bfloat16, device=dev)
    lib, st = B.load(), torch.cuda.current_stream().cuda_stream
    before = B.kernel_launch_count()
    assert lib.ssd_append(cache._h, 0, x.data_ptr() + 2, x.data_ptr(), st) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_append(cache._h, 0, x.data_ptr(), x.data_ptr() + 2, st) == B.SSD_ERR_INVALID_ARG
    assert B.kernel_launch_count() == before and cache.tokens(0) == 0
    assert lib.ssd_append(cache._h, 0, x.data_ptr(), x.data_ptr(), st) == B.SSD_OK
    cache.close()
