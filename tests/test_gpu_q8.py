"""GPU parity of the 8-bit K/V format (an extension; the paper cites quantisation as related work, Sec. 2):
the quantiser's codes and scales bit for bit against the oracle, and decode attention over the quantised store
against fp64 attention over the oracle's dequantised rows."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_18716_b200 import binding as B
from paper_2510_18716_b200 import workloads as wl

from parity_util import MAX_ABS, MEAN_ABS

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("n_rows", [1, 17, 1000])
def test_quantiser_codes_and_scales_are_the_oracles(n_rows):
    dev = torch.device("cuda:0")
    g = torch.Generator(device=dev).manual_seed(n_rows)
    mag = torch.logspace(-4, 3, n_rows, device=dev)[:, None]
    rows = (torch.randn((n_rows, 128), generator=g, device=dev) * mag).to(torch.bfloat16)
    if n_rows > 4:
        rows[3] = 0                                   # a row of zeros: scale 0, codes 0
        rows[4, 7] = rows[4].abs().max() * 2          # one dominant element
    codes, scales = B.quantize_rows_e4m3(rows)
    want_c, want_s = oracle.kv_quantize_rows(wl.to_u16(rows))
    assert np.array_equal(scales.cpu().numpy(), want_s)
    assert np.array_equal(codes.cpu().numpy(), want_c)


def _dequantised(rows_u16):
    """A row is quantised once, when it enters the cache, whatever step that is: the oracle's codes for all of them."""
    codes, scale = oracle.kv_quantize_rows(rows_u16)
    return oracle.kv_dequantize(codes, scale)


def _pair_reference(cfg, qu, Kq, Vq, is_sem, gidx_row, t):
    """fp64 attention of one (sequence, head) at image step t over the oracle's dequantised rows."""
    pos = oracle.retained_set(bool(is_sem), cfg.prompt_len, t, cfg.window, cfg.sink_recent, gidx_row)
    return oracle.attend_values(qu[t - 1], Kq, Vq, pos)


def _run(cfg, n_layers, seqs, steps, form, sample=None):
    dev = torch.device("cuda:0")
    L, n0, M, H, S = cfg.prompt_len, cfg.n0, cfg.sink_budget, cfg.n_heads, len(seqs)
    labels = np.stack([wl.sink_mask(cfg, l) for l in range(n_layers)])
    cache = B.SsdCache(B.config_from_workload(cfg, n_layers=n_layers, n_seqs=S), device=dev)
    cache.set_kv_format(1)
    cache.set_head_labels(labels)
    data = []
    for l in range(n_layers):
        q, k, v, _ = wl.gen_layer(cfg, l, seqs, device=dev)
        cache.compress(l, q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0)
        data.append((q, k, v))
    assert cache.kv_bytes_per_seq() == sum(int(L * H + labels[l].sum() * (M + cfg.sink_recent) +
                                               (H - labels[l].sum()) * cfg.window) for l in range(n_layers)) * 272
    gsets = [cache.get_indices(l) for l in range(n_layers)]
    if sample is None:
        sample = [(l, s, h) for l in range(n_layers) for s in range(S) for h in range(H)]
    host = {}
    worst = 0.0
    for t in range(n0 + 1, n0 + steps + 1):
        qs = torch.stack([d[0][:, :, t - 1] for d in data]).contiguous()
        ks = torch.stack([d[1][:, :, L + t - 1] for d in data]).contiguous()
        vs = torch.stack([d[2][:, :, L + t - 1] for d in data]).contiguous()
        if form == "layers":
            out = cache.append_decode_layers(0, ks, vs, qs)
        else:
            out = torch.stack([cache.append_decode(l, ks[l], vs[l], qs[l]) for l in range(n_layers)])
            if t == n0 + steps:
                # attention alone over the store the fused call left behind: same shares, same codes, same bits
                for l in range(n_layers):
                    assert torch.equal(cache.decode_attn(l, qs[l]), out[l])
        out = out.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(out).all()
        for (l, s, h) in sample:
            if (l, s, h) not in host:
                q, k, v = data[l]
                host[(l, s, h)] = (wl.to_u16(q[s, h]), _dequantised(wl.to_u16(k[s, h])), _dequantised(wl.to_u16(v[s, h])))
            qu, ku, vu = host[(l, s, h)]
            st = gsets[l][s, h, L:L + M]
            want = _pair_reference(cfg, qu, ku, vu, labels[l][h], (st[st >= 0] - L).astype(np.int32), t)
            err = np.abs(out[l, s, h] - want)
            worst = max(worst, err.max())
            assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (l, s, h, t, err.max(), err.mean())
    for l in range(n_layers):
        assert cache.tokens(l) == n0 + steps
    assert cache.device_status() == 0
    cache.close()
    return worst


@pytest.mark.parametrize("form", ["layers", "per_layer"])
def test_q8_tiny_every_step(form):
    cfg = wl.CONFIGS["tiny"]
    _run(cfg, 2, [0, 1], cfg.n_img - cfg.n0, form)


@pytest.mark.parametrize("form", ["layers", "per_layer"])
def test_q8_janus7b_slice(form):
    cfg = wl.CONFIGS["janus7b"]
    rng = np.random.default_rng(2)
    sample = [(int(rng.integers(0, 3)), int(rng.integers(0, 4)), int(rng.integers(0, 32))) for _ in range(12)]
    _run(cfg, 3, [0, 1, 2, 3], 70, form, sample)            # past one turn of the 64-slot rings


@pytest.mark.parametrize("form", ["layers", "per_layer"])
def test_q8_janus7b_launch_size_sampled_pairs(form):
    """The launches the benchmark's 8-bit leg times: 30 layers x 64 sequences x 32 heads, in one launch and as one
    launch per layer (every share boundary of the full-size layer cuts a head)."""
    cfg = wl.CONFIGS["janus7b"]
    rng = np.random.default_rng(6)
    sample = [(l, int(rng.integers(0, 64)), int(rng.integers(0, 32))) for l in (0, 9, 17, 29) for _ in range(2)]
    _run(cfg, cfg.n_layers, list(range(cfg.n_seqs)), 3, form, sample)


def test_q8_every_pair_of_a_full_size_layer():
    """One janus7b layer at full width (64 sequences: 1628 shares, most heads cut once, some crossing thread
    blocks), every (sequence, head) of the per-layer form against the one-launch form, which cuts no head: the two
    differ only in the order of the partial sums: at most one bf16 rounding step per element."""
    cfg = wl.CONFIGS["janus7b"]
    dev = torch.device("cuda:0")
    L, n0, S = cfg.prompt_len, cfg.n0, cfg.n_seqs
    caches = []
    q, k, v, _ = wl.gen_layer(cfg, 0, range(S), device=dev)
    for _ in range(2):
        cache = B.SsdCache(B.config_from_workload(cfg, n_layers=1), device=dev)
        cache.set_kv_format(1)
        cache.set_head_labels(wl.sink_mask(cfg, 0)[None])
        cache.compress(0, q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0)
        caches.append(cache)
    for t in range(n0 + 1, n0 + 4):
        args = (k[:, :, L + t - 1].contiguous(), v[:, :, L + t - 1].contiguous(), q[:, :, t - 1].contiguous())
        a = caches[0].append_decode(0, *args).float()
        b = caches[1].append_decode_layers(0, *(x[None] for x in args))[0].float()
        # bf16 outputs: the two orders of summation may round an element to neighbouring values (one unit in the last
        # place, 2^-8 of its magnitude), nothing more
        err = (a - b).abs()
        assert bool((err <= torch.clamp(b.abs() * 2.0 ** -7, min=MAX_ABS / 4)).all()), (t, err.max().item())
        assert err.mean().item() <= MEAN_ABS / 4, (t, err.mean().item())
    assert caches[0].device_status() == 0
    for c in caches:
        c.close()


def test_q8_unsupported_calls_are_refused():
    cfg = wl.CONFIGS["tiny"]
    dev = torch.device("cuda:0")
    cache = B.SsdCache(B.config_from_workload(cfg), device=dev)
    cache.set_kv_format(1)
    cache.set_head_labels(wl.sink_mask(cfg, 0))
    x = torch.zeros((cfg.n_seqs, cfg.n_heads, 128), dtype=torch.bfloat16, device=dev)
    lib, st = B.load(), torch.cuda.current_stream().cuda_stream
    before = B.kernel_launch_count()
    assert lib.ssd_append(cache._h, 0, x.data_ptr(), x.data_ptr(), st) == B.SSD_ERR_BAD_STATE
    assert lib.ssd_decode_attn_static(cache._h, 0, x.data_ptr(), x.data_ptr(), st) == B.SSD_ERR_BAD_STATE
    assert lib.ssd_cache_set_row_buffer(cache._h, 1) == B.SSD_ERR_BAD_STATE
    assert lib.ssd_cache_set_kv_format(cache._h, 2) == B.SSD_ERR_INVALID_ARG
    assert B.kernel_launch_count() == before
    cache.set_kv_format(0)
    cache.set_row_buffer(True)
    assert lib.ssd_cache_set_kv_format(cache._h, 1) == B.SSD_ERR_BAD_STATE
    cache.close()


@pytest.mark.parametrize("mode", ["q8", "row_buffer"])
def test_step_from_host_buffers_in_the_other_modes(mode):
    """ssd_step_host_layers issues the per-layer calls itself, so it serves the 8-bit format and the row-buffer mode
    too: same bits as the per-layer calls on device tensors, several steps in a row."""
    import dataclasses
    cfg = dataclasses.replace(wl.CONFIGS["tiny"], n_layers=6, n_seqs=2)
    dev = torch.device("cuda:0")
    L, n0, nl = cfg.prompt_len, cfg.n0, cfg.n_layers
    data = [wl.gen_layer(cfg, l, range(cfg.n_seqs), device=dev) for l in range(nl)]
    labels = np.concatenate([wl.sink_mask(cfg, l) for l in range(nl)])
    caches = []
    for _ in range(2):
        cache = B.SsdCache(B.config_from_workload(cfg), device=dev)
        if mode == "q8":
            cache.set_kv_format(1)
        else:
            cache.set_row_buffer(True)
        cache.set_head_labels(labels)
        for l, (q, k, v, _) in enumerate(data):
            cache.compress(l, q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0)
        caches.append(cache)
    dev_cache, host_cache = caches
    for t in range(n0 + 1, n0 + 6):
        qs = torch.stack([data[l][0][:, :, t - 1] for l in range(nl)]).contiguous()
        ks = torch.stack([data[l][1][:, :, L + t - 1] for l in range(nl)]).contiguous()
        vs = torch.stack([data[l][2][:, :, L + t - 1] for l in range(nl)]).contiguous()
        want = torch.stack([dev_cache.append_decode(l, ks[l], vs[l], qs[l]) for l in range(nl)]).cpu()
        hq, hk, hv = (x.cpu().pin_memory() for x in (qs, ks, vs))
        ho = torch.zeros_like(hq).pin_memory()
        host_cache.step_host_layers(0, hq, hk, hv, ho)
        torch.cuda.synchronize()
        assert torch.equal(ho, want), t
    for l in range(nl):
        assert np.array_equal(dev_cache.get_indices(l), host_cache.get_indices(l))
    if mode == "row_buffer":
        assert np.allclose(dev_cache.get_scores(2), host_cache.get_scores(2), rtol=0, atol=0)
    assert dev_cache.device_status() == 0 and host_cache.device_status() == 0
    for c in caches:
        c.close()
