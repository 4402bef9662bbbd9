"""The one-launch-per-step form (ssd_append_decode_layers) against the per-layer calls and the oracle.

A head is summed by a single warp there and by up to several here, so the two GPU paths agree up to
the rounding order of the softmax sums, not bit for bit; both must meet the oracle's bar, and both
must leave the same cache behind."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2510_18716_b200 import binding as B
from paper_2510_18716_b200 import workloads as wl

from parity_util import check_outputs

pytestmark = pytest.mark.gpu


def _labels(cfg, kind, n_layers):
    H = cfg.n_heads
    if kind == "generator":
        return np.stack([wl.sink_mask(cfg, l) for l in range(n_layers)])
    # layers that differ in layout: the generator's split, all spatial, all semantic, a random one
    rng = np.random.default_rng(5)
    rows = [wl.sink_mask(cfg, 0), np.zeros(H, np.uint8), np.ones(H, np.uint8), rng.integers(0, 2, H).astype(np.uint8)]
    return np.stack([rows[l % 4] for l in range(n_layers)])


@pytest.mark.parametrize("case", ["tiny_mixed_layouts", "tiny_ring_from_zero", "janus7b_slice"])
def test_layers_launch_matches_per_layer_calls_and_oracle(case):
    dev = torch.device("cuda:0")
    if case == "janus7b_slice":
        cfg, nl, seqs, n_steps, kind = wl.CONFIGS["janus7b"], 3, list(range(6)), 20, "generator"
    else:
        cfg, nl, seqs, n_steps, kind = wl.CONFIGS["tiny"], 4, [0, 1], 28, "mixed"
    L, N, n0, W, M, R, H, S = (cfg.prompt_len, cfg.n_img, cfg.n0, cfg.window, cfg.sink_budget, cfg.sink_recent,
                               cfg.n_heads, len(seqs))
    labels = _labels(cfg, kind, nl)
    data = [wl.gen_layer(cfg, l, seqs, device=dev) for l in range(nl)]
    compressed = case != "tiny_ring_from_zero"
    t0 = n0 if compressed else 0
    caches = []
    for _ in range(2):
        c = B.SsdCache(B.config_from_workload(cfg, n_layers=nl, n_seqs=S), device=dev)
        c.set_head_labels(labels)
        if compressed:
            for l, (q, k, v, _) in enumerate(data):
                c.compress(l, q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0)
        caches.append(c)
    per_layer, fused = caches
    gidx, gcnt = [], []
    for l in range(nl):
        gi = fused.get_indices(l)
        idx = np.full((S, H, M), -1, np.int32)
        for h in range(H):
            if labels[l][h]:
                st = gi[:, h, L:L + M]
                idx[:, h] = np.where(st >= 0, st - L, -1)
        gidx.append(idx)
        gcnt.append((idx >= 0).sum(-1).astype(np.int32))
    oracle_steps = {t0 + 1, t0 + n_steps // 2, t0 + n_steps}
    for t in range(t0 + 1, t0 + n_steps + 1):
        qs = torch.stack([data[l][0][:, :, t - 1] for l in range(nl)]).contiguous()
        ks = torch.stack([data[l][1][:, :, L + t - 1] for l in range(nl)]).contiguous()
        vs = torch.stack([data[l][2][:, :, L + t - 1] for l in range(nl)]).contiguous()
        want = torch.stack([per_layer.append_decode(l, ks[l], vs[l], qs[l]) for l in range(nl)])
        got = fused.append_decode_layers(0, ks, vs, qs)
        d = (got.float() - want.float()).abs()
        assert torch.isfinite(got.float()).all()
        assert d.max().item() <= 2e-2 and d.mean().item() <= 5e-4, f"step {t}: {d.max().item()} {d.mean().item()}"
        for l in range(nl):
            assert fused.tokens(l) == per_layer.tokens(l) == t
        if t in oracle_steps and compressed:
            for l in range(nl):
                q, k, v, _ = data[l]
                sem = labels[l][None, :].repeat(S, 0).astype(np.uint8)
                ref = oracle.decode_batch(wl.to_u16(q)[:, :, t - 1], wl.to_u16(k), wl.to_u16(v), sem, gidx[l], gcnt[l],
                                          L, t, W, M, R)
                check_outputs(got[l], ref, f"layer {l} step {t}")
    for l in range(nl):
        assert np.array_equal(fused.get_indices(l), per_layer.get_indices(l))
    # the cache it leaves is a full substitute: per-layer calls on it continue bit for bit
    t = t0 + n_steps + 1
    if t <= N:
        for l in range(nl):
            kt, vt, qt = (x.contiguous() for x in (data[l][1][:, :, L + t - 1], data[l][2][:, :, L + t - 1],
                                                   data[l][0][:, :, t - 1]))
            assert torch.equal(fused.append_decode(l, kt, vt, qt), per_layer.append_decode(l, kt, vt, qt))
    # layers need not be at the same step: layer 0 runs one step ahead, then one launch serves them all
    if t + 2 <= N:
        step_of = [t + 2] + [t + 1] * (nl - 1)
        kt, vt, qt = (x.contiguous() for x in (data[0][1][:, :, L + t], data[0][2][:, :, L + t], data[0][0][:, :, t]))
        assert torch.equal(fused.append_decode(0, kt, vt, qt), per_layer.append_decode(0, kt, vt, qt))
        qs = torch.stack([data[l][0][:, :, step_of[l] - 1] for l in range(nl)]).contiguous()
        ks = torch.stack([data[l][1][:, :, L + step_of[l] - 1] for l in range(nl)]).contiguous()
        vs = torch.stack([data[l][2][:, :, L + step_of[l] - 1] for l in range(nl)]).contiguous()
        want = torch.stack([per_layer.append_decode(l, ks[l], vs[l], qs[l]) for l in range(nl)])
        got = fused.append_decode_layers(0, ks, vs, qs)
        d = (got.float() - want.float()).abs()
        assert d.max().item() <= 2e-2 and d.mean().item() <= 5e-4
        assert [fused.tokens(l) for l in range(nl)] == step_of == [per_layer.tokens(l) for l in range(nl)]
        for l in range(nl):
            assert np.array_equal(fused.get_indices(l), per_layer.get_indices(l))
    assert fused.device_status() == 0 and per_layer.device_status() == 0
    for c in caches:
        c.close()


def test_layers_launch_argument_errors():
    cfg = dataclasses.replace(wl.CONFIGS["tiny"], n_layers=2)
    dev = torch.device("cuda:0")
    c = B.SsdCache(B.config_from_workload(cfg, n_layers=2, n_seqs=1), device=dev)
    x = torch.zeros((2, 1, cfg.n_heads, 128), dtype=torch.bfloat16, device=dev)
    lib = B.load()
    args = (x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), torch.cuda.current_stream().cuda_stream)
    before = B.kernel_launch_count()
    assert lib.ssd_append_decode_layers(c._h, 0, 2, *args) == B.SSD_ERR_BAD_STATE      # no labels yet
    c.set_head_labels(np.stack([wl.sink_mask(cfg, l) for l in range(2)]))
    assert lib.ssd_append_decode_layers(c._h, 1, 2, *args) == B.SSD_ERR_INVALID_ARG    # past the last layer
    assert lib.ssd_append_decode_layers(c._h, 0, 0, *args) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_append_decode_layers(c._h, 0, 2, x.data_ptr() + 2, *args[1:]) == B.SSD_ERR_INVALID_ARG   # misaligned
    assert B.kernel_launch_count() == before
    c.close()
    # a score row that a warp cannot keep in shared memory is a documented limit, not a launch failure: with a
    # buffer of one token the one-launch step needs three rows of M + 1 entries (rounded up to 4) per warp
    big = B.make_config(1, 1, 2, 4, 1300, 8, 1100, 1)
    c = B.SsdCache(big, device=dev)
    c.set_row_buffer(True)
    c.set_head_labels(np.ones(2, np.uint8))
    y = torch.zeros((1, 1, 2, 128), dtype=torch.bfloat16, device=dev)
    before = B.kernel_launch_count()
    assert lib.ssd_append_decode_layers(c._h, 0, 1, y.data_ptr(), y.data_ptr(), y.data_ptr(), y.data_ptr(),
                                        torch.cuda.current_stream().cuda_stream) == B.SSD_ERR_LIMIT
    assert B.kernel_launch_count() == before
    c.close()


@pytest.mark.parametrize("name,form", [("janus7b", "one_launch"), ("janus7b", "per_layer"), ("janus1b", "per_layer"),
                                       ("hires7b", "per_layer"), ("hires7b", "one_launch")])
def test_whole_step_launch_size_sampled_pairs(name, form):
    """The launches the benchmark times, at every workload's full size (all layers x all sequences x all heads):
    one launch per layer (ssd_append_decode, the headline form) or the whole step in one launch.  The oracle
    recomputes sampled (layer, sequence, head) pairs one by one: their selected sets (exact outside the tie
    band) and their outputs at three steps."""
    from parity_util import MAX_ABS, MEAN_ABS, bf16_to_f64, check_index_sets
    cfg = wl.CONFIGS[name]
    dev = torch.device("cuda:0")
    L, N, n0, W, M, R, H, S, NL = (cfg.prompt_len, cfg.n_img, cfg.n0, cfg.window, cfg.sink_budget, cfg.sink_recent,
                                   cfg.n_heads, cfg.n_seqs, cfg.n_layers)
    n_steps = 3
    labels = np.stack([wl.sink_mask(cfg, l) for l in range(NL)])
    rng = np.random.default_rng(42)
    sample = {}
    some_layers = sorted({0, NL // 3, (2 * NL) // 3, NL - 1})
    for i, layer in enumerate(sorted(some_layers * (2 if name != "hires7b" else 1))):
        heads = np.nonzero(labels[layer] == (i % 2))[0]         # alternately a spatial and a semantic head
        sample.setdefault(layer, []).append((int(rng.integers(0, S)), int(rng.choice(heads))))
    cache = B.SsdCache(B.config_from_workload(cfg), n_sink_heads_total=int(labels.sum()), device=dev)
    cache.set_head_labels(labels)
    step_in = [torch.empty((n_steps, NL, S, H, 128), dtype=torch.bfloat16, device=dev) for _ in range(3)]
    picked = {}
    n_cand = max(n0 - R, 0)
    for layer in range(NL):
        q, k, v, _ = wl.gen_layer(cfg, layer, list(range(S)), device=dev)
        cache.compress(layer, q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0)
        step_in[0][:, layer] = q[:, :, n0:n0 + n_steps].permute(2, 0, 1, 3)
        step_in[1][:, layer] = k[:, :, L + n0:L + n0 + n_steps].permute(2, 0, 1, 3)
        step_in[2][:, layer] = v[:, :, L + n0:L + n0 + n_steps].permute(2, 0, 1, 3)
        if layer in sample:
            gi = cache.get_indices(layer)
            for (s, h) in sample[layer]:
                qu, ku, vu = wl.to_u16(q[s, h]), wl.to_u16(k[s, h]), wl.to_u16(v[s, h])
                sem = np.array([[labels[layer][h]]], np.uint8)
                gidx = np.full((1, 1, M), -1, np.int32)
                if labels[layer][h]:
                    st = gi[s, h, L:L + M]
                    gidx[0, 0] = np.where(st >= 0, st - L, -1)
                    sc, oidx, ocnt = oracle.select_batch(qu[None, None, :n0], ku[None, None, : L + n0], sem, L, n0, M, R)
                    check_index_sets(gidx, sc, oidx, ocnt, sem, n_cand, M)
                picked[(layer, s, h)] = (qu, ku, vu, sem, gidx, (gidx >= 0).sum(-1).astype(np.int32))
        del q, k, v
    assert len(picked) == (8 if name != "hires7b" else 4)
    for i in range(n_steps):
        t = n0 + 1 + i
        if form == "one_launch":
            out = bf16_to_f64(cache.append_decode_layers(0, step_in[1][i], step_in[2][i], step_in[0][i]))
        else:
            out = bf16_to_f64(torch.stack([cache.append_decode(l, step_in[1][i, l], step_in[2][i, l], step_in[0][i, l])
                                           for l in range(NL)]))
        for (layer, s, h), (qu, ku, vu, sem, gidx, gcnt) in picked.items():
            want = oracle.decode_batch(qu[None, None, t - 1], ku[None, None], vu[None, None], sem, gidx, gcnt, L, t, W, M, R)
            err = np.abs(out[layer, s, h] - want[0, 0])
            assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (layer, s, h, t, err.max())
    assert cache.device_status() == 0
    cache.close()


@pytest.mark.parametrize("kv_format", [0, 1])
def test_per_layer_launch_is_reproducible_at_full_width(kv_format):
    """The per-layer launch cuts heads across warps and thread blocks and merges the pieces in a fixed order, whoever
    arrives last: two caches fed the same inputs must agree bit for bit at the width the benchmark runs (64
    sequences: every share boundary cuts a head, two heads per thread block are merged through global memory), step
    after step, and so must the slabs they leave behind (seen through one more step)."""
    cfg = wl.CONFIGS["janus7b"]
    dev = torch.device("cuda:0")
    L, n0, S, nl = cfg.prompt_len, cfg.n0, cfg.n_seqs, 2
    data = [wl.gen_layer(cfg, l, range(S), device=dev) for l in range(nl)]
    labels = np.stack([wl.sink_mask(cfg, l) for l in range(nl)])
    caches = []
    for _ in range(2):
        c = B.SsdCache(B.config_from_workload(cfg, n_layers=nl), device=dev)
        if kv_format:
            c.set_kv_format(kv_format)
        c.set_head_labels(labels)
        for l, (q, k, v, _) in enumerate(data):
            c.compress(l, q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0)
        caches.append(c)
    for t in range(n0 + 1, n0 + 13):
        for l, (q, k, v, _) in enumerate(data):
            args = (k[:, :, L + t - 1].contiguous(), v[:, :, L + t - 1].contiguous(), q[:, :, t - 1].contiguous())
            a = caches[0].append_decode(l, *args)
            # other work in between, so that the two launches do not meet the GPU in the same state
            caches[1].decode_attn(1 - l, args[2])
            b = caches[1].append_decode(l, *args)
            assert torch.equal(a, b), (t, l)
            assert torch.isfinite(a.float()).all()
    for c in caches:
        assert c.device_status() == 0
        c.close()
