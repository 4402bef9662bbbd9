"""Shared driver for the GPU-vs-oracle parity tests: runs the whole path through the C ABI on
seeded inputs and compares every stage with the fp64 CPU oracle."""
from __future__ import annotations

import dataclasses

import numpy as np
import torch

import oracle
from paper_2510_18716_b200 import binding as B
from paper_2510_18716_b200 import workloads as wl

MAX_ABS = 2e-2      # bf16 outputs vs fp64 oracle
MEAN_ABS = 2e-3
BAND = 1e-5         # relative tie band around the k-th score / around tau


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def check_outputs(got: torch.Tensor, want: np.ndarray, what=""):
    g = bf16_to_f64(got)
    err = np.abs(g - want)
    assert np.isfinite(g).all(), f"{what}: non-finite output"
    assert err.max() <= MAX_ABS, f"{what}: max abs err {err.max():.4g}"
    assert err.mean() <= MEAN_ABS, f"{what}: mean abs err {err.mean():.4g}"
    return err.max(), err.mean()


def check_index_sets(gpu_idx: np.ndarray, score: np.ndarray, ora_idx: np.ndarray, ora_cnt: np.ndarray,
                     sem: np.ndarray, n_cand: int, M: int):
    """Bit-exact index sets, except inside the 1e-5 relative band around the k-th score.

    gpu_idx [S,H,M] image indices (-1 padded, ascending); returns the number of pairs whose set
    differs from the oracle's (all of them legitimately, inside the band)."""
    S, H = sem.shape
    n_diff = 0
    for s in range(S):
        for h in range(H):
            g = gpu_idx[s, h]
            if not sem[s, h]:
                continue
            k = int(ora_cnt[s, h])
            assert k == min(M, n_cand)
            gs = g[:k]
            assert (g[k:] == -1).all(), "padding after the selected indices"
            assert (gs >= 0).all() and (gs < n_cand).all() and (np.diff(gs) > 0).all(), "sorted, unique, in range"
            o = ora_idx[s, h, :k]
            if np.array_equal(gs, o):
                continue
            n_diff += 1
            sc = score[s, h, :n_cand]
            kth = np.sort(sc)[::-1][k - 1]
            sure_in = set(np.nonzero(sc > kth * (1 + BAND))[0].tolist())
            band = set(np.nonzero(np.abs(sc - kth) <= BAND * abs(kth))[0].tolist())
            gset = set(gs.tolist())
            assert sure_in <= gset, f"pair ({s},{h}): a clearly better token was dropped"
            assert gset <= (sure_in | band), f"pair ({s},{h}): a clearly worse token was taken"
    return n_diff


def check_labels(s_gpu: np.ndarray, lab_gpu: np.ndarray, s_ora: np.ndarray, tau: float):
    lab_ora = oracle.labels(s_ora, tau)
    assert np.allclose(s_gpu, s_ora, rtol=2e-4, atol=2e-5), np.abs(s_gpu - s_ora).max()
    near = np.abs(s_ora - tau) <= BAND * abs(tau)
    assert np.array_equal(lab_gpu[~near], lab_ora[~near])
    return lab_ora


@dataclasses.dataclass
class RunResult:
    n_pairs: int = 0
    n_band_pairs: int = 0
    max_err: float = 0.0
    mean_err: float = 0.0
    steps_checked: int = 0


def run_workload(cfg: wl.Workload, layers, seqs, check_steps, classify=True, full_every_step=False,
                 n_obs=None, check_planted=False, device="cuda:0", labels_override=None, step_form="two") -> RunResult:
    """Drive the C-ABI path for `layers` x `seqs` of a workload and check every stage.

    The cache is created with len(layers) layers and len(seqs) sequences; layer i of the cache holds
    generator layer layers[i]."""
    dev = torch.device(device)
    L, N, n0, W, M, R = cfg.prompt_len, cfg.n_img, cfg.n0, cfg.window, cfg.sink_budget, cfg.sink_recent
    H = cfg.n_heads
    S = len(seqs)
    n_obs = n0 if n_obs is None else n_obs
    ccfg = B.config_from_workload(cfg, n_layers=len(layers), n_seqs=S)
    cache = B.SsdCache(ccfg, device=device)
    res = RunResult()

    gen_masks = np.stack([wl.sink_mask(cfg, l) for l in layers])
    if classify:
        qc, kc = wl.gen_calibration(cfg, layers, device=dev)
        s_gpu, lab_gpu = cache.classify_heads(qc, kc)
        s_ora = oracle.sparsity(wl.to_u16(qc), wl.to_u16(kc), L, cfg.cls_window)
        labels = check_labels(s_gpu, lab_gpu, s_ora, cfg.tau)
        assert np.array_equal(labels, gen_masks), "classifier must recover the generator's split"
        assert np.array_equal(cache.get_labels(), lab_gpu)
        del qc, kc
    else:
        labels = gen_masks if labels_override is None else np.asarray(labels_override, np.uint8).reshape(gen_masks.shape)
        cache.set_head_labels(labels)

    errs = []
    for li, layer in enumerate(layers):
        q, k, v, planted = wl.gen_layer(cfg, layer, seqs, device=dev)
        qu, ku, vu = wl.to_u16(q), wl.to_u16(k), wl.to_u16(v)
        sem = labels[li][None, :].repeat(S, 0).astype(np.uint8)
        q_obs = q[:, :, n0 - n_obs:n0].contiguous() if n_obs > 0 else None
        cache.compress(li, q_obs, k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0, n_obs)
        # --- selection parity
        n_cand = max(n0 - R, 0)
        sc, oidx, ocnt = oracle.select_batch(qu[:, :, n0 - n_obs:n0], ku[:, :, : L + n0], sem, L, n0, M, R)
        gi = cache.get_indices(li)
        ms = cache.max_slots()
        assert gi.shape == (S, H, ms)
        gidx = np.full((S, H, M), -1, np.int32)
        for h in range(H):
            if labels[li][h]:
                st = gi[:, h, L:L + M]
                gidx[:, h] = np.where(st >= 0, st - L, -1)
        res.n_band_pairs += check_index_sets(gidx, sc, oidx, ocnt, sem, n_cand, M)
        if check_planted and cfg.n_sink_heads > 0 and n_obs == n0:
            pl = planted.cpu().numpy()
            for s in range(S):
                for h in range(H):
                    if labels[li][h]:
                        assert set(pl[s, h].tolist()) <= set(gidx[s, h].tolist()), "planted sink lost"
        gcnt = (gidx >= 0).sum(-1).astype(np.int32)
        # --- decode steps
        steps = list(range(n0 + 1, N + 1))
        for t in steps:
            kt, vt = k[:, :, L + t - 1].contiguous(), v[:, :, L + t - 1].contiguous()
            if not (full_every_step or t in check_steps):
                cache.append(li, kt, vt)
                continue
            qt = q[:, :, t - 1].contiguous()
            if step_form == "fused":           # ssd_append_decode
                out = cache.append_decode(li, kt, vt, qt)
            elif step_form == "layers":        # ssd_append_decode_layers on this one layer
                out = cache.append_decode_layers(li, kt[None], vt[None], qt[None])[0]
            else:                              # ssd_append, ssd_decode_attn
                cache.append(li, kt, vt)
                out = cache.decode_attn(li, qt)
            # attention over the GPU's own (validated) index set, so band cases compare like with like
            want = oracle.decode_batch(qu[:, :, t - 1], ku, vu, sem, gidx, gcnt, L, t, W, M, R)
            errs.append(check_outputs(out, want, f"layer {layer} step {t}"))
            res.steps_checked += 1
            # retained positions, slot by slot
            gi = cache.get_indices(li)
            ln = cache.get_lengths(li)
            for h in range(H):
                want_pos = oracle.retained_set(bool(labels[li][h]), L, t, W, R, gidx[0, h, : gcnt[0, h]])
                got_pos = np.sort(gi[0, h][gi[0, h] >= 0])
                assert np.array_equal(got_pos, want_pos), (layer, h, t)
                assert ln[h] == len(want_pos) <= cfg.slots(bool(labels[li][h]))
        assert cache.tokens(li) == N
        res.n_pairs += S * H
        del q, k, v
    if errs:
        res.max_err = max(e[0] for e in errs)
        res.mean_err = float(np.mean([e[1] for e in errs]))
    assert cache.device_status() == 0, "a decode warp gave up a bounded wait"
    cache.close()
    return res


def run_sampled(cfg: wl.Workload, layer: int, sample, steps, device="cuda:0"):
    """Full launch size on the GPU (all cfg.n_seqs sequences of one layer, the launch configuration the
    benchmark times); the oracle recomputes only the sampled (sequence, head) pairs one by one: their
    selected index sets (exact outside the tie band) and their outputs at the given image steps."""
    dev = torch.device(device)
    L, N, n0, W, M, R, H, S = (cfg.prompt_len, cfg.n_img, cfg.n0, cfg.window, cfg.sink_budget, cfg.sink_recent,
                               cfg.n_heads, cfg.n_seqs)
    labels = wl.sink_mask(cfg, layer)
    cache = B.SsdCache(B.config_from_workload(cfg, n_layers=1), device=device)
    cache.set_head_labels(labels)
    q, k, v, _ = wl.gen_layer(cfg, layer, list(range(S)), device=dev)
    cache.compress(0, q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0)
    gi = cache.get_indices(0)
    n_cand = max(n0 - R, 0)
    picked = {}
    for (s, h) in sample:
        qu, ku, vu = wl.to_u16(q[s, h]), wl.to_u16(k[s, h]), wl.to_u16(v[s, h])
        sem = np.array([[labels[h]]], np.uint8)
        gidx = np.full((1, 1, M), -1, np.int32)
        if labels[h]:
            st = gi[s, h, L:L + M]
            gidx[0, 0] = np.where(st >= 0, st - L, -1)
            sc, oidx, ocnt = oracle.select_batch(qu[None, None, :n0], ku[None, None, : L + n0], sem, L, n0, M, R)
            check_index_sets(gidx, sc, oidx, ocnt, sem, n_cand, M)
        picked[(s, h)] = (qu, ku, vu, sem, gidx, (gidx >= 0).sum(-1).astype(np.int32))
    steps = sorted(steps)
    for t in range(n0 + 1, steps[-1] + 1):
        kt, vt, qt = (x.contiguous() for x in (k[:, :, L + t - 1], v[:, :, L + t - 1], q[:, :, t - 1]))
        if t not in steps:
            cache.append_decode(0, kt, vt, qt) if t % 2 else cache.append(0, kt, vt)
            continue
        out = bf16_to_f64(cache.append_decode(0, kt, vt, qt))
        for (s, h), (qu, ku, vu, sem, gidx, gcnt) in picked.items():
            want = oracle.decode_batch(qu[None, None, t - 1], ku[None, None], vu[None, None], sem, gidx, gcnt, L, t, W, M, R)
            err = np.abs(out[s, h] - want[0, 0])
            assert err.max() <= MAX_ABS and err.mean() <= MEAN_ABS, (s, h, t, err.max())
    assert cache.device_status() == 0
    cache.close()
