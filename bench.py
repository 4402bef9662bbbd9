#!/usr/bin/env python
"""Benchmark of the SSD decode hot path (append + decode attention over every layer, per step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload janus7b] [--impl reference]

Prints ONE JSON line.  A "step" is one decoded image token for every sequence: for each layer,
append the new K/V and attend.  `value` is decoded image tokens per second (one per CFG pair per
step) over the whole job with inputs resident in HBM and the step issued the way a model issues it:
one ssd_append_decode call (one kernel launch) per layer.  `one_launch` is the same step as a single
launch over all layers (ssd_append_decode_layers: an upper bound that needs every layer's inputs up
front); `e2e` is the step through ssd_step_host_layers with pinned HOST buffers (copies inside the
timed region).  Under torchrun each rank owns its own block of sequences (weak scaling, no data-path
collective); time is the max over ranks.  `--impl reference` times the fp64 CPU oracle as it stands on
a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2510_18716_b200 import workloads as wl  # noqa: E402

# DRAM bytes (read + written) from the ncu captures summarised under profiles/: one ssd_decode_kernel
# launch on a janus7b layer, and one ssd_decode_layers_kernel launch per layer it covers (captured on
# 4 layers; every layer moves the same bytes, so a launch over n layers moves n times that).
# Reported only while the kernels' sources still hash to what was captured; otherwise `traffic` is
# null until the counters are taken again.
DECODE_TRAFFIC = {"workload": "janus7b", "per_layer": 163.34e6, "per_layer_of_step": 160.74e6,
                  "sha256": "9ddc1973d04d2b83e3ff1282d7c7629396a25d96fd39e6cf8b66f0d593d4cfaa"}


def decode_traffic(cfg):
    import hashlib
    h = hashlib.sha256()
    for f in ("ssd_decode.cu", "ssd_decode_layer.cuh", "ssd_decode_step.cuh", "ssd_device.cuh", "ssd_plan.h", "ssd_internal.cuh"):
        with open(os.path.join(ROOT, "paper_2510_18716_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    if h.hexdigest() != DECODE_TRAFFIC["sha256"] or not cfg.name.startswith(DECODE_TRAFFIC["workload"]):
        return None
    return DECODE_TRAFFIC


METRIC = "decoded image tokens/sec (attention+cache ops)"
NOSCORE_REPS = 5          # calls of ssd_compress without scoring that are timed together (one layer)
UNIT = "image tokens/s"


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            with open(p) as f:
                d = json.load(f)
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                smax.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def config_dict(cfg, world, kv_bytes_per_seq=None):
    """The `config` object of the JSON line, the same for both arms."""
    slots = cfg.n_sink_heads * (cfg.prompt_len + cfg.sink_budget + cfg.sink_recent) + \
        (cfg.n_heads - cfg.n_sink_heads) * (cfg.prompt_len + cfg.window)
    layer_mb = cfg.n_seqs * slots * 512 / 1e6
    return {"workload": cfg.name, "n_layers": cfg.n_layers, "n_seqs_per_gpu": cfg.n_seqs, "n_heads": cfg.n_heads,
            "prompt_len": cfg.prompt_len, "image_tokens": cfg.n_img, "compressed_at": cfg.n0, "window": cfg.window,
            "sink_budget": cfg.sink_budget, "sink_recent": cfg.sink_recent, "sink_heads_per_layer": cfg.n_sink_heads,
            "kv_dtype": "bf16", "parallelism": f"sequence-sharded x{world}",
            "l2": f"no flush: a layer's slab ({layer_mb:.0f} MB) is touched once per step and a step touches "
                  f"{layer_mb * cfg.n_layers / 1e3:.2f} GB, against 126 MB of L2",
            "kv_bytes_per_seq": cfg.n_layers * slots * 512 if kv_bytes_per_seq is None else kv_bytes_per_seq}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


# ----------------------------------------------------------------------------- reference arm
def oracle_sample(cfg: wl.Workload, layers, n_steps, device):
    """Inputs (host, bf16 bits) and the oracle's own selection for a bounded sample of the workload."""
    import oracle
    L, n0 = cfg.prompt_len, cfg.n0
    seqs = list(range(cfg.n_seqs))
    data = []
    for layer in layers:
        q, k, v, _ = wl.gen_layer(cfg, layer, seqs, device=device)
        sem = wl.sink_mask(cfg, layer)[None, :].repeat(len(seqs), 0)
        qu, ku, vu = wl.to_u16(q), wl.to_u16(k), wl.to_u16(v)
        _, idx, cnt = oracle.select_batch(qu[:, :, :n0], ku[:, :, : L + n0], sem, L, n0, cfg.sink_budget,
                                          cfg.sink_recent)
        data.append((qu, ku, vu, sem, idx, cnt))
    return data


def oracle_time_steps(cfg: wl.Workload, data, t_first, n_steps):
    """Seconds the oracle needs for n_steps decode steps over the sampled layers."""
    import oracle
    L = cfg.prompt_len
    t0 = time.perf_counter()
    for i in range(n_steps):
        t = t_first + i
        for (qu, ku, vu, sem, idx, cnt) in data:
            oracle.decode_batch(np.ascontiguousarray(qu[:, :, t - 1]), ku, vu, sem, idx, cnt, L, t, cfg.window,
                                cfg.sink_budget, cfg.sink_recent)
    return time.perf_counter() - t0


def run_reference(args, cfg):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    import oracle
    layers = sorted({0, cfg.n_layers - 1})
    data = oracle_sample(cfg, layers, 0, "cuda" if torch.cuda.is_available() else "cpu")
    scale = cfg.n_layers / len(layers)
    for _ in range(args.warmup):
        oracle_time_steps(cfg, data, cfg.n0 + 1, 1)
    secs = oracle_time_steps(cfg, data, cfg.n0 + 1, args.steps)
    ms_per_step = secs / args.steps * scale * 1e3
    value = cfg.images_per_step / (ms_per_step * 1e-3)
    sample = (f"decode attention of layers {layers} (of {cfg.n_layers}) x all {cfg.n_seqs} sequences x "
              f"{cfg.n_heads} heads per step, time scaled by {scale:g} (extrapolated)")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(cfg, args.gpus),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- our arm
def build_cache(cfg: wl.Workload, device, seq_lo, rank, world, full_cache=False, t_steps=0, row_buffer=False,
                classify=True, kv_format=0):
    """Create, classify, load and compress every layer; returns the cache and per-layer step inputs."""
    from paper_2510_18716_b200 import binding as B
    from paper_2510_18716_b200 import dist as D
    L, N, n0, H, S = cfg.prompt_len, cfg.n_img, cfg.n0, cfg.n_heads, cfg.n_seqs
    setup = {}                      # one-time costs: head classification, per-layer compression
    if full_cache:
        ccfg = B.make_config(cfg.n_layers, S, H, L, N, N, 0, 1, cfg.cls_window, cfg.tau)
        cache = B.SsdCache(ccfg, n_sink_heads_total=0, device=device)
        cache.set_head_labels(np.zeros(cfg.n_layers * H, np.uint8))
    else:
        ccfg = B.config_from_workload(cfg)
        cache = B.SsdCache(ccfg, n_sink_heads_total=cfg.n_layers * cfg.n_sink_heads, device=device)
        if row_buffer:
            cache.set_row_buffer(True)
        if kv_format:
            cache.set_kv_format(kv_format)
        if not classify:
            cache.set_head_labels(np.stack([wl.sink_mask(cfg, l) for l in range(cfg.n_layers)]))
        mine = D.shard_calibration(cfg.n_cal, rank, world) if classify else None
        qs, ks = [], []
        for layer in range(cfg.n_layers):
            if mine:
                q, k, _, _ = wl.gen_layer(cfg, layer, [wl.CAL_SEQ_BASE + p for p in mine], device=device)
                qs.append(q)
                ks.append(k)
        qc = torch.stack(qs) if mine else None
        kc = torch.stack(ks) if mine else None
        if classify:
            torch.cuda.synchronize()
            t_c = time.perf_counter()
            labels = D.classify_sharded(cache, qc, kc, cfg.n_cal, N, cfg.tau)     # synchronises: returns host results
            setup["classify_ms"] = (time.perf_counter() - t_c) * 1e3
            want = np.stack([wl.sink_mask(cfg, l) for l in range(cfg.n_layers)])
            if not np.array_equal(labels, want):
                raise RuntimeError("classifier did not recover the generator's head split")
        del qc, kc, qs, ks
    # step inputs of all layers in three tensors [T, n_layers, S, H, D]: entry [i] is what the one-launch
    # step takes, entry [i, layer] (contiguous) what the per-layer calls take
    T = min(t_steps, N - n0)
    step_all = tuple(torch.empty((T, cfg.n_layers, S, H, 128), dtype=torch.bfloat16, device=device) for _ in range(3))
    steps_in = []
    comp_events = []
    seqs = list(range(seq_lo, seq_lo + S))
    for layer in range(cfg.n_layers):
        q, k, v, _ = wl.gen_layer(cfg, layer, seqs, device=device)
        if full_cache:
            cache.compress(layer, None, k[:, :, :L].contiguous(), v[:, :, :L].contiguous(), 0, 0)
            # bulk-append the first n0 tokens so both caches sit at the same image step
            for j in range(n0):
                cache.append(layer, k[:, :, L + j].contiguous(), v[:, :, L + j].contiguous())
        else:
            args_c = (q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous())
            if layer == 0:
                # the same call without observed queries does everything but the scoring (scores all zero):
                # the difference to the full call is the scoring kernel's time
                ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
                for _ in range(2):
                    cache.compress(layer, None, args_c[1], args_c[2], n0, 0)
                ev[0].record()
                for _ in range(NOSCORE_REPS):
                    cache.compress(layer, None, args_c[1], args_c[2], n0, 0)
                ev[1].record()
                noscore_events = ev
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            cache.compress(layer, *args_c, n0)          # score (tcgen05), select, gather
            e1.record()
            comp_events.append((e0, e1))
        step_all[0][:, layer] = q[:, :, n0:n0 + T].permute(2, 0, 1, 3)
        step_all[1][:, layer] = k[:, :, L + n0:L + n0 + T].permute(2, 0, 1, 3)
        step_all[2][:, layer] = v[:, :, L + n0:L + n0 + T].permute(2, 0, 1, 3)
        steps_in.append(tuple(x[:, layer] for x in step_all))
        del q, k, v
    torch.cuda.synchronize()
    if comp_events:
        ms_c = [a.elapsed_time(b) for a, b in comp_events]
        setup["compress_ms_per_layer_median"] = float(np.median(ms_c))
        setup["compress_ms_all_layers"] = float(np.sum(ms_c))
        setup.update(one_time_rooflines(cfg, S, float(np.median(ms_c)), noscore_events[0].elapsed_time(noscore_events[1]) / NOSCORE_REPS))
    cache.step_all = step_all
    cache.setup_times = setup
    return cache, steps_in


def one_time_rooflines(cfg, S, compress_ms, noscore_ms):
    """Rooflines of the one-time kernels of ssd_compress on one layer: the scoring contraction (tcgen05;
    flops after causal skipping, i.e. of the 128 x 128 tiles it computes, in both sweeps) against the bf16
    peak, and select + gather as a copy against the HBM peak."""
    L, n0, H = cfg.prompt_len, cfg.n0, cfg.n_heads
    tiles = 0
    nb = -(-n0 // 128)
    for bi in range(nb):                       # blocks of 128 observed queries, aligned to the end (the first is the short one)
        ctx = L + n0 - (nb - 1 - bi) * 128
        tiles += -(-ctx // 128) + -(-(ctx - (L // 128) * 128) // 128)
    pairs = S * cfg.n_sink_heads
    flops = tiles * 2 * 128 ** 3 * pairs
    exps = tiles * 128 * 128 * pairs
    score_ms = max(compress_ms - noscore_ms, 1e-6)
    tf_peak = 1620.8
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            tf_peak = float(json.load(f)["bf16_tflops"])
    except Exception:
        pass
    sms, mhz = 148, 1965.0
    exp_peak = 16 * sms * mhz * 1e6            # 16 special-function results per clock and SM
    n_sp = H - cfg.n_sink_heads
    slots = n_sp * (L + min(cfg.window, n0)) + cfg.n_sink_heads * (L + min(cfg.sink_budget, max(n0 - cfg.sink_recent, 0)) + min(cfg.sink_recent, n0))
    gbytes = S * slots * 512 * 2
    hbm, kind = measured_peaks()
    return {"score": {"kernel": "ssd_score_kernel (tcgen05)", "ms_per_layer": score_ms, "tiles_per_pair": tiles,
                      "roofline": {"bound": "tensor", "achieved": flops / (score_ms * 1e-3) / 1e12, "peak": tf_peak,
                                   "unit": "TFLOP/s", "frac": flops / (score_ms * 1e-3) / 1e12 / tf_peak,
                                   "peak_kind": f"of {kind} (burst)", "traffic": None,
                                   "co_limit": {"what": "exponentials (special-function unit), one per logit and sweep",
                                                "achieved_per_s": exps / (score_ms * 1e-3), "peak_per_s": exp_peak,
                                                "frac": exps / (score_ms * 1e-3) / exp_peak}}},
            "select_gather": {"kernels": "memset + ssd_select_kernel + ssd_gather_kernel", "ms_per_layer": noscore_ms,
                              "roofline": {"bound": "hbm", "achieved": gbytes / (noscore_ms * 1e-3) / 1e9, "peak": hbm,
                                           "unit": "GB/s", "frac": gbytes / (noscore_ms * 1e-3) / 1e9 / hbm,
                                           "peak_kind": f"of {kind}", "bytes_per_layer": gbytes, "traffic": None}}}


class Stepper:
    """Replays decode steps n0+1.. over all layers, wrapping back to n0 when the grid is full."""

    def __init__(self, cfg, cache, steps_in, out):
        self.cfg, self.cache, self.steps_in, self.out = cfg, cache, steps_in, out
        self.i = 0
        self.T = steps_in[0][0].shape[0]
        self.out_all = torch.empty((cfg.n_layers,) + tuple(out.shape), dtype=out.dtype, device=out.device)
        # device addresses of every step's inputs: the per-layer loop below makes 30 calls per 0.85 ms,
        # so the host must not spend its time slicing tensors and re-checking shapes at every call
        qa, ka, va = cache.step_all
        per = qa[0, 0].numel() * qa.element_size()
        base = (qa.data_ptr(), ka.data_ptr(), va.data_ptr())
        self.addr = lambda j, i, layer: base[j] + (i * cfg.n_layers + layer) * per
        self.call = cache.lib.ssd_append_decode
        self.h = cache._h
        self.args = [[(layer, self.addr(1, i, layer), self.addr(2, i, layer), self.addr(0, i, layer))
                      for layer in range(cfg.n_layers)] for i in range(self.T)]

    def step(self, fused=True, one_launch=False):
        """One decoded token per sequence: for every layer append the new K/V and attend
        (ssd_append_decode: one launch per layer; fused=False: ssd_append then ssd_decode_attn;
        one_launch: ssd_append_decode_layers, the whole step in one launch)."""
        if self.i == self.T:
            for layer in range(self.cfg.n_layers):
                self.cache.rewind(layer, self.cfg.n0)
            self.i = 0
        i = self.i
        if one_launch:
            q, k, v = self.cache.step_all
            for l0 in range(0, self.cfg.n_layers, 64):         # the call takes up to 64 layers
                l1 = min(l0 + 64, self.cfg.n_layers)
                self.cache.append_decode_layers(l0, k[i, l0:l1], v[i, l0:l1], q[i, l0:l1], self.out_all[l0:l1])
            self.i += 1
            return
        if fused:
            stream, outp, call, h = torch.cuda.current_stream().cuda_stream, self.out.data_ptr(), self.call, self.h
            for layer, ka, va, qa in self.args[i]:
                rc = call(h, layer, ka, va, qa, outp, stream)
                if rc != 0:
                    raise RuntimeError(f"ssd_append_decode: status {rc}")
            self.i += 1
            return
        for layer in range(self.cfg.n_layers):
            q, k, v = self.steps_in[layer]
            self.cache.append(layer, k[i], v[i])
            self.cache.decode_attn(layer, q[i], self.out)
        self.i += 1


def timed(fn, n, barrier):
    barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n):
        fn()
    e1.record()
    torch.cuda.synchronize()
    barrier()
    return e0.elapsed_time(e1)


def run_ours(args, cfg):
    from paper_2510_18716_b200 import binding as B
    import torch.distributed as dist
    rank, world, local = dist_env()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    def barrier():
        if world > 1:
            dist.barrier()

    def max_over_ranks(ms):
        if world == 1:
            return ms
        t = torch.tensor([ms], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    B.load()
    K, W = args.steps, args.warmup
    S, H, N, n0 = cfg.n_seqs, cfg.n_heads, cfg.n_img, cfg.n0
    cache, steps_in = build_cache(cfg, device, rank * S, rank, world, t_steps=K + W + 2 * min(K, 50) + 1)
    out = torch.empty((S, H, 128), dtype=torch.bfloat16, device=device)
    stepper = Stepper(cfg, cache, steps_in, out)

    # ---- device-resident timing (the headline `value`): the step as a model issues it, one
    # ssd_append_decode call (one launch of ssd_decode_kernel) per layer; consecutive launches overlap by
    # programmatic dependent launch
    for _ in range(W):
        stepper.step()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    l0 = B.kernel_launch_count()
    ms = timed(stepper.step, K, barrier)
    launches = B.kernel_launch_count() - l0
    ms = max_over_ranks(ms)
    ms_per_step = ms / K
    value = cfg.images_per_step * world / (ms_per_step * 1e-3)
    # stability: five more passes of the same region, shorter
    Ks = min(K, 50)
    repeats = [max_over_ranks(timed(stepper.step, Ks, barrier)) / Ks for _ in range(5)]
    # what the host needs to issue a launch (Python call + library + driver), measured on a queue that is
    # never full: if this approaches the launch duration, the number above is the host's, not the GPU's
    torch.cuda.synchronize()
    Kh = max(1, min(K, 600 // cfg.n_layers))
    t_h0 = time.perf_counter()
    for _ in range(Kh):
        stepper.step()
    host_us = (time.perf_counter() - t_h0) / (Kh * cfg.n_layers) * 1e6
    torch.cuda.synchronize()
    # the same steps again with a CUDA event on either side of every decode launch (the events stand
    # between the kernels, so these launches do not overlap with their neighbours)
    Kr = min(K, 50)
    cache.profile_enable(Kr * cfg.n_layers)
    ms_r = timed(stepper.step, Kr, barrier)
    dec_ms = cache.profile_collect()
    cache.profile_enable(0)
    # as two launches per layer (ssd_append, ssd_decode_attn), for comparison
    Kt = min(K, 50)
    two_step = lambda: stepper.step(fused=False)
    two_step()
    ms_two = max_over_ranks(timed(two_step, Kt, barrier)) / Kt

    # ---- the whole step as ONE launch (ssd_append_decode_layers: every layer's append + attention, heads
    # handed out from a counter): an upper bound, since it needs all layers' inputs before the first layer runs
    one_step = lambda: stepper.step(one_launch=True)
    for _ in range(3):
        one_step()
    ms_one = max_over_ranks(timed(one_step, K, barrier)) / K
    clocks = sampler.stop()

    # ---- roofline of the dominant kernel: algorithmic bytes per launch / launch duration (CUDA events)
    slots_layer = int(sum(int(cache.get_lengths(l).sum()) for l in range(cfg.n_layers))) / cfg.n_layers
    # K+V rows of the valid slots, q in and out, and the fused append's 512 B per head read and written
    bytes_launch = S * (slots_layer * 512 + H * 2 * 256 + H * 2 * 512)
    bytes_step = bytes_launch * cfg.n_layers
    peak, peak_kind = measured_peaks()
    n_calls = (cfg.n_layers + 63) // 64
    traffic = decode_traffic(cfg)
    dec_mean_ms = float(np.mean(dec_ms)) if len(dec_ms) else float("nan")
    # The timed region holds nothing but launches of ssd_decode_kernel (n_layers per step), so its launch
    # duration is the region time per launch; launches overlap by design, so timed one at a time (an event
    # between launches forbids the overlap) a launch takes longer ("isolated").
    launch_ms = ms_per_step / cfg.n_layers
    achieved = bytes_launch / (launch_ms * 1e-3) / 1e9
    iso = bytes_launch / (dec_mean_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "ssd_decode_kernel (one launch per layer, fused append)", "achieved": achieved,
                "peak": peak, "unit": "GB/s", "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                "traffic": traffic["per_layer"] if traffic else None,
                "bytes_per_launch": bytes_launch, "launch_ms_mean": launch_ms, "launches_in_region": K * cfg.n_layers,
                "isolated": {"launch_ms_mean": dec_mean_ms, "achieved": iso, "frac": iso / peak,
                             "launch_ms_median": float(np.median(dec_ms)) if len(dec_ms) else None,
                             "launches_timed": int(len(dec_ms)),
                             "ms_per_step_while_timing_launches": ms_r / Kr},
                "frac_of_8TBs_nominal": achieved / 8000.0}
    ach_one = bytes_step / (ms_one * 1e-3) / 1e9
    one_launch = {"value": cfg.images_per_step * world / (ms_one * 1e-3), "unit": UNIT, "ms_per_step": ms_one,
                  "launches_per_step": n_calls,
                  "roofline": {"bound": "hbm", "kernel": "ssd_decode_layers_kernel (whole step, fused append)",
                               "achieved": ach_one, "peak": peak, "unit": "GB/s", "frac": ach_one / peak,
                               "peak_kind": f"of {peak_kind}",
                               "traffic": traffic["per_layer_of_step"] * cfg.n_layers / n_calls if traffic else None,
                               "bytes_per_launch": bytes_step / n_calls, "launch_ms_mean": ms_one / n_calls,
                               "frac_of_8TBs_nominal": ach_one / 8000.0}}
    host = {"enqueue_us_per_launch": host_us, "launches_per_step": cfg.n_layers, "steps": Kh,
            "share_of_launch_time": host_us / (launch_ms * 1e3),
            "ms_per_step_two_launches_per_layer": ms_two}

    # ---- end to end: the same step through ssd_step_host_layers with pinned host buffers: one call
    # per step takes every layer's q, k_new, v_new from the host and returns every layer's output
    pool = 4
    stack = lambda j, i: torch.stack([steps_in[l][j][i] for l in range(cfg.n_layers)]).cpu().pin_memory()
    hq = [stack(0, i) for i in range(pool)]
    hk = [stack(1, i) for i in range(pool)]
    hv = [stack(2, i) for i in range(pool)]
    ho = torch.empty((cfg.n_layers, S, H, 128), dtype=torch.bfloat16).pin_memory()
    state = {"i": 0}

    def host_step():
        if cache.tokens(0) >= N:
            for layer in range(cfg.n_layers):
                cache.rewind(layer, n0)
        i = state["i"] % pool
        cache.step_host_layers(0, hq[i], hk[i], hv[i], ho)
        state["i"] += 1

    Ke = max(4, min(K, 16))
    for _ in range(3):
        host_step()
    ms_e = max_over_ranks(timed(host_step, Ke, barrier))
    e2e_val = cfg.images_per_step * world / (ms_e / Ke * 1e-3)
    tensor_bytes = S * H * 128 * 2
    e2e = {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": 3 * tensor_bytes * cfg.n_layers,
           "d2h_bytes_per_step": tensor_bytes * cfg.n_layers, "steps": Ke, "ms_per_step": ms_e / Ke,
           "h2d_gbs": 3 * tensor_bytes * cfg.n_layers / (ms_e / Ke * 1e-3) / 1e9,
           "d2h_gbs": tensor_bytes * cfg.n_layers / (ms_e / Ke * 1e-3) / 1e9}

    kv_bytes_per_seq = cache.kv_bytes_per_seq()
    setup_times = cache.setup_times
    cache.close()
    del cache, steps_in, stepper
    torch.cuda.empty_cache()

    # ---- same library, uncompressed full cache (every head keeps everything)
    full = None
    if not args.no_full_cache:
        Kf = max(2, min(K, 8))
        fcache, fsteps = build_cache(cfg, device, rank * S, rank, world, full_cache=True, t_steps=2 * Kf + 5)
        fst = Stepper(cfg, fcache, fsteps, out)
        for _ in range(3):
            fst.step()
        ms_fl = max_over_ranks(timed(fst.step, Kf, barrier))                       # one launch per layer
        f_one = lambda: fst.step(one_launch=True)
        f_one()
        ms_f = max_over_ranks(timed(f_one, Kf, barrier))                           # one launch per step
        t_mid = n0 + 3 + Kf + 1 + (Kf + 1) / 2
        fbytes = cfg.n_layers * S * H * ((cfg.prompt_len + t_mid) * 512 + 512)
        full = {"value": cfg.images_per_step * world / (ms_fl / Kf * 1e-3), "unit": UNIT, "ms_per_step": ms_fl / Kf,
                "steps": Kf, "image_step": t_mid - Kf - 1, "gbs": (fbytes - cfg.n_layers * S * H * (Kf + 1) * 512) / (ms_fl / Kf * 1e-3) / 1e9,
                "ms_per_step_one_launch": ms_f / Kf, "gbs_one_launch": fbytes / (ms_f / Kf * 1e-3) / 1e9,
                "kv_bytes_per_seq": fcache.kv_bytes_per_seq()}
        fcache.close()
        del fcache, fsteps, fst
        torch.cuda.empty_cache()

    # ---- Algorithm 2 (row buffer): append + decode with score accumulation, re-selection every R steps
    rowbuf = None
    if not args.no_row_buffer and cfg.n_sink_heads > 0:
        R = cfg.sink_recent
        Kb = max(R, min(2 * R, (N - n0) // 2 - R) // R * R)   # both forms, each with a warm-up cycle, fit in the image
        rcache, rsteps = build_cache(cfg, device, rank * S, rank, world, t_steps=2 * (Kb + R), row_buffer=True)
        rst = Stepper(cfg, rcache, rsteps, out)          # per-layer calls with precomputed addresses
        rout = torch.empty((cfg.n_layers, S, H, 128), dtype=torch.bfloat16, device=device)

        def reselect(c):
            for l0 in range(0, cfg.n_layers, 64):
                c.recompress_layers(l0, min(64, cfg.n_layers - l0))

        def rb_step(one_launch):
            # ssd_append_decode per layer (one launch each: the kernel also keeps the scores up to date), or the
            # whole step in one launch; every R steps ssd_recompress_layers re-selects all layers in one launch
            rst.step(one_launch=one_launch)
            if rst.i % R == 0:
                reselect(rcache)

        ms_rb = {}
        for form in (False, True):    # per-layer launches, then the one-launch step
            for _ in range(R):        # one whole cycle as warm-up, so the timed region starts on an empty buffer
                rb_step(form)
            ms_rb[form] = max_over_ranks(timed(lambda: rb_step(form), Kb, barrier))
        ms_b = ms_rb[False]
        rowbuf = {"value": cfg.images_per_step * world / (ms_b / Kb * 1e-3), "unit": UNIT, "ms_per_step": ms_b / Kb,
                  "steps": Kb, "reselect_every": R, "ms_per_step_one_launch": ms_rb[True] / Kb,
                  "device_status": rcache.device_status()}
        rcache.close()
        del rcache, rsteps, rst
        torch.cuda.empty_cache()
        # Algorithm 1 taken literally: a re-selection after every step = a row buffer of one token with the
        # same number of slots per head (M + R - 1 static, 1 buffered)
        import dataclasses
        ecfg = dataclasses.replace(cfg, sink_budget=cfg.sink_budget + R - 1, sink_recent=1, name=cfg.name + "_evict_every_step")
        Kv = min(K, 48)
        ecache, esteps = build_cache(ecfg, device, rank * S, rank, world, t_steps=2 * Kv + 8, row_buffer=True, classify=False)
        est = Stepper(ecfg, ecache, esteps, out)

        def ev_step(one_launch):
            # one launch per layer, then one re-selection launch for all layers; or everything in one launch
            # (with a buffer of one token the one-launch step re-selects as well)
            est.step(one_launch=one_launch)
            if not one_launch:
                reselect(ecache)

        ms_ev = {}
        for form in (False, True):
            for _ in range(3):
                ev_step(form)
            ms_ev[form] = max_over_ranks(timed(lambda: ev_step(form), Kv, barrier))
        rowbuf["evict_every_step"] = {"value": cfg.images_per_step * world / (ms_ev[False] / Kv * 1e-3), "unit": UNIT,
                                      "ms_per_step": ms_ev[False] / Kv, "ms_per_step_one_launch": ms_ev[True] / Kv,
                                      "steps": Kv, "sink_budget": ecfg.sink_budget,
                                      "sink_recent": 1, "device_status": ecache.device_status()}
        ecache.close()
        del ecache, esteps, est
        torch.cuda.empty_cache()

    # ---- 8-bit K/V (an extension the paper only cites, Sec. 2): a leg of its own, never the headline.  The same
    # steps over a cache of 272-byte slots, as one launch per step and as one launch per layer (the equal-shares
    # kernel of the bf16 path with this format's arithmetic)
    q8 = None
    if not args.no_q8:
        Kq = min(K, 40)
        qcache, qsteps = build_cache(cfg, device, rank * S, rank, world, t_steps=2 * Kq + 8, classify=False, kv_format=1)
        qst = Stepper(cfg, qcache, qsteps, out)
        ms_q = {}
        for form in (False, True):
            for _ in range(3):
                qst.step(one_launch=form)
            ms_q[form] = max_over_ranks(timed(lambda: qst.step(one_launch=form), Kq, barrier)) / Kq
        slots_q = int(sum(int(qcache.get_lengths(l).sum()) for l in range(cfg.n_layers))) / cfg.n_layers
        # codes and scales of the valid slots, q in and out, the new token's bf16 rows read and its slot written
        qbytes = S * (slots_q * 272 + H * 2 * 256 + H * (512 + 272)) * cfg.n_layers
        def q8_roofline(kernel, ms, launches):
            return {"bound": "hbm", "kernel": kernel, "achieved": qbytes / (ms * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                    "frac": qbytes / (ms * 1e-3) / 1e9 / peak, "peak_kind": f"of {peak_kind}",
                    "bytes_per_launch": qbytes / launches, "traffic": None}

        # like the headline: `value` is the form a model can call (one launch per layer), the whole step in one
        # launch is reported beside it
        q8 = {"kv_dtype": "e4m3 codes + float32 scale per row (272 B per slot)", "unit": UNIT,
              "form": "one launch per layer (ssd_append_decode); one_launch = the whole step in one launch",
              "value": cfg.images_per_step * world / (ms_q[False] * 1e-3), "ms_per_step": ms_q[False],
              "steps": Kq, "kv_bytes_per_seq": qcache.kv_bytes_per_seq(),
              "roofline": dict(q8_roofline("ssd_decode_kernel<Q8Slots> (one launch per layer, fused append)", ms_q[False], cfg.n_layers),
                               note="this instance is limited by instruction issue (twice the bf16 kernel's instructions per byte), "
                                    "not by HBM; the fraction is still taken against the HBM peak"),
              "one_launch": {"value": cfg.images_per_step * world / (ms_q[True] * 1e-3), "unit": UNIT, "ms_per_step": ms_q[True],
                             "roofline": q8_roofline("ssd_decode_layers_kernel<Q8Slots<12, 24>> (whole step, fused append)",
                                                     ms_q[True], 1)},
              "device_status": qcache.device_status()}
        qcache.close()
        del qcache, qsteps, qst
        torch.cuda.empty_cache()

    # ---- analysis utility (Sec. 3.2, MSE_token): per-token divergence of two uncompressed caches of one layer
    analysis = None
    if rank == 0 and world == 1:
        g = torch.Generator(device=device).manual_seed(1)
        shape = (S, H, cfg.prompt_len + N, 128)
        t4 = [torch.randn(shape, generator=g, device=device).to(torch.bfloat16) for _ in range(4)]
        mo = torch.empty(shape[:-1], dtype=torch.float32, device=device)
        mse = lambda: B.kv_token_mse(*t4, out=mo)
        for _ in range(3):
            mse()
        ms_m = timed(mse, 20, barrier) / 20
        mbytes = mo.numel() * (4 * 256 + 4)
        analysis = {"kernel": "ssd_kv_token_mse_kernel", "rows": mo.numel(), "ms": ms_m,
                    "roofline": {"bound": "hbm", "achieved": mbytes / (ms_m * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                                 "frac": mbytes / (ms_m * 1e-3) / 1e9 / peak, "peak_kind": f"of {peak_kind}",
                                 "bytes_per_launch": mbytes, "traffic": None}}
        del t4, mo
        torch.cuda.empty_cache()

    # ---- CPU oracle on the host cores (rank 0, N = 1 only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        layers = sorted({0, cfg.n_layers // 2, cfg.n_layers - 1})
        data = oracle_sample(cfg, layers, 0, device)
        oracle_time_steps(cfg, data, n0 + 1, 1)
        n_pass = min(N - n0, 288)
        secs, n_cpu = 0.0, 0
        while secs < 10.0 and n_cpu < 12 * n_pass:      # about 10-30 s of CPU work: repeat the pass until it is
            secs += oracle_time_steps(cfg, data, n0 + 1, n_pass)
            n_cpu += n_pass
        scale = cfg.n_layers / len(layers)
        cpu_ms = secs / n_cpu * scale * 1e3
        cpu = {"value": cfg.images_per_step / (cpu_ms * 1e-3), "unit": UNIT, "cores": oracle.threads(),
               "kind": "oracle", "ms_per_step": cpu_ms, "seconds_timed": secs,
               "sample": (f"{n_cpu} decode steps ({n_cpu // n_pass} passes over image steps {n0 + 1}..{n0 + n_pass}) over layers {layers} of {cfg.n_layers}, all {S} sequences x {H} "
                          f"heads; time scaled by {scale:g} (extrapolated)")}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": config_dict(cfg, world, kv_bytes_per_seq),
            "sequence_tokens_per_s": value * 2 if S > 1 else value,
            "step_form": "one launch per layer (ssd_append_decode); one_launch = the whole step in one launch",
            "ms_per_step_repeats": repeats,
            "host": host,
            "one_launch": one_launch,
            "one_time": setup_times,
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
            "cpu_baseline": cpu, "full_cache": full, "row_buffer": rowbuf, "kv_8bit": q8, "analysis": analysis,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_sweep(args):
    """Large-batch sweep on the 7B shape (batch x compression ratio x sink-head fraction): one JSON line
    per point, timed on `--layers` layers (default 6; every layer has the same shape, so the step time
    scales with the layer count) with the generator's head split installed directly."""
    import dataclasses
    from paper_2510_18716_b200 import binding as B
    torch.cuda.set_device(0)
    device = torch.device("cuda", 0)
    B.load()
    n_layers = args.layers if args.layers > 0 else 6
    K = min(args.steps, 40)
    points = []
    for batch in (32, 64, 128):
        points.append((batch, 1, 0.0))
        for ratio in (2, 5, 10):
            for frac in (0.25, 0.5, 0.75):
                points.append((batch, ratio, frac))
    for batch, ratio, frac in points:
        cfg = dataclasses.replace(wl.sweep(batch, ratio, frac), n_layers=n_layers)
        full = ratio == 1
        if full:
            cfg = dataclasses.replace(cfg, n0=288)
        S, H = cfg.n_seqs, cfg.n_heads
        cache, steps_in = build_cache(cfg, device, 0, 0, 1, full_cache=full, t_steps=K + 4, classify=False)
        out = torch.empty((S, H, 128), dtype=torch.bfloat16, device=device)
        st = Stepper(cfg, cache, steps_in, out)
        for _ in range(3):
            st.step()
        ms = timed(st.step, K, lambda: None) / K
        one = lambda: st.step(one_launch=True)
        one()
        ms_one = timed(one, K, lambda: None) / K
        slots = sum(int(cache.get_lengths(l).sum()) for l in range(n_layers)) / n_layers
        bytes_layer = S * (slots * 512 + H * 2 * 256 + H * 2 * 512)
        line = {"sweep": cfg.name, "batch": batch, "n_seqs": S, "ratio": ratio, "sink_frac": frac,
                "window": cfg.window, "sink_budget": cfg.sink_budget, "sink_recent": cfg.sink_recent,
                "layers_timed": n_layers, "us_per_layer": ms / n_layers * 1e3,
                "ms_per_step_30_layers": ms / n_layers * 30, "image_tokens_per_s": batch / (ms / n_layers * 30 * 1e-3),
                "gbs": bytes_layer / (ms / n_layers * 1e-3) / 1e9,
                "one_launch": {"us_per_layer": ms_one / n_layers * 1e3, "gbs": bytes_layer / (ms_one / n_layers * 1e-3) / 1e9},
                "kv_bytes_per_seq_30_layers": cache.kv_bytes_per_seq() // n_layers * 30,
                "slots_per_head_mean": slots / H, "status": cache.device_status()}
        print(json.dumps(line), flush=True)
        cache.close()
        del cache, steps_in, st
        torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="janus7b", choices=sorted(wl.CONFIGS))
    ap.add_argument("--layers", type=int, default=0, help="use only the first LAYERS layers (small profiling case)")
    ap.add_argument("--no-full-cache", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-row-buffer", action="store_true")
    ap.add_argument("--no-q8", action="store_true", help="skip the 8-bit K/V leg")
    ap.add_argument("--sweep", action="store_true", help="large-batch sweep on the 7B shape: one JSON line per point")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.sweep:
        run_sweep(args)
        return
    cfg = wl.CONFIGS[args.workload]
    if args.layers > 0:
        import dataclasses
        cfg = dataclasses.replace(cfg, n_layers=min(args.layers, cfg.n_layers), name=f"{cfg.name}[:{args.layers} layers]")
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
