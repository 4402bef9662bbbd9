"""Seeded synthetic workloads shaped like the paper's Janus-Pro runs.

This module only draws inputs (and names the configurations).  It contains none
of the method's arithmetic -- no softmax, score, selection or attention -- and is
the one piece of code that both the CUDA path's callers and the CPU checker's
callers use, so that the two sides see the very same bf16 tensors.

Recipe (per layer, per sequence, per head; Sec. 4.1 and Table 5 give the shapes:
24x24 = 576 image tokens, 24/30 layers, 16/32 heads of dimension 128, sequences
in classifier-free-guidance pairs):

* base       Q, K, V ~ N(0,1) i.i.d. for the L prompt and N image positions.
* grid field image positions get ``g * F[row, col, :]`` added to Q and K (one
             shared field) and an independent field added to V.  F is white noise
             per channel smoothed on the h x w grid with a separable Gaussian of
             ``sigma`` cells whose rows are L2-normalised (unit variance at every
             cell, borders included).  g = G_SPATIAL for spatial-locality heads
             (peak field logit ~ 8, so attention sits on the last 1-2 grid rows)
             and G_SINK for semantic-sink heads (nearly flat).
* sink heads a unit direction mu per (layer, head); image queries get ``C_MU*mu``
             added; N_PLANTED image positions per (sequence, head), drawn without
             replacement from [0, n0 - R), have their key replaced by
             ``PLANT_NORM * |k| * mu`` (norm x6, aligned with the mean query).
* head split ``n_sink_heads`` heads per layer are sink heads, at positions
             permuted by the seed.
* rounding   everything is produced in fp32 and rounded to bf16 once.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional, Tuple

import numpy as np
import torch

G_SPATIAL = 0.84
G_SINK = 0.30
C_MU = 2.0
PLANT_NORM = 6.0
N_PLANTED = 4
CAL_SEQ_BASE = 1_000_000  # calibration sequences use ids disjoint from the batch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int
    n_seqs: int                # sequences; a CFG pair is two of them (Sec. 3.1)
    n_heads: int
    prompt_len: int            # L
    grid: Tuple[int, int]      # (h, w); N = h * w
    window: int                # W
    sink_budget: int           # M
    sink_recent: int           # R
    cls_window: int            # w of the sparsity metric
    n_sink_heads: int          # per layer
    n0: int                    # image step at which the cache is compressed
    n_cal: int                 # P calibration sequences
    sigma: float
    tau: float = 0.45
    head_dim: int = 128
    seed: int = 20251018

    @property
    def images_per_step(self) -> int:
        """Decoded image tokens per step: one per CFG pair (a lone sequence counts as one)."""
        return max(1, self.n_seqs // 2)

    @property
    def n_img(self) -> int:
        return self.grid[0] * self.grid[1]

    @property
    def n_pairs(self) -> int:
        return self.n_layers * self.n_seqs * self.n_heads

    def slots(self, semantic: bool) -> int:
        return self.prompt_len + (self.sink_budget + self.sink_recent if semantic else self.window)

    def kv_bytes_per_step(self) -> int:
        """Algorithmic K+V bytes one decode step reads once every ring is full."""
        per_layer = (self.n_sink_heads * self.slots(True)
                     + (self.n_heads - self.n_sink_heads) * self.slots(False))
        return per_layer * self.n_layers * self.n_seqs * self.head_dim * 2 * 2


CONFIGS: Dict[str, Workload] = {
    "tiny": Workload("tiny", 1, 1, 8, 32, (8, 8), 16, 16, 8, 16, 4, 32, 1, 1.5, tau=0.30),
    "janus1b": Workload("janus1b", 24, 32, 16, 64, (24, 24), 64, 64, 24, 32, 8, 288, 4, 1.5),
    "janus7b": Workload("janus7b", 30, 64, 32, 64, (24, 24), 64, 96, 24, 32, 13, 288, 4, 1.5),
    "hires7b": Workload("hires7b", 30, 16, 32, 128, (64, 64), 256, 256, 64, 256, 13, 3840, 2, 3.0),
}


def sweep(batch: int, ratio: int, sink_frac: float) -> Workload:
    """Large-batch sweep point on the 7B shape (``batch`` prompts = 2*batch sequences).

    ``ratio`` is N / (visual slots per head): W = M + R = ceil(N / ratio) and
    R = min(24, slots // 4).  ratio 1 keeps everything (all heads spatial, W = N).
    """
    N = 576
    slots = math.ceil(N / ratio)
    if ratio == 1:
        return Workload(f"sweep_b{batch}_full", 30, 2 * batch, 32, 64, (24, 24), N, 0, 1, 32, 0, 0,
                        4, 1.5)
    R = min(24, slots // 4)
    return Workload(f"sweep_b{batch}_r{ratio}_s{int(round(sink_frac * 100))}", 30, 2 * batch, 32, 64,
                    (24, 24), slots, slots - R, R, 32, int(round(sink_frac * 32)), 288, 4, 1.5)


# --------------------------------------------------------------------------- seeding
def _mix(*xs: int) -> int:
    """Counter-style integer hash (splitmix64 finaliser) -> 63-bit seed."""
    z = 0x9E3779B97F4A7C15
    for x in xs:
        z = (z ^ (int(x) & 0xFFFFFFFFFFFFFFFF)) & 0xFFFFFFFFFFFFFFFF
        z = (z + 0x9E3779B97F4A7C15) & 0xFFFFFFFFFFFFFFFF
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & 0xFFFFFFFFFFFFFFFF
        z = z ^ (z >> 31)
    return z & 0x7FFFFFFFFFFFFFFF


def _rng(device, *key: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_mix(*key))
    return g


def sink_mask(cfg: Workload, layer: int) -> np.ndarray:
    """uint8 [H]: 1 where the generator builds a semantic-sink head."""
    rs = np.random.Generator(np.random.Philox(key=_mix(cfg.seed, 11, layer)))
    perm = rs.permutation(cfg.n_heads)
    m = np.zeros(cfg.n_heads, np.uint8)
    m[perm[: cfg.n_sink_heads]] = 1
    return m


def _smoother(n: int, sigma: float, device) -> torch.Tensor:
    i = torch.arange(n, dtype=torch.float32, device=device)
    G = torch.exp(-((i[:, None] - i[None, :]) ** 2) / (2.0 * sigma * sigma))
    return G / G.pow(2).sum(dim=1, keepdim=True).sqrt()


def _field(cfg: Workload, gen: torch.Generator, device) -> torch.Tensor:
    """Unit-variance smoothed field [H, N, D] on the h x w grid."""
    h, w = cfg.grid
    z = torch.randn((cfg.n_heads, h, w, cfg.head_dim), generator=gen, device=device,
                    dtype=torch.float32)
    Gr, Gc = _smoother(h, cfg.sigma, device), _smoother(w, cfg.sigma, device)
    f = torch.einsum("ri,cj,hijd->hrcd", Gr, Gc, z)
    return f.reshape(cfg.n_heads, h * w, cfg.head_dim)


def gen_sequence(cfg: Workload, layer: int, seq: int, device="cpu", plant_below: Optional[int] = None):
    """One sequence of one layer: q [H,N,D] (image queries), k, v [H,L+N,D] (bf16),
    planted [H, N_PLANTED] int64 (image indices; -1 on spatial heads)."""
    H, L, N, D = cfg.n_heads, cfg.prompt_len, cfg.n_img, cfg.head_dim
    gen = _rng(device, cfg.seed, 1, layer, seq)
    q = torch.randn((H, N, D), generator=gen, device=device, dtype=torch.float32)
    k = torch.randn((H, L + N, D), generator=gen, device=device, dtype=torch.float32)
    v = torch.randn((H, L + N, D), generator=gen, device=device, dtype=torch.float32)
    f_qk = _field(cfg, gen, device)
    f_v = _field(cfg, gen, device)
    sem = torch.from_numpy(sink_mask(cfg, layer).astype(np.bool_)).to(device)
    gain = torch.where(sem, torch.tensor(G_SINK, device=device), torch.tensor(G_SPATIAL, device=device))
    gain = gain.view(H, 1, 1)
    q += gain * f_qk
    k[:, L:] += gain * f_qk
    v[:, L:] += gain * f_v
    # semantic-sink structure: one direction per (layer, head), shared by all sequences
    gmu = _rng(device, cfg.seed, 2, layer)
    mu = torch.randn((H, D), generator=gmu, device=device, dtype=torch.float32)
    mu = mu / mu.norm(dim=1, keepdim=True)
    q += torch.where(sem.view(H, 1, 1), C_MU * mu.view(H, 1, D), torch.zeros((), device=device))
    hi = plant_below if plant_below is not None else max(cfg.n0 - cfg.sink_recent, 0)
    planted = torch.full((H, N_PLANTED), -1, dtype=torch.int64, device=device)
    if hi >= N_PLANTED and cfg.n_sink_heads > 0:
        r = torch.rand((H, hi), generator=gen, device=device)
        pick = r.argsort(dim=1)[:, :N_PLANTED]          # without replacement
        planted = torch.where(sem.view(H, 1), pick, planted)
        for h in torch.nonzero(sem).flatten().tolist():
            rows = L + pick[h]
            norms = k[h, rows].norm(dim=1, keepdim=True)
            k[h, rows] = PLANT_NORM * norms * mu[h].view(1, D)
    return (q.to(torch.bfloat16), k.to(torch.bfloat16), v.to(torch.bfloat16), planted)


def gen_layer(cfg: Workload, layer: int, seqs, device="cpu"):
    """Stack ``gen_sequence`` over sequence ids -> q [S,H,N,D], k, v [S,H,L+N,D], planted [S,H,4]."""
    outs = [gen_sequence(cfg, layer, int(s), device) for s in seqs]
    return tuple(torch.stack([o[i] for o in outs]) for i in range(4))


def gen_calibration(cfg: Workload, layers, device="cpu"):
    """Calibration batch for head classification: q [layers,P,H,N,D], k [layers,P,H,L+N,D]."""
    qs, ks = [], []
    for layer in layers:
        q, k, _, _ = gen_layer(cfg, layer, [CAL_SEQ_BASE + p for p in range(cfg.n_cal)], device)
        qs.append(q)
        ks.append(k)
    return torch.stack(qs), torch.stack(ks)


def to_u16(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 bit patterns on the host (what the CPU checker consumes)."""
    assert t.dtype == torch.bfloat16
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def from_f32(a: np.ndarray) -> np.ndarray:
    """float array -> bf16 bit patterns (round to nearest even), for hand-made test inputs."""
    t = torch.from_numpy(np.ascontiguousarray(a, np.float32)).to(torch.bfloat16)
    return to_u16(t)
