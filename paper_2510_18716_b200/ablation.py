"""Host-side helpers for the paper's ablations of the head split (Sec. 4.4): a random partition
with the same budgets, and the partitions a sweep of the threshold tau produces from measured
sparsity values.  They only build label arrays (uint8 [n_layers, n_heads], 1 = semantic) for
``SsdCache.set_head_labels``; the kernels are the same for any labelling."""
from __future__ import annotations

from typing import Dict, Iterable

import numpy as np


def labels_for_tau(s: np.ndarray, tau: float) -> np.ndarray:
    """Labels the library's threshold rule (ssd_labels_from_sparsity) gives for sparsity values s."""
    from . import binding
    return binding.labels_from_sparsity(s, tau)


def tau_sweep(s: np.ndarray, taus: Iterable[float]) -> Dict[float, np.ndarray]:
    """Labels for every threshold of a sweep (the paper sweeps 0, 0.45 and 0.9)."""
    return {float(t): labels_for_tau(s, t) for t in taus}


def random_partition(labels: np.ndarray, seed: int) -> np.ndarray:
    """Same number of semantic heads in every layer as `labels`, at random positions: the
    paper's control in which the policies are kept and the assignment of heads is not."""
    labels = np.asarray(labels, np.uint8)
    rng = np.random.Generator(np.random.Philox(key=seed))
    out = np.zeros_like(labels)
    for l in range(labels.shape[0]):
        n_sem = int(labels[l].sum())
        out[l, rng.permutation(labels.shape[1])[:n_sem]] = 1
    return out


def kv_slots_per_sequence(labels: np.ndarray, prompt_len: int, window: int, sink_budget: int, sink_recent: int) -> int:
    """Slots (tokens kept) per sequence over all layers under a labelling: what a threshold costs."""
    labels = np.asarray(labels, np.uint8)
    n_sem = int(labels.sum())
    return n_sem * (prompt_len + sink_budget + sink_recent) + (labels.size - n_sem) * (prompt_len + window)
