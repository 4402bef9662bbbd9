"""Multi-GPU plumbing: the path shards by sequence with no data-path collective.

Every (layer, sequence, head) is independent in compress / append / decode, so rank r simply owns
a contiguous block of sequences, with both sequences of a classifier-free-guidance pair on the
same rank (the logit mix after the LM head needs both).  The only exchange is in head
classification, where the per-(layer, head) ratio sums of the sparsity metric (Sec. 3.3) over a
sharded calibration batch are added across ranks so that all ranks install identical labels: one
all-reduce of n_layers * n_heads doubles.
"""
from __future__ import annotations

from typing import List, Tuple

import numpy as np
import torch


def shard_sequences(n_seqs_total: int, rank: int, world: int) -> Tuple[int, int]:
    """[lo, hi) of the sequences rank owns; CFG pairs (2k, 2k+1) are never split."""
    if n_seqs_total % 2:
        units, per = n_seqs_total, 1
    else:
        units, per = n_seqs_total // 2, 2
    base, extra = divmod(units, world)
    lo = rank * base + min(rank, extra)
    hi = lo + base + (1 if rank < extra else 0)
    return lo * per, hi * per


def shard_calibration(n_cal: int, rank: int, world: int) -> List[int]:
    """Indices of the calibration sequences rank measures (round robin; may be empty)."""
    return list(range(rank, n_cal, world))


def reduce_ratio_sums(local_sums: np.ndarray, group=None) -> np.ndarray:
    """Sum the per-(layer, head) ratio sums over all ranks (identity without a process group)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return np.asarray(local_sums, np.float64)
    backend = dist.get_backend(group)
    t = torch.from_numpy(np.ascontiguousarray(local_sums, np.float64).copy())
    if backend == "nccl":
        t = t.cuda()
    dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return t.cpu().numpy()


def labels_from_sums(total_sums: np.ndarray, n_cal_total: int, n_img: int, tau: float) -> np.ndarray:
    """Labels from ratio sums added over ranks: the library's own threshold rule
    (ssd_labels_from_ratio_sums, the arithmetic ssd_classify_heads uses), not a restatement of it."""
    from . import binding
    return binding.labels_from_ratio_sums(total_sums, n_cal_total, n_img, tau)[1]


def classify_sharded(cache, q_cal_local, k_cal_local, n_cal_total: int, n_img: int, tau: float, group=None):
    """Classify heads from a calibration batch sharded over ranks and install the labels.

    q_cal_local / k_cal_local hold this rank's calibration sequences (None if it has none)."""
    n = cache.cfg.n_layers * cache.cfg.n_heads
    if q_cal_local is not None and q_cal_local.shape[1] > 0:
        sums = cache.classify_partial(q_cal_local, k_cal_local).reshape(-1)
    else:
        sums = np.zeros(n, np.float64)
    total = reduce_ratio_sums(sums, group)
    labels = labels_from_sums(total, n_cal_total, n_img, tau)
    cache.set_head_labels(labels)
    return labels.reshape(cache.cfg.n_layers, cache.cfg.n_heads)
