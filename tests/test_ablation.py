"""Host-side ablation helpers (no GPU): threshold sweep and random partition of the heads."""
import numpy as np

from paper_2510_18716_b200 import ablation as A
from paper_2510_18716_b200 import binding as B


def test_tau_sweep_is_monotone_and_equality_is_spatial():
    rng = np.random.default_rng(0)
    s = rng.random((6, 16)).astype(np.float32)
    s[0, 0] = np.float32(0.45)
    sweep = A.tau_sweep(s, (0.0, 0.45, 0.9))
    counts = [int(sweep[t].sum()) for t in (0.0, 0.45, 0.9)]
    assert counts[0] >= counts[1] >= counts[2] and counts[0] > counts[2]
    assert sweep[0.45][0, 0] == 0                      # s == tau is spatial (Sec. 3.3)
    assert sweep[0.0].sum() == (s > 0).sum()
    # fewer semantic heads = fewer slots when a semantic head holds more than a spatial one, and the
    # library's own size arithmetic agrees with the count
    slots = [A.kv_slots_per_sequence(sweep[t], 64, 64, 96, 24) for t in (0.0, 0.45, 0.9)]
    assert slots[0] >= slots[1] >= slots[2]
    cfg = B.make_config(6, 1, 16, 64, 576, 64, 96, 24)
    for t in (0.0, 0.9):
        a = B.required_bytes(cfg, int(sweep[t].sum()))
        b = B.required_bytes(cfg, 0)
        assert a - b == (A.kv_slots_per_sequence(sweep[t], 64, 64, 96, 24) - 6 * 16 * 128) * 512


def test_random_partition_keeps_the_budgets():
    labels = np.zeros((5, 32), np.uint8)
    labels[:, :13] = 1
    labels[3, :] = 0
    r = A.random_partition(labels, seed=7)
    assert (r.sum(1) == labels.sum(1)).all() and r.shape == labels.shape
    assert not np.array_equal(r, labels)
    assert np.array_equal(r, A.random_partition(labels, seed=7))        # seeded
    assert not np.array_equal(r, A.random_partition(labels, seed=8))
