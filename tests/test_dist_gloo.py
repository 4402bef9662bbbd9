"""Multi-rank host logic on CPU (gloo, world size 2): sequence sharding and the one exchange the
path has, the all-reduce of the sparsity-metric ratio sums (Sec. 3.3) over a sharded calibration
batch, after which every rank must hold identical head labels."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2510_18716_b200 import dist as D
from paper_2510_18716_b200 import workloads as wl


def test_shard_sequences_keeps_cfg_pairs_together_and_covers_everything():
    for total in (2, 6, 64, 128, 7, 1):
        for world in (1, 2, 3, 4, 8):
            got = []
            for r in range(world):
                lo, hi = D.shard_sequences(total, r, world)
                assert 0 <= lo <= hi <= total
                if total % 2 == 0:
                    assert lo % 2 == 0 and hi % 2 == 0      # (2k, 2k+1) never split
                got += list(range(lo, hi))
            assert got == list(range(total))
            sizes = [D.shard_sequences(total, r, world) for r in range(world)]
            per = [hi - lo for lo, hi in sizes]
            assert max(per) - min(per) <= (2 if total % 2 == 0 else 1)


def test_shard_calibration_round_robin():
    for n in (0, 1, 4, 5):
        for world in (1, 2, 3):
            parts = [D.shard_calibration(n, r, world) for r in range(world)]
            assert sorted(sum(parts, [])) == list(range(n))


def test_labels_from_sums_equality_is_spatial():
    P, N = 2, 10
    sums = np.array([0.45 * P * N, 0.45 * P * N + 1e-3, 0.0, P * N])
    # s is taken in float32, like the single-GPU entry point does
    want = (np.float32(1) * (sums / (P * N)).astype(np.float32) > np.float32(0.45)).astype(np.uint8)
    assert D.labels_from_sums(sums, P, N, 0.45).tolist() == want.tolist()
    assert D.labels_from_sums(sums, P, N, 0.45)[0] == 0 and D.labels_from_sums(sums, P, N, 0.45)[-1] == 1


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


class _FakeCache:
    """Stands in for the CUDA cache on a CPU machine: ratio sums come from the fp64 checker, which is
    fine here because the subject of the test is the exchange, not the kernel."""

    class _Cfg:
        pass

    def __init__(self, cfg):
        self.cfg = self._Cfg()
        self.cfg.n_layers, self.cfg.n_heads = 1, cfg.n_heads
        self.w, self.L = cfg.cls_window, cfg.prompt_len
        self.labels = None

    def classify_partial(self, q, k):
        P, N = q.shape[1], q.shape[3]
        return oracle.sparsity(wl.to_u16(q), wl.to_u16(k), self.L, self.w) * (P * N)

    def set_head_labels(self, labels):
        self.labels = np.asarray(labels).copy()


def _worker(rank, world, port, n_cal, ret):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = wl.Workload("g", 1, 2, 6, 8, (6, 8), 8, 8, 4, 12, 3, 24, n_cal, 1.5, tau=0.30, seed=5)
        mine = D.shard_calibration(cfg.n_cal, rank, world)
        cache = _FakeCache(cfg)
        if mine:
            q, k, _, _ = wl.gen_layer(cfg, 0, [wl.CAL_SEQ_BASE + p for p in mine])
            q, k = q[None], k[None]
        else:
            q = k = None
        labels = D.classify_sharded(cache, q, k, cfg.n_cal, cfg.n_img, cfg.tau)
        # every rank must agree with the unsharded measurement
        qa, ka = wl.gen_calibration(cfg, [0])
        s = oracle.sparsity(wl.to_u16(qa), wl.to_u16(ka), cfg.prompt_len, cfg.cls_window)
        want = D.labels_from_sums(s * cfg.n_cal * cfg.n_img, cfg.n_cal, cfg.n_img, cfg.tau)
        ok = np.array_equal(labels, want) and np.array_equal(cache.labels.reshape(1, -1), want)
        # the reduced sums themselves
        part = cache.classify_partial(q, k).reshape(-1) if mine else np.zeros(cfg.n_heads)
        tot = D.reduce_ratio_sums(part)
        ok = ok and np.allclose(tot, (s * cfg.n_cal * cfg.n_img).reshape(-1), rtol=1e-12)
        t = torch.tensor([1.0 if ok else 0.0])
        dist.all_reduce(t, op=dist.ReduceOp.MIN)
        ret[rank] = float(t.item())
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("n_cal", [3, 1])
def test_sharded_classification_two_ranks_gloo(n_cal):
    world = 2
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), n_cal, ret), nprocs=world, join=True)
    assert dict(ret) == {0: 1.0, 1: 1.0}


def test_reduce_without_process_group_is_identity():
    x = np.arange(6, dtype=np.float64)
    assert np.array_equal(D.reduce_ratio_sums(x), x)
