"""The decode kernel's work decomposition, enumerated on the host by the very code the kernel
runs: every copy must stay inside the layer's slab, every valid slot must be copied exactly once,
no chunk may cross a (sequence, head) boundary or exceed a stage, and shares must be balanced."""
import numpy as np
import pytest

from paper_2510_18716_b200 import binding as B


def layout(labels, L, W, M, R):
    recs, off = [], 0
    for sem in labels:
        y, z = (M, R) if sem else (0, W)
        recs.append((off, y, z, int(sem)))
        off += L + y + z
    return np.array(recs, np.int32), off


def valid_slots(recs, L, prompt_valid, static_valid, t_img):
    """Per head: sorted physical slots (relative to the head) that hold a token."""
    out = []
    for (x, y, z, w) in recs:
        s = list(range(prompt_valid))
        if w:
            s += [L + m for m in range(static_valid)]
        s += [L + y + r for r in range(min(t_img, z))]
        out.append(s)
    return out


def check_plan(labels, L, W, M, R, n_seqs, prompt_valid, static_valid, t_img, max_workers, chunk):
    recs, seq_slots = layout(labels, L, W, M, R)
    H = len(labels)
    plan = B.decode_plan(recs, L, n_seqs, prompt_valid, static_valid, t_img, max_workers, chunk)
    per_head = valid_slots(recs, L, prompt_valid, static_valid, t_img)
    want = []
    for s in range(n_seqs):
        for h in range(H):
            want += [s * seq_slots + recs[h][0] + p for p in per_head[h]]
    total = len(want)
    got = []
    assert (plan[:, 4] >= 1).all()
    for wk, k, src, dst, n, pair in plan:
        s, h = divmod(int(pair), H)
        lo = s * seq_slots + recs[h][0]
        hi = lo + L + recs[h][1] + recs[h][2]
        assert lo <= src and src + n <= hi, "copy leaves the head's region"
        assert 0 <= dst and dst + n <= chunk, "copy leaves the stage"
        got += list(range(int(src), int(src + n)))
    # the stream is ordered by (sequence, head, slot) and the plan walks it in order, worker by worker
    assert got == want, "every valid slot exactly once, in stream order"
    # one chunk = one (worker, k): a single head, at most `chunk` slots, destinations tile [0, n)
    key = plan[:, 0] * (1 << 32) + plan[:, 1]
    for kk in np.unique(key):
        rows = plan[key == kk]
        assert len(set(rows[:, 5].tolist())) == 1
        assert rows[:, 4].sum() <= chunk and len(rows) <= 3
        d = 0
        for r in rows:
            assert r[3] == d
            d += r[4]
    # balance: shares differ by less than one alignment unit plus rounding
    if total >= 16 * 2:
        per_worker = np.bincount(plan[:, 0].astype(np.int64), weights=plan[:, 4]).astype(np.int64)
        per_worker = per_worker[per_worker > 0]
        assert per_worker.max() - per_worker.min() <= 16
        assert len(per_worker) == min(max_workers, max(total // 16, 1))
    return plan


def test_steady_state_7b_shape_is_one_copy_per_chunk():
    labels = [1, 0, 0, 1, 0, 1, 0, 0] * 4
    plan = check_plan(labels, 64, 64, 96, 24, 4, 64, 96, 400, 148 * 8, 16)
    # full prompt, full static set, full ring: every head is one physical run
    key = plan[:, 0] * (1 << 32) + plan[:, 1]
    assert len(np.unique(key)) == len(plan)
    assert (plan[:, 4] == 16).mean() > 0.8


@pytest.mark.parametrize("seed", range(40))
def test_random_layouts_and_occupancies(seed):
    rng = np.random.default_rng(seed)
    H = int(rng.integers(1, 9))
    labels = rng.integers(0, 2, H).tolist()
    L = int(rng.integers(0, 9))
    W, M, R = int(rng.integers(1, 20)), int(rng.integers(0, 20)), int(rng.integers(1, 9))
    n_seqs = int(rng.integers(1, 5))
    prompt_valid = L if rng.random() < 0.6 else 0
    static_valid = int(rng.integers(0, M + 1))
    t_img = int(rng.integers(0 if prompt_valid else 1, 40))
    if prompt_valid + t_img == 0:
        t_img = 1
    check_plan(labels, L, W, M, R, n_seqs, prompt_valid, static_valid, t_img,
               int(rng.integers(1, 40)), int(rng.choice([8, 16, 32])))


def test_full_cache_shape_long_heads_split_over_many_workers():
    labels = [0] * 6
    check_plan(labels, 64, 576, 0, 1, 3, 64, 0, 576, 64, 16)
    check_plan(labels, 64, 576, 0, 1, 3, 0, 0, 5, 64, 16)      # before any compress: prompt slots unused
    check_plan([0, 1], 8, 4000, 100, 50, 1, 8, 100, 3000, 1184, 16)   # few long heads, many workers


def test_bad_plans_are_rejected():
    lib = B.load()
    recs = np.array([[0, 0, 4, 0]], np.int32)
    out = np.zeros((4, 6), np.int64)
    assert lib.ssd_debug_decode_plan(1, recs.ctypes.data, 2, 1, 1, 0, 1, 4, 8, out.ctypes.data, 4) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_debug_decode_plan(1, recs.ctypes.data, 2, 1, 0, 0, 0, 4, 8, out.ctypes.data, 4) == B.SSD_ERR_BAD_STATE
    assert lib.ssd_debug_decode_plan(0, recs.ctypes.data, 2, 1, 2, 0, 1, 4, 8, out.ctypes.data, 4) == B.SSD_ERR_INVALID_ARG
    bad = np.array([[3, 0, 4, 0]], np.int32)    # heads must be packed from slot 0
    assert lib.ssd_debug_decode_plan(1, bad.ctypes.data, 2, 1, 2, 0, 1, 4, 8, out.ctypes.data, 4) == B.SSD_ERR_INVALID_ARG
