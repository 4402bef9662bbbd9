"""ssd_decode_attn_static: decode attention for callers that cannot give the library scratch memory.

Some users of this library cannot allocate where they call it: code between the capture calls of a
stream, a plugin whose host program owns all device memory, a loop that must never hit an
allocation's hidden synchronisation.  For them the decode kernel's scratch sits in an array inside
the library image.  The entry point must give exactly what ssd_decode_attn gives, call after call
(the array is shared by all calls and keeps the previous call's contents), and must refuse sizes
its fixed array cannot serve."""
import numpy as np
import pytest
import torch

from paper_2510_18716_b200 import binding as B
from paper_2510_18716_b200 import workloads as wl

from parity_util import MAX_ABS, MEAN_ABS

pytestmark = pytest.mark.gpu


def _filled_cache(cfg, seqs, device):
    """A one-layer cache compressed at n0, and the layer's inputs."""
    L, n0 = cfg.prompt_len, cfg.n0
    cache = B.SsdCache(B.config_from_workload(cfg, n_layers=1, n_seqs=len(seqs)), device=device)
    cache.set_head_labels(wl.sink_mask(cfg, 0))
    q, k, v, _ = wl.gen_layer(cfg, 0, seqs, device=device)
    cache.compress(0, q[:, :, :n0].contiguous(), k[:, :, : L + n0].contiguous(), v[:, :, : L + n0].contiguous(), n0)
    return cache, q, k, v


@pytest.mark.parametrize("name,seqs", [("tiny", [0]), ("janus7b", list(range(6)))])
def test_static_scratch_matches_regular_entry_point_on_consecutive_calls(name, seqs):
    cfg = wl.CONFIGS[name]
    dev = torch.device("cuda:0")
    L, n0 = cfg.prompt_len, cfg.n0
    cache, q, k, v = _filled_cache(cfg, seqs, dev)
    out_static = torch.empty((len(seqs), cfg.n_heads, 128), dtype=torch.bfloat16, device=dev)
    for t in (n0 + 1, n0 + 2, n0 + 3):                 # calls in a row reuse the same array
        cache.append(0, k[:, :, L + t - 1].contiguous(), v[:, :, L + t - 1].contiguous())
        qt = q[:, :, t - 1].contiguous()
        want = cache.decode_attn(0, qt)
        out_static.fill_(float("nan"))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info(dev)[0]
        got = cache.decode_attn_static(0, qt, out_static)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info(dev)[0] == free_before, "the call must not allocate device memory"
        assert torch.isfinite(got.float()).all()
        err = (got.float() - want.float()).abs()
        assert err.max().item() <= MAX_ABS and err.mean().item() <= MEAN_ABS
        assert torch.equal(got, want), "same kernel, same merge order: expected identical bits"
    assert cache.device_status() == 0
    cache.close()


def test_static_scratch_refuses_more_pairs_than_it_has_counters_for():
    dev = torch.device("cuda:0")
    n_seqs, H = 1024, 33                               # 33792 pairs > 32768
    cfg = B.make_config(1, n_seqs, H, 0, 4, 1, 0, 1)
    cache = B.SsdCache(cfg, device=dev)
    cache.set_head_labels(np.zeros(H, np.uint8))
    x = torch.zeros((n_seqs, H, 128), dtype=torch.bfloat16, device=dev)
    cache.append(0, x, x)
    before = B.kernel_launch_count()
    with pytest.raises(B.SsdError) as e:
        cache.decode_attn_static(0, x)
    assert e.value.code == B.SSD_ERR_LIMIT
    assert B.kernel_launch_count() == before            # refused on the host, nothing launched
    out = cache.decode_attn(0, x)                       # the regular entry point still serves it
    torch.cuda.synchronize()
    assert torch.equal(out, x)                          # one token per head: output = its V row = 0
    cache.close()
