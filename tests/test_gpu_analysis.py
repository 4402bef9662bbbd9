"""GPU parity of the analysis utility: per-token divergence of two KV caches (Sec. 3.2, MSE_token)
against the fp64 oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_18716_b200 import binding as B
from paper_2510_18716_b200 import workloads as wl

pytestmark = pytest.mark.gpu

RTOL = 1e-5      # fp32 sums of 256 squared differences of exactly widened bf16 values against fp64


def _pair_of_caches(shape, seed, dev):
    g = torch.Generator(device=dev).manual_seed(seed)
    return [(torch.randn(shape, generator=g, device=dev) * (1.0 + i)).to(torch.bfloat16) for i in range(4)]


@pytest.mark.parametrize("shape", [(1, 128), (7, 128), (33, 128), (3, 5, 641, 128), (2, 16, 4224, 128)])
def test_kv_token_mse_matches_oracle(shape):
    dev = torch.device("cuda:0")
    ka, va, kb, vb = _pair_of_caches(shape, 7 + len(shape), dev)
    got = B.kv_token_mse(ka, va, kb, vb).cpu().numpy().astype(np.float64)
    want = oracle.kv_token_mse(*(wl.to_u16(x) for x in (ka, va, kb, vb)))
    assert got.shape == want.shape == shape[:-1]
    assert np.allclose(got, want, rtol=RTOL, atol=0.0), np.abs(got / want - 1).max()
    # identical caches: exactly zero; one token of one tensor changed: only that row moves
    zero = B.kv_token_mse(ka, va, ka, va)
    assert (zero == 0).all()
    vb2 = va.clone()
    vb2.view(-1, 128)[-1, 5] += 1.0
    one = B.kv_token_mse(ka, va, ka, vb2).view(-1)
    assert (one[:-1] == 0).all() and one[-1] > 0


def test_kv_token_mse_on_generated_branches():
    """Two sequences of a CFG pair as the generator makes them (one layer of the 7B shape, all heads): the
    shapes and value ranges the analysis is run on."""
    cfg = wl.CONFIGS["janus7b"]
    dev = torch.device("cuda:0")
    _, k, v, _ = wl.gen_layer(cfg, 4, [0, 1], device=dev)
    got = B.kv_token_mse(k[0].contiguous(), v[0].contiguous(), k[1].contiguous(), v[1].contiguous())
    want = oracle.kv_token_mse(wl.to_u16(k[0]), wl.to_u16(v[0]), wl.to_u16(k[1]), wl.to_u16(v[1]))
    assert got.shape == (cfg.n_heads, cfg.prompt_len + cfg.n_img)
    assert np.allclose(got.cpu().numpy().astype(np.float64), want, rtol=RTOL, atol=0.0)


def test_kv_token_mse_argument_errors():
    dev = torch.device("cuda:0")
    lib, st = B.load(), torch.cuda.current_stream().cuda_stream
    x = torch.zeros((4, 128 + 8), dtype=torch.bfloat16, device=dev)
    o = torch.zeros(4, dtype=torch.float32, device=dev)
    p = x.data_ptr()
    before = B.kernel_launch_count()
    assert lib.ssd_kv_token_mse(None, p, p, p, 4, o.data_ptr(), st) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_kv_token_mse(p, p, p, p, 4, None, st) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_kv_token_mse(p + 2, p, p, p, 4, o.data_ptr(), st) == B.SSD_ERR_INVALID_ARG       # misaligned
    assert lib.ssd_kv_token_mse(p, p, p, p, -1, o.data_ptr(), st) == B.SSD_ERR_INVALID_ARG
    assert lib.ssd_kv_token_mse(p, p, p, p, 0, o.data_ptr(), st) == B.SSD_OK                        # nothing to do
    assert B.kernel_launch_count() == before
