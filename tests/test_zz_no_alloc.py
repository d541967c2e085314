"""bt_block_decode_attn_noalloc: the decode attention for callers that cannot allocate device
memory (a server whose pool already owns the GPU, a latency-bound loop that must not trigger
cudaMalloc's device-wide synchronisation).  Its split scratch is a fixed array inside the library,
shared by every call, so the checks here are: same output as bt_block_decode_attn with a
caller-owned workspace, on two calls in a row with different shapes (the second call finds the
first one's leftovers in the scratch), and a clean refusal when the scratch would not fit.

Collected last on purpose (file name): a run that stops at the first failure has then already
run every other test."""
import ctypes

import numpy as np
import pytest
import torch

from workloads import gen

from util import ATOL, RTOL, status_word, to_dev, to_f64


@pytest.fixture(scope="module")
def bt():
    import paper_2406_02657_b200 as bt
    return bt


def _case(bt, seed, B, H, hd, N, splits, lens):
    cfg = bt.make_config(B, H, hd, 4, 1, N, 1, decode_splits=splits)
    assert 0 < bt.bt_workspace_bytes(cfg) <= bt.BT_STATIC_WORKSPACE_BYTES  # the scratch is really used
    cache = bt.BlockCache(cfg)
    cache.k[0].copy_(to_dev(gen.normal_bf16_bits(seed, 1, (B, H, N, hd))))
    cache.v[0].copy_(to_dev(gen.normal_bf16_bits(seed, 2, (B, H, N, hd))))
    cache.len[0].copy_(torch.from_numpy(np.asarray(lens, np.int32)).cuda())
    q = to_dev(gen.normal_bf16_bits(seed, 0, (B, H, hd)))
    return cfg, cache, q


@pytest.mark.gpu
def test_noalloc_matches_workspace_entry_point_twice_in_a_row(bt):
    assert torch.cuda.is_available()
    cases = [(901, 5, 3, 64, 300, 5, [300, 1, 77, 128, 299]),
             (902, 3, 2, 128, 131, 3, [131, 64, 2])]
    for seed, B, H, hd, N, splits, lens in cases:
        cfg, cache, q = _case(bt, seed, B, H, hd, N, splits, lens)
        st = status_word()
        want = torch.full((B, H, hd), 7.0, dtype=torch.bfloat16, device="cuda")
        bt.bt_block_decode_attn(cfg, cache, 0, q, want, bt.alloc_workspace(cfg), dev_status=st)
        got = torch.full((B, H, hd), -7.0, dtype=torch.bfloat16, device="cuda")
        bt.bt_block_decode_attn_noalloc(cfg, cache, 0, q, got, dev_status=st)
        torch.cuda.synchronize()
        g, r = to_f64(got), to_f64(want)
        assert np.isfinite(g).all()
        err = np.abs(g - r)
        assert (err <= ATOL + RTOL * np.abs(r)).all(), f"seed {seed}: max err {err.max():.3e}"
        assert st.item() == 0


def test_noalloc_rejects_scratch_beyond_the_limit(bt):
    # 64 splits x 64 x 16 (b,h) x (128+4) floats = 34.6 MB of partials: refused before any CUDA call
    cfg = bt.make_config(64, 16, 128, 4, 1, 4096, 1, decode_splits=64)
    assert bt.bt_workspace_bytes(cfg) > bt.BT_STATIC_WORKSPACE_BYTES
    fake = ctypes.c_void_p(0x1000)  # never dereferenced
    bc = bt.binding.bt_block_cache(0x1000, 0x1000, 0x1000)
    rc = bt.lib().bt_block_decode_attn_noalloc(ctypes.byref(cfg), ctypes.byref(bc), 0, fake, fake, None, None)
    assert rc == bt.BT_ERR_WORKSPACE
    bad = bt.make_config(4, 8, 96, 4, 1, 64, 1)  # invalid configs get bt_block_decode_attn's own error
    assert bt.lib().bt_block_decode_attn_noalloc(ctypes.byref(bad), ctypes.byref(bc), 0, fake, fake, None, None) \
        == bt.BT_ERR_UNSUPPORTED
