"""bt_block_decode_attn_noalloc: the decode attention for callers that cannot allocate device
memory (a server whose pool already owns the GPU, a latency-bound loop that must not trigger
cudaMalloc's device-wide synchronisation).  Its split scratch is a fixed array inside the library,
shared by every call, so the checks here are: the oracle's result within the stated tolerance and,
bit for bit, the output of bt_block_decode_attn with a caller-owned workspace (same kernel, same
splits, same merge order), on two calls in a row with different shapes (the second call finds the
first one's leftovers in the scratch), and a clean refusal when the scratch would not fit.

Collected last on purpose (file name): a run that stops at the first failure has then already
run every other test."""
import ctypes

import numpy as np
import pytest
import torch

from workloads import gen

import oracle

from util import assert_close, status_word, to_dev


@pytest.fixture(scope="module")
def bt():
    import paper_2406_02657_b200 as bt
    return bt


def _case(bt, seed, B, H, hd, N, splits, lens):
    cfg = bt.make_config(B, H, hd, 4, 1, N, 1, decode_splits=splits)
    assert 0 < bt.bt_workspace_bytes(cfg) <= bt.BT_STATIC_WORKSPACE_BYTES  # the scratch is really used
    cache = bt.BlockCache(cfg)
    k, v, q = (gen.normal_bf16_bits(seed, i, (B, H, N, hd) if i else (B, H, hd)) for i in (1, 2, 0))
    cache.k[0].copy_(to_dev(k))
    cache.v[0].copy_(to_dev(v))
    cache.len[0].copy_(torch.from_numpy(np.asarray(lens, np.int32)).cuda())
    oc = oracle.Cache(B, H, N, hd)
    oc.k[...], oc.v[...], oc.len[...] = k, v, lens
    return cfg, cache, to_dev(q), oracle.block_decode_attn(oc, q)


@pytest.mark.gpu
def test_noalloc_matches_workspace_entry_point_twice_in_a_row(bt):
    assert torch.cuda.is_available()
    cases = [(901, 5, 3, 64, 300, 5, [300, 1, 77, 128, 299]),
             (902, 3, 2, 128, 131, 3, [131, 64, 2])]
    for seed, B, H, hd, N, splits, lens in cases:
        cfg, cache, q, ref = _case(bt, seed, B, H, hd, N, splits, lens)
        st = status_word()
        want = torch.full((B, H, hd), 7.0, dtype=torch.bfloat16, device="cuda")
        bt.bt_block_decode_attn(cfg, cache, 0, q, want, bt.alloc_workspace(cfg), dev_status=st)
        got = torch.full((B, H, hd), -7.0, dtype=torch.bfloat16, device="cuda")
        bt.bt_block_decode_attn_noalloc(cfg, cache, 0, q, got, dev_status=st)
        torch.cuda.synchronize()
        assert_close(got, ref, f"no-alloc decode, seed {seed}")   # the oracle, at the stated tolerance
        assert torch.equal(got, want)                              # the workspace entry point, bit for bit
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
