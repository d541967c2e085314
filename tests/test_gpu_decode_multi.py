"""GPU parity of the densified block-decoder step (m new rows and m queries per (sequence, head)
in one launch, tensor-core arithmetic) against the oracle.  Cache bytes and lengths bit-exact;
outputs within |g - r| <= 1e-2 + 2e-2 |r| (the softmax weights meet V in bf16)."""
import numpy as np
import pytest
import torch

import oracle
from workloads import gen

from util import assert_close, status_word, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bt():
    import paper_2406_02657_b200 as bt
    assert torch.cuda.is_available()
    return bt


def rnd(seed, tid, shape):
    return gen.normal_bf16_bits(seed, tid, shape)


@pytest.mark.parametrize("hd", [64, 128])
@pytest.mark.parametrize("m", [1, 2, 4, 8])
def test_multi_step_ragged_lengths_three_steps(bt, m, hd):
    """Lengths around every chunk boundary, an empty cache, caches with exactly room, one row short of
    room and full; rows past each length hold NaN; three steps in a row on one workspace."""
    B, H, N = 12, 3, 168
    cfg = bt.make_config(B, H, hd, m, 1, N, 1)
    lens = np.array([0, 1, 15, 16, 31, 32, 33, 95, N - 3 * m, N - m, N - m + 1, N], np.int32)
    k, v = rnd(400 + m + hd, 1, (B, H, N, hd)), rnd(400 + m + hd, 2, (B, H, N, hd))
    oc = oracle.Cache(B, H, N, hd)
    oc.k[...], oc.v[...], oc.len[...] = k, v, lens
    kp, vp = k.copy(), v.copy()
    for b in range(B):
        kp[b, :, lens[b]:] = 0x7FC0
        vp[b, :, lens[b]:] = 0x7FC0
    cache = bt.BlockCache(cfg)
    cache.k[0].copy_(to_dev(kp))
    cache.v[0].copy_(to_dev(vp))
    cache.len[0].copy_(torch.from_numpy(lens).cuda())
    ws = bt.alloc_workspace(cfg)
    out = torch.empty((B, H, m, hd), dtype=torch.bfloat16, device="cuda")
    for step in range(3):
        q, kn, vn = (rnd(410 + m + hd, 3 * step + i, (B, H, m, hd)) for i in range(3))
        st = status_word()
        out.fill_(7.0)
        bt.bt_block_decode_step_multi(cfg, cache, 0, to_dev(q), to_dev(kn), to_dev(vn), out, ws, dev_status=st)
        oc.status[...] = 0
        ref = oracle.block_decode_step_multi(oc, q, kn, vn)
        assert cache.len[0].cpu().tolist() == oc.len.tolist(), f"step {step}: lengths"
        assert st.item() == int(oc.status[0]) and st.item() & bt.BT_DEV_OVERFLOW  # the full cache at least
        assert_close(out, ref, f"multi step {step} m={m} hd={hd}", p_bf16=True)
        gk, gv = gen.torch_to_bits(cache.k[0]), gen.torch_to_bits(cache.v[0])
        for b in range(B):
            n = int(oc.len[b])
            assert np.array_equal(gk[b, :, :n], oc.k[b, :, :n]) and np.array_equal(gv[b, :, :n], oc.v[b, :, :n])
            assert (gk[b, :, n:] == 0x7FC0).all() and (gv[b, :, n:] == 0x7FC0).all()
    assert not ws.view(torch.int32)[-(B * H + B):].any()   # the arrival counters are back at zero


@pytest.mark.parametrize("hd,n0", [(64, 45), (128, 45), (64, 62), (128, 14)])
def test_multi_step_causal_rule_among_the_new_rows(bt, hd, n0):
    """New row j carries a key that dominates everything: query i must return the value of the last
    new row it may see (row i), never a later one.  (n0 = 62 and 14: the new rows straddle a chunk end.)"""
    B, H, N, m = 2, 2, 128, 4
    cfg = bt.make_config(B, H, hd, m, 1, N, 1)
    cache = bt.BlockCache(cfg)
    cache.k[0].copy_(to_dev(rnd(420, 1, (B, H, N, hd))))
    cache.v[0].copy_(to_dev(rnd(420, 2, (B, H, N, hd))))
    cache.len[0].fill_(n0)
    q = gen.f32_to_bf16_bits(np.full((B, H, m, hd), 2.0, np.float32))
    kn = np.zeros((B, H, m, hd), np.float32)
    vn = np.zeros((B, H, m, hd), np.float32)
    for j in range(m):
        kn[:, :, j] = 6.0 + 3.0 * j            # later rows dominate earlier ones by e^(2*3*sqrt(hd)) each
        vn[:, :, j] = np.arange(hd) - 30.0 + 100.0 * j
    out = torch.empty((B, H, m, hd), dtype=torch.bfloat16, device="cuda")
    bt.bt_block_decode_step_multi(cfg, cache, 0, to_dev(q), to_dev(gen.f32_to_bf16_bits(kn)), to_dev(gen.f32_to_bf16_bits(vn)),
                                  out, bt.alloc_workspace(cfg))
    got = out.double().cpu().numpy()
    for i in range(m):
        want = gen.bf16_bits_to_f32(gen.f32_to_bf16_bits(vn[0, 0, i]))
        assert np.abs(got[:, :, i] - want).max() <= 1e-2 + 2e-2 * np.abs(want).max(), f"query {i} saw another row"
    assert (cache.len[0] == n0 + m).all()


def test_multi_step_many_items_per_warp_and_single_query_entry_points_agree(bt):
    """More (b,h) pairs than warps on the GPU, two layers; with m = 1 the launch computes what
    bt_block_decode_step computes (other arithmetic, same definition)."""
    B, H, hd, N, m = 96, 16, 64, 160, 4
    cfg = bt.make_config(B, H, hd, m, 1, N, 2)
    fill = lambda tid, shape: gen.normal_bf16_device(430, tid, shape, device="cuda")
    cache = bt.BlockCache(cfg, k=fill(0, (2, B, H, N, hd)), v=fill(1, (2, B, H, N, hd)))
    cache.len.fill_(N - 2 * m)
    ws = bt.alloc_workspace(cfg)
    st = status_word()
    out = torch.empty((2, B, H, m, hd), dtype=torch.bfloat16, device="cuda")
    sel = [0, 50, 95]
    ocs = []
    for l in range(2):
        oc = oracle.Cache(len(sel), H, N, hd)
        oc.k[...], oc.v[...] = gen.torch_to_bits(cache.k[l][sel]), gen.torch_to_bits(cache.v[l][sel])
        oc.len[...] = N - 2 * m
        ocs.append(oc)
    for step in range(2):
        q, kn, vn = (fill(10 + 3 * step + i, (2, B, H, m, hd)) for i in range(3))
        for l in range(2):
            bt.bt_block_decode_step_multi(cfg, cache, l, q[l], kn[l], vn[l], out[l], ws, dev_status=st)
        torch.cuda.synchronize()
        for l in range(2):
            ref = oracle.block_decode_step_multi(ocs[l], *(gen.torch_to_bits(x[l][sel]) for x in (q, kn, vn)))
            assert_close(out[l][sel], ref, f"step {step} layer {l}", p_bf16=True)
            assert torch.equal(cache.k[l][:, :, N - 2 * m + step * m:N - m + step * m], kn[l])
    assert st.item() == 0 and (cache.len == N).all()
    # m = 1 against the CUDA-core fused step
    cfg1 = bt.make_config(B, H, hd, 1, 1, N, 2)
    a = bt.BlockCache(cfg1, k=cache.k.clone(), v=cache.v.clone())
    b = bt.BlockCache(cfg1, k=cache.k.clone(), v=cache.v.clone())
    a.len.fill_(N - 1)
    b.len.fill_(N - 1)
    q, kn, vn = (fill(30 + i, (B, H, 1, hd)) for i in range(3))
    oa, ob = torch.empty_like(q), torch.empty_like(q)
    bt.bt_block_decode_step_multi(cfg1, a, 0, q, kn, vn, oa, ws, dev_status=st)
    bt.bt_block_decode_step(cfg1, b, 0, q, kn, vn, ob, ws, dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0 and torch.equal(a.k, b.k) and torch.equal(a.v, b.v) and torch.equal(a.len, b.len)
    assert (oa.float() - ob.float()).abs().max().item() <= 1e-2


def test_multi_step_rejects_what_it_does_not_support(bt):
    x = torch.zeros((2, 2, 4, 128), dtype=torch.bfloat16, device="cuda")
    cfg = bt.make_config(2, 2, 128, 4, 1, 24, 1)   # a cache shorter than one chunk
    with pytest.raises(bt.BtError) as e:
        bt.bt_block_decode_step_multi(cfg, bt.BlockCache(cfg), 0, x, x, x, torch.empty_like(x), bt.alloc_workspace(cfg))
    assert "BT_ERR_UNSUPPORTED" in str(e.value)
    cfg = bt.make_config(2, 2, 64, 4, 1, 64, 1)
    y = torch.zeros((2, 2, 9, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(bt.BtError) as e:
        bt.bt_block_decode_step_multi(cfg, bt.BlockCache(cfg), 0, y, y, y, torch.empty_like(y), bt.alloc_workspace(cfg))
    assert "BT_ERR_UNSUPPORTED" in str(e.value)
