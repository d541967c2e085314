"""GPU parity of the fused block-decoder step (append the new block's row and attend over the
cache including it, one launch) against the oracle's append followed by its attention, and of the
in-launch merge of split row ranges.  Cache bytes and lengths bit-exact; outputs within
|g - r| <= 1e-2 + 2e-2 |r|."""
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
@pytest.mark.parametrize("splits", [1, 2, 3, 7])
def test_fused_step_equals_append_then_attend(bt, hd, splits):
    """Ragged lengths around every chunk boundary, an empty cache, a cache one row short of full and a
    full one (no room: skipped, flagged, attended as it is); three steps in a row on one workspace."""
    B, H, N = 9, 3, 261
    cfg = bt.make_config(B, H, hd, 4, 1, N, 1, decode_splits=splits)
    lens = np.array([0, 1, 31, 32, 33, 127, 258, 260, 261], np.int32)
    k, v = rnd(300 + hd, 1, (B, H, N, hd)), rnd(300 + hd, 2, (B, H, N, hd))
    oc = oracle.Cache(B, H, N, hd)
    oc.k[...], oc.v[...], oc.len[...] = k, v, lens
    kp, vp = k.copy(), v.copy()
    for b in range(B):  # rows at and past the length are never read from the cache: NaN there
        kp[b, :, lens[b]:] = 0x7FC0
        vp[b, :, lens[b]:] = 0x7FC0
    cache = bt.BlockCache(cfg)
    cache.k[0].copy_(to_dev(kp))
    cache.v[0].copy_(to_dev(vp))
    cache.len[0].copy_(torch.from_numpy(lens).cuda())
    ws = bt.alloc_workspace(cfg)
    out = torch.empty((B, H, hd), dtype=torch.bfloat16, device="cuda")
    for step in range(3):
        q = rnd(310 + hd, 3 * step, (B, H, hd))
        kn, vn = rnd(310 + hd, 3 * step + 1, (B, H, 1, hd)), rnd(310 + hd, 3 * step + 2, (B, H, 1, hd))
        st = status_word()
        out.fill_(7.0)
        bt.bt_block_decode_step(cfg, cache, 0, to_dev(q), to_dev(kn), to_dev(vn), out, ws, dev_status=st)
        oc.status[...] = 0
        oracle.kv_append(oc, kn, vn)
        ref = oracle.block_decode_attn(oc, q)
        assert cache.len[0].cpu().tolist() == oc.len.tolist(), f"step {step}: lengths"
        assert st.item() == int(oc.status[0]) != 0  # the full caches overflow at every step
        assert st.item() & bt.BT_DEV_OVERFLOW
        assert_close(out, ref, f"fused step {step} hd={hd} splits={splits}")
        gk, gv = gen.torch_to_bits(cache.k[0]), gen.torch_to_bits(cache.v[0])
        for b in range(B):  # the valid rows are the oracle's, bit for bit; the rest still holds the poison
            n = int(oc.len[b])
            assert np.array_equal(gk[b, :, :n], oc.k[b, :, :n]) and np.array_equal(gv[b, :, :n], oc.v[b, :, :n])
            assert (gk[b, :, n:] == 0x7FC0).all() and (gv[b, :, n:] == 0x7FC0).all()
    # the arrival counters are back at zero: B*H + B int32 at the end of the workspace
    n_cnt = B * H + B
    assert not ws.view(torch.int32)[-n_cnt:].any()


def test_fused_step_new_row_is_what_the_query_sees(bt):
    """A new row whose key dominates must own the output: the fused launch scores the row it is handed,
    not what the cache held at that position."""
    B, H, hd, N, n0 = 2, 2, 64, 200, 131
    for splits in (1, 4):
        cfg = bt.make_config(B, H, hd, 4, 1, N, 1, decode_splits=splits)
        k, v = rnd(320, 1, (B, H, N, hd)), rnd(320, 2, (B, H, N, hd))
        cache = bt.BlockCache(cfg)
        cache.k[0].copy_(to_dev(k))
        cache.v[0].copy_(to_dev(v))
        cache.len[0].fill_(n0)
        q = gen.f32_to_bf16_bits(np.full((B, H, hd), 2.0, np.float32))
        kn = gen.f32_to_bf16_bits(np.full((B, H, 1, hd), 12.0, np.float32))
        vn = gen.f32_to_bf16_bits(np.broadcast_to((np.arange(hd) - 30.0).astype(np.float32), (B, H, 1, hd)).copy())
        out = torch.empty((B, H, hd), dtype=torch.bfloat16, device="cuda")
        bt.bt_block_decode_step(cfg, cache, 0, to_dev(q), to_dev(kn), to_dev(vn), out, bt.alloc_workspace(cfg))
        got = out.double().cpu().numpy()
        assert np.abs(got - (np.arange(hd) - 30.0)).max() < 1e-2
        assert (cache.len[0] == n0 + 1).all()
        assert np.array_equal(gen.torch_to_bits(cache.k[0, :, :, n0]), kn[:, :, 0])
        assert np.array_equal(gen.torch_to_bits(cache.k[0, :, :, :n0]), k[:, :, :n0])  # older rows untouched


def test_fused_step_matches_the_two_separate_calls_at_a_bench_like_shape(bt):
    """Several waves of items per warp (more (b,h) pairs than warps on the GPU), uniform lengths: the
    fused launch and append + attention leave identical caches and lengths and outputs that differ by
    at most the rounding of one row's position in the sum."""
    B, H, hd, N = 160, 16, 64, 96
    cfg = bt.make_config(B, H, hd, 4, 1, N, 2)
    fill = lambda tid, shape: gen.normal_bf16_device(330, tid, shape, device="cuda")
    k, v = fill(0, (2, B, H, N, hd)), fill(1, (2, B, H, N, hd))
    a = bt.BlockCache(cfg, k=k.clone(), v=v.clone())
    b = bt.BlockCache(cfg, k=k.clone(), v=v.clone())
    a.len.fill_(N - 1)
    b.len.fill_(N - 1)
    q, kn, vn = fill(2, (2, B, H, 1, hd)), fill(3, (2, B, H, 1, hd)), fill(4, (2, B, H, 1, hd))
    oa, ob = torch.empty_like(q), torch.empty_like(q)
    ws = bt.alloc_workspace(cfg)
    st = status_word()
    for l in range(2):
        bt.bt_block_decode_step(cfg, a, l, q[l], kn[l], vn[l], oa[l], ws, dev_status=st)
        bt.bt_block_kv_append(cfg, b, l, kn[l], vn[l], dev_status=st)
        bt.bt_block_decode_attn(cfg, b, l, q[l], ob[l], ws, dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    assert torch.equal(a.len, b.len) and (a.len == N).all()
    assert torch.equal(a.k, b.k) and torch.equal(a.v, b.v)
    assert (oa.float() - ob.float()).abs().max().item() <= 4e-3
    sel = [0, 77, 159]
    oc = oracle.Cache(len(sel), H, N, hd)
    oc.k[...], oc.v[...] = gen.torch_to_bits(a.k[1][sel]), gen.torch_to_bits(a.v[1][sel])
    oc.len[...] = N
    assert_close(oa[1][sel][:, :, 0], oracle.block_decode_attn(oc, gen.torch_to_bits(q[1][sel][:, :, 0])), "fused step, layer 1")


def test_fused_step_needs_a_workspace(bt):
    cfg = bt.make_config(2, 2, 64, 4, 1, 64, 1)
    cache = bt.BlockCache(cfg)
    x = torch.zeros((2, 2, 1, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(bt.BtError) as e:
        bt.bt_block_decode_step(cfg, cache, 0, x, x, x, torch.empty_like(x), torch.empty(1, device="cuda"))
    assert "BT_ERR_WORKSPACE" in str(e.value)
    assert (cache.len == 0).all()
