"""Out-of-bounds checks without a memory checker: every buffer handed to the library sits between
guard regions filled with a known pattern, lengths are drawn at random (including empty and full
caches), and after each call the guards and every byte outside the rows the call may write must be
unchanged."""
import numpy as np
import pytest
import torch

import oracle
from workloads import gen

from util import assert_close, status_word, to_dev

pytestmark = pytest.mark.gpu

GUARD = 4096  # bytes on each side
PATTERN = 0x5A


@pytest.fixture(scope="module")
def bt():
    import paper_2406_02657_b200 as bt
    assert torch.cuda.is_available()
    return bt


class Guarded:
    """A device tensor of `shape` carved out of a larger byte buffer with guard bytes on both sides."""

    def __init__(self, shape, dtype):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        pad = (-n) % 256
        self.raw = torch.full((GUARD + n + pad + GUARD,), PATTERN, dtype=torch.uint8, device="cuda")
        self.t = self.raw[GUARD:GUARD + n].view(dtype).view(shape)
        self.n = n

    def guards_intact(self):
        return bool((self.raw[:GUARD] == PATTERN).all()) and bool((self.raw[GUARD + self.n:] == PATTERN).all())


def test_block_path_touches_nothing_outside_its_rows(bt):
    rng = np.random.default_rng(7)
    B, H, hd, N = 37, 5, 64, 96
    for trial, (splits, fused) in enumerate(((0, False), (1, False), (3, False), (0, True), (1, True), (3, True))):
        cfg = bt.make_config(B, H, hd, 4, 1, N, 1, decode_splits=splits)
        k, v = Guarded((1, B, H, N, hd), torch.bfloat16), Guarded((1, B, H, N, hd), torch.bfloat16)
        ln = Guarded((1, B), torch.int32)
        q, kn, vn, out = (Guarded((B, H, 1, hd), torch.bfloat16) for _ in range(4))
        ws = Guarded((max(bt.bt_workspace_bytes(cfg), 4) // 4,), torch.float32)
        bt.bt_workspace_init(cfg, ws.t)  # zeroes the arrival counters; the partial results keep the pattern
        lens = rng.integers(0, N + 1, B).astype(np.int32)
        lens[0], lens[1] = 0, N  # an empty cache (append fits) and a full one (append must be refused)
        kb, vb = gen.normal_bf16_bits(300 + trial, 1, (B, H, N, hd)), gen.normal_bf16_bits(300 + trial, 2, (B, H, N, hd))
        k.t[0].copy_(to_dev(kb)); v.t[0].copy_(to_dev(vb)); ln.t[0].copy_(torch.from_numpy(lens).cuda())
        qb, knb, vnb = (gen.normal_bf16_bits(300 + trial, 3 + i, (B, H, 1, hd)) for i in range(3))
        q.t.copy_(to_dev(qb)); kn.t.copy_(to_dev(knb)); vn.t.copy_(to_dev(vnb))
        cache = bt.BlockCache(cfg, k=k.t, v=v.t, length=ln.t)
        st = status_word()
        if fused:
            bt.bt_block_decode_step(cfg, cache, 0, q.t[:, :, 0], kn.t, vn.t, out.t[:, :, 0], ws.t, dev_status=st)
        else:
            bt.bt_block_kv_append(cfg, cache, 0, kn.t, vn.t, n_new=1, dev_status=st)
            bt.bt_block_decode_attn(cfg, cache, 0, q.t[:, :, 0], out.t[:, :, 0], ws.t, dev_status=st)
        torch.cuda.synchronize()
        oc = oracle.Cache(B, H, N, hd)
        oc.k[...], oc.v[...], oc.len[...] = kb, vb, lens
        oracle.kv_append(oc, knb, vnb)
        ref = oracle.block_decode_attn(oc, np.ascontiguousarray(qb[:, :, 0]))
        for g in (k, v, ln, q, kn, vn, out, ws):
            assert g.guards_intact()
        # the cache differs from before only in the appended rows; lengths advanced except the full one
        assert np.array_equal(gen.torch_to_bits(k.t[0]), oc.k) and np.array_equal(gen.torch_to_bits(v.t[0]), oc.v)
        assert np.array_equal(ln.t[0].cpu().numpy(), oc.len) and oc.len[1] == N and oc.len[0] == 1
        assert np.array_equal(gen.torch_to_bits(q.t), qb) and np.array_equal(gen.torch_to_bits(kn.t), knb)
        assert_close(out.t[:, :, 0], ref, f"guarded decode, splits {splits}, fused {fused}")
        assert st.item() == bt.BT_DEV_OVERFLOW == int(oc.status[0])


@pytest.mark.parametrize("hd", [64, 128])
def test_multi_query_step_touches_nothing_outside_its_rows(bt, hd):
    rng = np.random.default_rng(11)
    B, H, N, m = 23, 5, 80, 4
    cfg = bt.make_config(B, H, hd, m, 1, N, 1)
    k, v = Guarded((1, B, H, N, hd), torch.bfloat16), Guarded((1, B, H, N, hd), torch.bfloat16)
    ln = Guarded((1, B), torch.int32)
    q, kn, vn, out = (Guarded((B, H, m, hd), torch.bfloat16) for _ in range(4))
    ws = Guarded((max(bt.bt_workspace_bytes(cfg), 4) // 4,), torch.float32)
    bt.bt_workspace_init(cfg, ws.t)
    lens = rng.integers(0, N + 1, B).astype(np.int32)
    lens[0], lens[1], lens[2] = 0, N, N - m + 1   # empty; full; one row short of room for the m rows
    kb, vb = gen.normal_bf16_bits(500 + hd, 1, (B, H, N, hd)), gen.normal_bf16_bits(500 + hd, 2, (B, H, N, hd))
    k.t[0].copy_(to_dev(kb)); v.t[0].copy_(to_dev(vb)); ln.t[0].copy_(torch.from_numpy(lens).cuda())
    qb, knb, vnb = (gen.normal_bf16_bits(500 + hd, 3 + i, (B, H, m, hd)) for i in range(3))
    q.t.copy_(to_dev(qb)); kn.t.copy_(to_dev(knb)); vn.t.copy_(to_dev(vnb))
    cache = bt.BlockCache(cfg, k=k.t, v=v.t, length=ln.t)
    st = status_word()
    bt.bt_block_decode_step_multi(cfg, cache, 0, q.t, kn.t, vn.t, out.t, ws.t, dev_status=st)
    torch.cuda.synchronize()
    oc = oracle.Cache(B, H, N, hd)
    oc.k[...], oc.v[...], oc.len[...] = kb, vb, lens
    ref = oracle.block_decode_step_multi(oc, qb, knb, vnb)
    for g in (k, v, ln, q, kn, vn, out, ws):
        assert g.guards_intact()
    # the cache differs from before only in the appended rows; lengths advanced except where there was no room
    assert np.array_equal(gen.torch_to_bits(k.t[0]), oc.k) and np.array_equal(gen.torch_to_bits(v.t[0]), oc.v)
    assert np.array_equal(ln.t[0].cpu().numpy(), oc.len) and oc.len[1] == N and oc.len[2] == N - m + 1 and oc.len[0] == m
    assert np.array_equal(gen.torch_to_bits(q.t), qb) and np.array_equal(gen.torch_to_bits(kn.t), knb)
    assert_close(out.t, ref, f"guarded multi-query step hd={hd}", p_bf16=True)
    assert st.item() == bt.BT_DEV_OVERFLOW == int(oc.status[0])


def test_token_step_touches_nothing_outside_its_rows(bt):
    rng = np.random.default_rng(11)
    B, H, hd, L_B, P = 53, 16, 64, 4, 1
    cap = P + L_B
    cfg = bt.make_config(B, H, hd, L_B, P, 8, 1)
    kv = Guarded((1, B, H, cap, 2, hd), torch.bfloat16)
    ln = Guarded((1, B), torch.int32)
    q, kn, vn, out = (Guarded((B, H, 1, hd), torch.bfloat16) for _ in range(4))
    lc = bt.LocalCache(cfg)
    lc.kv, lc.len = kv.t, ln.t
    lc.c = bt.binding.bt_local_cache(kv.t.data_ptr(), ln.t.data_ptr())
    lens = rng.integers(0, cap + 1, B).astype(np.int32)  # includes full caches: the step must skip those
    lens[0], lens[1] = 0, cap
    kb, vb = gen.normal_bf16_bits(310, 1, (B, H, cap, hd)), gen.normal_bf16_bits(310, 2, (B, H, cap, hd))
    both = np.stack([kb, vb], axis=3)  # [B,H,cap,2,hd]
    kv.t[0].copy_(to_dev(both)); ln.t[0].copy_(torch.from_numpy(lens).cuda())
    qb, knb, vnb = (gen.normal_bf16_bits(310, 3 + i, (B, H, 1, hd)) for i in range(3))
    q.t.copy_(to_dev(qb)); kn.t.copy_(to_dev(knb)); vn.t.copy_(to_dev(vnb))
    st = status_word()
    bt.bt_token_decode_attn(cfg, lc, 0, q.t, kn.t, vn.t, out.t, n_q=1, reset_first=False, dev_status=st)
    torch.cuda.synchronize()
    oc = oracle.Cache(B, H, cap, hd)
    oc.k[...], oc.v[...], oc.len[...] = kb, vb, lens
    ref = oracle.token_decode_attn(oc, qb, knb, vnb, reset_first=False)
    for g in (kv, ln, q, kn, vn, out):
        assert g.guards_intact()
    got = gen.torch_to_bits(kv.t[0])
    assert np.array_equal(got[:, :, :, 0], oc.k) and np.array_equal(got[:, :, :, 1], oc.v)
    assert np.array_equal(ln.t[0].cpu().numpy(), oc.len)
    assert_close(out.t, ref, "guarded token step")
    assert st.item() == bt.BT_DEV_OVERFLOW == int(oc.status[0])


def test_prefill_touches_nothing_outside_its_output(bt):
    B, H, hd, T = 2, 3, 128, 200  # T not a multiple of the 128-row tiles: the last tile's store is clipped
    cfg = bt.make_config(B, H, hd, 4, 1, T, 1)
    q, k, v, out = (Guarded((B, H, T, hd), torch.bfloat16) for _ in range(4))
    qb, kb, vb = (gen.normal_bf16_bits(320, i, (B, H, T, hd)) for i in range(3))
    q.t.copy_(to_dev(qb)); k.t.copy_(to_dev(kb)); v.t.copy_(to_dev(vb))
    st = status_word()
    bt.bt_block_prefill_attn(cfg, q.t, k.t, v.t, out.t, dev_status=st)
    torch.cuda.synchronize()
    for g in (q, k, v, out):
        assert g.guards_intact()
    assert np.array_equal(gen.torch_to_bits(k.t), kb) and np.array_equal(gen.torch_to_bits(v.t), vb)
    assert_close(out.t, oracle.block_prefill_attn(qb, kb, vb), "guarded prefill", p_bf16=True)
    assert st.item() == 0
