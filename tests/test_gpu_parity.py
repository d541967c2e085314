"""GPU parity: every entry point of the C-ABI library against the CPU oracle on identical
seeded bytes.  Cache contents, lengths and reset positions bit-exact; attention outputs within
|g - r| <= 1e-2 + 2e-2 |r| (and within bf16 rounding of the fp32-accumulated result)."""
import numpy as np
import pytest
import torch

import oracle
from workloads import configs, gen

from util import assert_close, local_kv_split, status_word, to_dev, to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bt():
    import paper_2406_02657_b200 as bt
    assert torch.cuda.is_available()
    return bt


def rnd(seed, tid, shape):
    return gen.normal_bf16_bits(seed, tid, shape)


def fill_block_cache(bt, cfg, cache, layer, kbits, vbits, lens):
    """Write known rows straight into the caller-owned cache tensors (public layout)."""
    cache.k[layer].copy_(to_dev(kbits))
    cache.v[layer].copy_(to_dev(vbits))
    cache.len[layer].copy_(torch.from_numpy(np.asarray(lens, np.int32)).cuda())


def oracle_cache(B, H, cap, hd, kbits, vbits, lens):
    c = oracle.Cache(B, H, cap, hd)
    c.k[...] = kbits
    c.v[...] = vbits
    c.len[...] = lens
    return c


# ------------------------------------------------------------------ config 1: tiny, every entry point

def test_tiny_step_by_step_block_decode_equals_full_recompute(bt):
    w = configs.TINY
    B, H, hd, N = w.batch, w.heads, w.head_dim, w.max_blocks
    cfg = bt.make_config(B, H, hd, w.block_len, w.prefix_len, N, w.n_layers)
    cache = bt.BlockCache(cfg)
    ws = bt.alloc_workspace(cfg)
    st = status_word()
    layer = 1
    q, k, v = (rnd(w.seed, i, (B, H, N, hd)) for i in range(3))
    full = oracle.block_prefill_attn(q, k, v)  # recompute without a cache
    oc = oracle.Cache(B, H, N, hd)
    out = torch.empty((B, H, hd), dtype=torch.bfloat16, device="cuda")
    for t in range(N):
        kt, vt = np.ascontiguousarray(k[:, :, t:t + 1]), np.ascontiguousarray(v[:, :, t:t + 1])
        bt.bt_block_kv_append(cfg, cache, layer, to_dev(kt), to_dev(vt), dev_status=st)
        bt.bt_block_decode_attn(cfg, cache, layer, to_dev(np.ascontiguousarray(q[:, :, t])), out, ws, dev_status=st)
        oracle.kv_append(oc, kt, vt)
        assert_close(out, full[:, :, t], f"decode step {t}")
        assert np.array_equal(cache.len[layer].cpu().numpy(), oc.len)
    assert np.array_equal(gen.torch_to_bits(cache.k[layer]), oc.k)
    assert np.array_equal(gen.torch_to_bits(cache.v[layer]), oc.v)
    assert not cache.k[0].any() and not cache.len[0].any()  # other layer untouched
    assert st.item() == 0


def test_tiny_prefill_packed_and_from_cache(bt):
    w = configs.TINY
    B, H, hd, T = w.batch, w.heads, w.head_dim, w.prompt_blocks
    cfg = bt.make_config(B, H, hd, w.block_len, w.prefix_len, 2 * T, 1)
    q, k, v = (rnd(w.seed + 50, i, (B, H, T, hd)) for i in range(3))
    ref = oracle.block_prefill_attn(q, k, v)
    out = torch.empty((B, H, T, hd), dtype=torch.bfloat16, device="cuda")
    bt.bt_block_prefill_attn(cfg, to_dev(q), to_dev(k), to_dev(v), out)
    assert_close(out, ref, "prefill packed", p_bf16=True)
    # bulk append of the prompt's rows, then prefill reading K,V in place from the cache
    cache = bt.BlockCache(cfg)
    st = status_word()
    bt.bt_block_kv_append(cfg, cache, 0, to_dev(k), to_dev(v), dev_status=st)
    assert (cache.len[0] == T).all() and st.item() == 0
    assert np.array_equal(gen.torch_to_bits(cache.k[0, :, :, :T]), k)
    out2 = torch.empty_like(out)
    bt.bt_block_prefill_attn(cfg, to_dev(q), cache.k[0], cache.v[0], out2, n_blocks=T, kv_seq_stride=2 * T)
    assert torch.equal(out, out2)


@pytest.mark.parametrize("L_B,P,hd,H", [
    (4, 1, 64, 8), (4, 2, 64, 8), (1, 1, 64, 3), (8, 2, 128, 4), (2, 4, 128, 16),
    # prefix length 8 (the longest of the prefix-length ablation): the block start is an 8-row causal step,
    # the steps after it run over 8 .. 8 + L_B - 2 cached rows
    (4, 8, 64, 4), (4, 8, 128, 3), (8, 8, 64, 2), (8, 8, 128, 2), (1, 8, 64, 5),
    # local caches of 7, 8 and 9 rows at both head sizes (the deepest of the pipelined step kernels)
    (8, 1, 128, 4), (6, 2, 128, 4), (6, 1, 128, 2), (8, 1, 64, 5), (6, 2, 64, 16)])
def test_token_decoder_blocks(bt, L_B, P, hd, H):
    """Fused reset + append + local attention over several blocks; lengths, reset positions and
    cache rows bit-exact, outputs within tolerance."""
    B, n_blocks, layer = 5, 3, 1
    cfg = bt.make_config(B, H, hd, L_B, P, 8, 2)
    lc = bt.LocalCache(cfg)
    lc.kv.copy_(to_dev(rnd(77, 1, tuple(lc.kv.shape))))  # stale garbage from "earlier blocks"
    oc = oracle.Cache(B, H, P + L_B, hd)
    st = status_word()
    for t, (reset, n_app, len_after) in enumerate(oracle.token_step_schedule(L_B, P, n_blocks * L_B)):
        q, k, v = (rnd(300 + hd, 10 * t + i, (B, H, n_app, hd)) for i in range(3))
        out = torch.empty((B, H, n_app, hd), dtype=torch.bfloat16, device="cuda")
        bt.bt_token_decode_attn(cfg, lc, layer, to_dev(q), to_dev(k), to_dev(v), out, reset_first=bool(reset),
                                dev_status=st)
        ref = oracle.token_decode_attn(oc, q, k, v, reset_first=bool(reset))
        assert_close(out, ref, f"token step {t}")
        lens = lc.len[layer].cpu().numpy()
        assert np.array_equal(lens, oc.len) and (lens == len_after).all()
        gk, gv = local_kv_split(lc.kv[layer])
        assert np.array_equal(gk[:, :, :len_after], oc.k[:, :, :len_after])
        assert np.array_equal(gv[:, :, :len_after], oc.v[:, :, :len_after])
    assert st.item() == 0 and not lc.len[0].any()


def test_token_masked_reset_attend_only_append_and_overflow(bt):
    B, H, hd, L_B, P = 6, 8, 64, 4, 1
    cfg = bt.make_config(B, H, hd, L_B, P, 8, 1)
    lc = bt.LocalCache(cfg)
    oc = oracle.Cache(B, H, P + L_B, hd)
    st = status_word()
    out = torch.empty((B, H, 1, hd), dtype=torch.bfloat16, device="cuda")
    # two rows through the plain append entry point
    k2, v2 = rnd(41, 1, (B, H, 2, hd)), rnd(41, 2, (B, H, 2, hd))
    bt.bt_local_kv_append(cfg, lc, 0, to_dev(k2), to_dev(v2), dev_status=st)
    oracle.kv_append(oc, k2, v2)
    # attend only
    q = rnd(41, 3, (B, H, 1, hd))
    bt.bt_token_decode_attn(cfg, lc, 0, to_dev(q), None, None, out, dev_status=st)
    assert_close(out, oracle.token_decode_attn(oc, q, None, None), "attend only")
    assert np.array_equal(lc.len[0].cpu().numpy(), oc.len) and st.item() == 0
    # masked reset: sequences 1 and 4 start a new block, the others continue
    mask = np.array([0, 1, 0, 0, 1, 0], np.uint8)
    q, k, v = (rnd(41, 10 + i, (B, H, 1, hd)) for i in range(3))
    bt.bt_token_decode_attn(cfg, lc, 0, to_dev(q), to_dev(k), to_dev(v), out,
                            reset_mask=torch.from_numpy(mask).cuda(), dev_status=st)
    assert_close(out, oracle.token_decode_attn(oc, q, k, v, reset_mask=mask), "masked reset")
    assert lc.len[0].cpu().tolist() == oc.len.tolist() == [3, 1, 3, 3, 1, 3]
    # reset entry point with a mask, then for everyone
    m2 = np.array([1, 0, 0, 0, 0, 0], np.uint8)
    bt.bt_local_kv_reset(cfg, lc, 0, torch.from_numpy(m2).cuda())
    oracle.local_kv_reset(oc, m2)
    assert lc.len[0].cpu().tolist() == oc.len.tolist()
    # run into the capacity: sequences at length 3 overflow after two more rows
    for step in range(3):
        q, k, v = (rnd(41, 20 + 3 * step + i, (B, H, 1, hd)) for i in range(3))
        bt.bt_token_decode_attn(cfg, lc, 0, to_dev(q), to_dev(k), to_dev(v), out, dev_status=st)
        ref = oracle.token_decode_attn(oc, q, k, v)
        assert_close(out, ref, f"overflow step {step}")
        assert lc.len[0].cpu().tolist() == oc.len.tolist()
    assert st.item() == bt.BT_DEV_OVERFLOW == int(oc.status[0])
    gk, gv = local_kv_split(lc.kv[0])
    for b in range(B):
        n = oc.len[b]
        assert np.array_equal(gk[b, :, :n], oc.k[b, :, :n]) and np.array_equal(gv[b, :, :n], oc.v[b, :, :n])
    # empty cache, attend only -> zeros and the EMPTY bit
    bt.bt_local_kv_reset(cfg, lc, 0)
    st.zero_()
    bt.bt_token_decode_attn(cfg, lc, 0, to_dev(q), None, None, out, dev_status=st)
    assert not out.any() and st.item() == bt.BT_DEV_EMPTY


@pytest.mark.parametrize("P,hd", [(2, 64), (4, 64), (2, 128), (4, 128), (8, 64)])
def test_token_masked_reset_with_prefix_steps(bt, P, hd):
    """Ragged batch (prompts whose partial last block was prefilled for some sequences while others
    start a block): one call in which the sequences named by reset_mask drop their cache and take the P
    prefix rows as a causal P-query step, while the others append the same number of rows to what
    they hold - or are skipped, untouched and flagged, when those rows do not fit."""
    B, H, L_B = 7, 4, 4
    cap = P + L_B
    cfg = bt.make_config(B, H, hd, L_B, P, 8, 2)
    layer = 1
    lc = bt.LocalCache(cfg)
    lc.kv.copy_(to_dev(rnd(51, 1, tuple(lc.kv.shape))))
    oc = oracle.Cache(B, H, cap, hd)
    st = status_word()
    # uneven starting lengths through single-row steps with a mask that keeps some sequences empty
    lens0 = [0, 1, 2, 3, cap - P, cap - P + 1, cap]   # the last but one has no room for P more rows
    for b, n in enumerate(lens0):
        if n:
            kb, vb = rnd(52, 10 + b, (1, H, n, hd)), rnd(52, 20 + b, (1, H, n, hd))
            oc.k[b, :, :n], oc.v[b, :, :n] = kb[0], vb[0]
            oc.len[b] = n
    kv = np.zeros(tuple(lc.kv[layer].shape), np.uint16)
    kv[:, :, :, 0], kv[:, :, :, 1] = oc.k, oc.v
    lc.kv[layer].copy_(to_dev(kv))
    lc.len[layer].copy_(torch.from_numpy(oc.len.copy()).cuda())
    for step, mask in enumerate(([1, 0, 0, 1, 0, 0, 1], [0, 1, 0, 0, 1, 0, 0])):
        mask = np.array(mask, np.uint8)
        q, k, v = (rnd(53 + hd, 10 * step + i, (B, H, P, hd)) for i in range(3))
        out = torch.full((B, H, P, hd), 3.0, dtype=torch.bfloat16, device="cuda")
        before = gen.torch_to_bits(lc.kv[layer])
        bt.bt_token_decode_attn(cfg, lc, layer, to_dev(q), to_dev(k), to_dev(v), out,
                                reset_mask=torch.from_numpy(mask).cuda(), dev_status=st)
        len_before = oc.len.copy()
        ref = oracle.token_decode_attn(oc, q, k, v, reset_mask=mask)
        assert_close(out, ref, f"masked reset, {P} rows, step {step}")
        assert lc.len[layer].cpu().tolist() == oc.len.tolist()
        gk, gv = local_kv_split(lc.kv[layer])
        after = gen.torch_to_bits(lc.kv[layer])
        for b in range(B):
            n = oc.len[b]
            assert np.array_equal(gk[b, :, :n], oc.k[b, :, :n]) and np.array_equal(gv[b, :, :n], oc.v[b, :, :n])
            skipped = not mask[b] and len_before[b] + P > cap
            if skipped:  # no room: nothing written, zeros out
                assert np.array_equal(after[b], before[b]) and not out[b].any() and oc.len[b] == len_before[b]
    assert st.item() == bt.BT_DEV_OVERFLOW == int(oc.status[0])
    assert not lc.len[0].any()


# ------------------------------------------------------------------ block decode: tiles, tails, splits

@pytest.mark.parametrize("hd", [64, 128])
@pytest.mark.parametrize("splits", [1, 2, 3, 7])
def test_block_decode_ragged_lengths_poison_and_splits(bt, hd, splits):
    B, H, N = 7, 3, 517  # several 128-row CTA tiles plus a ragged tail
    cfg = bt.make_config(B, H, hd, 4, 1, N, 1, decode_splits=splits)
    lens = np.array([517, 1, 128, 129, 0, 333, 64], np.int32)
    k, v = rnd(60 + hd, 1, (B, H, N, hd)), rnd(60 + hd, 2, (B, H, N, hd))
    q = rnd(60 + hd, 0, (B, H, hd))
    oc = oracle_cache(B, H, N, hd, k, v, lens)
    ref = oracle.block_decode_attn(oc, q)
    kp, vp = k.copy(), v.copy()
    for b in range(B):  # anything past the length must never be read: poison it with NaN
        kp[b, :, lens[b]:] = 0x7FC0
        vp[b, :, lens[b]:] = 0x7FC0
    cache = bt.BlockCache(cfg)
    fill_block_cache(bt, cfg, cache, 0, kp, vp, lens)
    ws = bt.alloc_workspace(cfg)
    ws.fill_(float("nan"))  # the partial results need no initialisation, only the arrival counters do
    bt.bt_workspace_init(cfg, ws)
    st = status_word()
    out = torch.full((B, H, hd), 7.0, dtype=torch.bfloat16, device="cuda")
    bt.bt_block_decode_attn(cfg, cache, 0, to_dev(q), out, ws, dev_status=st)
    assert_close(out, ref, f"ragged decode hd={hd} splits={splits}")
    assert not out[4].any() and st.item() == bt.BT_DEV_EMPTY == int(oc.status[0])


@pytest.mark.parametrize("splits", [1, 4])
def test_block_decode_spike_rows_at_every_boundary(bt, splits):
    """With N(0,1) data one row moves the output by ~1/n, below the tolerance.  A planted row whose
    key dominates flips the output to its value, so including or excluding it is visible."""
    B, H, hd, N, n = 1, 1, 64, 600, 515
    cfg = bt.make_config(B, H, hd, 4, 1, N, 1, decode_splits=splits)
    k, v = rnd(70, 1, (B, H, N, hd)), rnd(70, 2, (B, H, N, hd))
    q = gen.f32_to_bf16_bits(np.full((B, H, hd), 2.0, np.float32))
    spike_k = gen.f32_to_bf16_bits(np.full(hd, 12.0, np.float32))
    spike_v = gen.f32_to_bf16_bits((np.arange(hd) - 30.0).astype(np.float32))
    cache = bt.BlockCache(cfg)
    ws = bt.alloc_workspace(cfg)
    out = torch.empty((B, H, hd), dtype=torch.bfloat16, device="cuda")
    per = -(-n // splits)
    rows = sorted({0, 1, 3, 4, 31, 32, 127, 128, 129, 255, 256, 511, 512, n - 2, n - 1, n, n + 1,
                   per - 1, per, per + 1, 2 * per - 1, 2 * per} & set(range(N)))
    for row in rows:
        kk, vv = k.copy(), v.copy()
        kk[0, 0, row], vv[0, 0, row] = spike_k, spike_v
        fill_block_cache(bt, cfg, cache, 0, kk, vv, [n])
        bt.bt_block_decode_attn(cfg, cache, 0, to_dev(q), out, ws)
        ref = oracle.block_decode_attn(oracle_cache(B, H, N, hd, kk, vv, [n]), q)
        assert_close(out, ref, f"spike at row {row}")
        got = to_f64(out)[0, 0]
        if row < n:
            assert np.abs(got - gen.bf16_bits_to_f32(spike_v)).max() < 1e-2, f"row {row} should dominate"
        else:
            assert np.abs(got - gen.bf16_bits_to_f32(spike_v)).max() > 10.0, f"row {row} lies past the length and must be invisible"


def test_block_append_overflow_is_skipped_and_flagged(bt):
    B, H, hd, N = 3, 2, 64, 4
    cfg = bt.make_config(B, H, hd, 4, 1, N, 1)
    cache = bt.BlockCache(cfg)
    cache.len[0].copy_(torch.tensor([3, 4, 0], dtype=torch.int32))
    oc = oracle.Cache(B, H, N, hd)
    oc.len[...] = [3, 4, 0]
    st = status_word()
    k, v = rnd(80, 1, (B, H, 1, hd)), rnd(80, 2, (B, H, 1, hd))
    bt.bt_block_kv_append(cfg, cache, 0, to_dev(k), to_dev(v), dev_status=st)
    oracle.kv_append(oc, k, v)
    assert cache.len[0].cpu().tolist() == oc.len.tolist() == [4, 4, 1]
    assert st.item() == bt.BT_DEV_OVERFLOW == int(oc.status[0])
    assert np.array_equal(gen.torch_to_bits(cache.k[0]), oc.k) and np.array_equal(gen.torch_to_bits(cache.v[0]), oc.v)
    # bulk path (two launches): 3 more rows fit only for the last sequence
    k3, v3 = rnd(80, 3, (B, H, 3, hd)), rnd(80, 4, (B, H, 3, hd))
    big = bt.make_config(B, 16, 128, 4, 1, 600, 1)
    cache2 = bt.BlockCache(big)
    cache2.len[0].copy_(torch.tensor([100, 599, 0], dtype=torch.int32))
    oc2 = oracle.Cache(B, 16, 600, 128)
    oc2.len[...] = [100, 599, 0]
    kb, vb = rnd(80, 5, (B, 16, 300, 128)), rnd(80, 6, (B, 16, 300, 128))
    st.zero_()
    bt.bt_block_kv_append(big, cache2, 0, to_dev(kb), to_dev(vb), dev_status=st)
    oracle.kv_append(oc2, kb, vb)
    assert cache2.len[0].cpu().tolist() == oc2.len.tolist() == [400, 599, 300]
    assert st.item() == bt.BT_DEV_OVERFLOW
    assert np.array_equal(gen.torch_to_bits(cache2.k[0]), oc2.k) and np.array_equal(gen.torch_to_bits(cache2.v[0]), oc2.v)
    del k3, v3


def test_l_b_one_block_decoder_is_vanilla_causal_attention(bt):
    """At L_B = 1 every token is a block: cached block decode over a token-level cache reproduces
    token-level causal attention (library routine in float64)."""
    B, H, hd, L = 2, 4, 64, 48
    cfg = bt.make_config(B, H, hd, 1, 1, L, 1)
    q, k, v = (rnd(90, i, (B, H, L, hd)) for i in range(3))
    f = lambda b: torch.from_numpy(gen.bf16_bits_to_f32(b).astype(np.float64))
    ref = torch.nn.functional.scaled_dot_product_attention(f(q), f(k), f(v), is_causal=True).numpy()
    cache = bt.BlockCache(cfg)
    ws = bt.alloc_workspace(cfg)
    out = torch.empty((B, H, hd), dtype=torch.bfloat16, device="cuda")
    for t in range(L):
        bt.bt_block_kv_append(cfg, cache, 0, to_dev(np.ascontiguousarray(k[:, :, t:t + 1])),
                              to_dev(np.ascontiguousarray(v[:, :, t:t + 1])))
        bt.bt_block_decode_attn(cfg, cache, 0, to_dev(np.ascontiguousarray(q[:, :, t])), out, ws)
        assert_close(out, ref[:, :, t], f"L_B=1 step {t}")


# ------------------------------------------------------------------ prefill: tiles, diagonal, strides

@pytest.mark.parametrize("plain", [0, 1])
@pytest.mark.parametrize("hd,T,B,H", [(128, 128, 2, 2), (128, 300, 1, 3), (64, 257, 2, 2), (128, 512, 1, 2), (64, 33, 3, 1),
                                      (128, 1, 1, 1), (64, 640, 1, 2), (128, 1024, 1, 1), (128, 2048, 1, 2), (64, 2048, 1, 1)])
def test_block_prefill_shapes(bt, hd, T, B, H, plain):
    cfg = bt.make_config(B, H, hd, 4, 1, T, 1, prefill_plain=plain)
    q, k, v = (rnd(100 + T, i, (B, H, T, hd)) for i in range(3))
    out = torch.full((B, H, T, hd), 9.0, dtype=torch.bfloat16, device="cuda")
    st = status_word()
    bt.bt_block_prefill_attn(cfg, to_dev(q), to_dev(k), to_dev(v), out, dev_status=st)
    assert st.item() == 0
    assert_close(out, oracle.block_prefill_attn(q, k, v), f"prefill T={T} hd={hd} plain={plain}", p_bf16=not plain)


@pytest.mark.parametrize("plain", [0, 1])
def test_block_prefill_reads_cache_in_place_and_ignores_rows_past_T(bt, plain):
    """K, V taken in place from a block cache (stride N_max > T); rows past T hold NaN and must not matter."""
    B, H, hd, T, N = 2, 3, 128, 200, 320
    cfg = bt.make_config(B, H, hd, 4, 1, N, 1, prefill_plain=plain)
    q = rnd(120, 0, (B, H, T, hd))
    k, v = rnd(120, 1, (B, H, N, hd)), rnd(120, 2, (B, H, N, hd))
    ref = oracle.block_prefill_attn(q, k, v, kv_seq_stride=N)
    k[:, :, T:] = 0x7FC0
    v[:, :, T:] = 0x7FC0
    out = torch.empty((B, H, T, hd), dtype=torch.bfloat16, device="cuda")
    st = status_word()
    bt.bt_block_prefill_attn(cfg, to_dev(q), to_dev(k), to_dev(v), out, n_blocks=T, kv_seq_stride=N, dev_status=st)
    assert st.item() == 0
    assert_close(out, ref, f"prefill from cache plain={plain}", p_bf16=not plain)


@pytest.mark.parametrize("plain", [0, 1])
def test_block_prefill_spikes_on_and_next_to_the_diagonal(bt, plain):
    """A dominant key at block j must take over every query t >= j and no query t < j."""
    B, H, hd, T = 1, 1, 128, 384
    cfg = bt.make_config(B, H, hd, 4, 1, T, 1, prefill_plain=plain)
    q = gen.f32_to_bf16_bits(np.full((B, H, T, hd), 1.5, np.float32))
    k, v = rnd(110, 1, (B, H, T, hd)), rnd(110, 2, (B, H, T, hd))
    spike_v = gen.f32_to_bf16_bits((np.arange(hd) - 60.0).astype(np.float32))
    out = torch.empty((B, H, T, hd), dtype=torch.bfloat16, device="cuda")
    for j in (0, 1, 63, 64, 127, 128, 129, 255, 256, 383):
        kk, vv = k.copy(), v.copy()
        kk[0, 0, j] = gen.f32_to_bf16_bits(np.full(hd, 8.0, np.float32))
        vv[0, 0, j] = spike_v
        bt.bt_block_prefill_attn(cfg, to_dev(q), to_dev(kk), to_dev(vv), out)
        assert_close(out, oracle.block_prefill_attn(q, kk, vv), f"diagonal spike at {j}", p_bf16=not plain)
        got = to_f64(out)[0, 0]
        hit = np.abs(got - gen.bf16_bits_to_f32(spike_v)).max(axis=1) < 0.3
        assert hit[j:].all() and not hit[:j].any(), f"causal boundary wrong around block {j}"


def test_block_prefill_late_large_keys_force_a_rescale(bt):
    """Keys that grow along the sequence push the running row maximum up by far more than the
    lazy-rescale threshold in every later tile, so the accumulator rescale path is exercised."""
    B, H, hd, T = 1, 2, 128, 512
    cfg = bt.make_config(B, H, hd, 4, 1, T, 1)
    q = gen.f32_to_bf16_bits(np.abs(gen.bf16_bits_to_f32(rnd(130, 0, (B, H, T, hd)))))
    ramp = (1.0 + np.arange(T, dtype=np.float32) / 16.0)[None, None, :, None]
    k = gen.f32_to_bf16_bits(np.abs(gen.bf16_bits_to_f32(rnd(130, 1, (B, H, T, hd)))) * ramp)
    v = rnd(130, 2, (B, H, T, hd))
    out = torch.empty((B, H, T, hd), dtype=torch.bfloat16, device="cuda")
    st = status_word()
    bt.bt_block_prefill_attn(cfg, to_dev(q), to_dev(k), to_dev(v), out, dev_status=st)
    assert st.item() == 0
    assert_close(out, oracle.block_prefill_attn(q, k, v), "prefill with growing keys", p_bf16=True)
