"""GPU parity of the linear maps either side of the attention path: the prefix projection and the QKV
projection whose epilogue writes K and V into the caches.  Where the arithmetic is exact (identity and
small-integer weights) q, the cache rows and everything around them are compared bit for bit; with
random weights the values are compared with the oracle's float64 product (the cache rows with that
product rounded to bf16) within fp32-accumulation tolerance, and rows outside the appended window,
lengths and status bits exactly."""
import numpy as np
import pytest
import torch

import oracle
from workloads import gen

from util import assert_close, assert_close_proj, local_kv_split, status_word, to_dev, to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bt():
    import paper_2406_02657_b200 as bt
    assert torch.cuda.is_available()
    return bt


def rnd(seed, tid, shape):
    return gen.normal_bf16_bits(seed, tid, shape)


def widen(b):
    return gen.bf16_bits_to_f32(b).astype(np.float64)


def bits(x):
    return gen.f32_to_bf16_bits(np.asarray(x, np.float32))


def unit_rows(seed, tid, shape):
    """Inputs of variance 1/D, so that the projected q and k have unit variance like the N(0,1) tensors the
    attention tests use (larger ones make the softmax so peaked that one bf16 step in q or k moves the output
    by more than the attention tolerance - a property of the inputs, not of either implementation)."""
    return bits(widen(rnd(seed, tid, shape)) / np.sqrt(shape[-1]))


# ------------------------------------------------------------------ prefix projection

@pytest.mark.parametrize("B,H,hd,P,with_bias", [(5, 2, 64, 1, True), (300, 16, 64, 2, False), (131, 4, 128, 4, True),
                                                (6400, 3, 64, 3, True), (260, 16, 64, 8, True)])
def test_prefix_projection(bt, B, H, hd, P, with_bias):
    D = H * hd
    cfg = bt.make_config(B, H, hd, 4, P, 8, 1)
    ctx, W = rnd(700 + P, 0, (B, D)), rnd(700 + P, 1, (P * D, D))
    bias = rnd(700 + P, 2, (P * D,)) if with_bias else None
    out = torch.full((B, P, D), 9.0, dtype=torch.bfloat16, device="cuda")
    st = status_word()
    bt.bt_prefix_project(cfg, to_dev(ctx), to_dev(W), None if bias is None else to_dev(bias), out, dev_status=st)
    rows = np.unique(np.concatenate([np.arange(min(B, 40)), np.arange(max(0, B - 40), B), [B // 2]]))
    ref = oracle.prefix_project(np.ascontiguousarray(ctx[rows]), W, bias, P)
    assert_close_proj(out[torch.from_numpy(rows).cuda()], ref, f"prefix projection B={B} D={D} P={P}")
    assert st.item() == 0


def test_prefix_projection_with_selector_weights_is_exact(bt):
    """Prefix token 0 = the context embedding, token 1 = its mirror image times -2: exact in any precision."""
    B, H, hd, P = 37, 2, 64, 2
    D = H * hd
    cfg = bt.make_config(B, H, hd, 4, P, 8, 1)
    ctx = rnd(710, 0, (B, D))
    W = np.zeros((P * D, D))
    W[:D] = np.eye(D)
    W[D:] = -2.0 * np.eye(D)[::-1]
    out = torch.empty((B, P, D), dtype=torch.bfloat16, device="cuda")
    bt.bt_prefix_project(cfg, to_dev(ctx), to_dev(bits(W)), None, out)
    got = gen.torch_to_bits(out)
    assert np.array_equal(got[:, 0], ctx) and np.array_equal(got[:, 1], bits(-2.0 * widen(ctx)[:, ::-1]))
    assert np.array_equal(to_f64(out), oracle.prefix_project(ctx, bits(W), None, P))


# ------------------------------------------------------------------ QKV projection into the block cache

def _block_setup(bt, seed, B, H, hd, N, lens, layers=2, layer=1):
    cfg = bt.make_config(B, H, hd, 4, 1, N, layers)
    cache = bt.BlockCache(cfg)
    k0, v0 = rnd(seed, 1, (B, H, N, hd)), rnd(seed, 2, (B, H, N, hd))
    cache.k[layer].copy_(to_dev(k0))
    cache.v[layer].copy_(to_dev(v0))
    cache.len[layer].copy_(torch.from_numpy(np.asarray(lens, np.int32)).cuda())
    oc = oracle.Cache(B, H, N, hd)
    oc.k[...], oc.v[...], oc.len[...] = k0, v0, lens
    return cfg, cache, oc


@pytest.mark.parametrize("hd,n", [(64, 1), (128, 1), (64, 3)])
def test_block_qkv_identity_weights_cache_the_input_bit_for_bit(bt, hd, n):
    B, H, N, layer = 9, 3, 40, 1
    D = H * hd
    lens = [0, 1, 39, 40, 17, 40 - n, 40 - n + 1 if n > 1 else 5, 8, 33]
    cfg, cache, oc = _block_setup(bt, 720 + hd, B, H, hd, N, lens)
    x = rnd(720 + hd, 3, (B, n, D))
    W = bits(np.concatenate([np.eye(D), 2 * np.eye(D), -np.eye(D)]))
    q = torch.full((B, H, n, hd), 5.0, dtype=torch.bfloat16, device="cuda")
    st = status_word()
    bt.bt_block_qkv_project_append(cfg, cache, layer, to_dev(x), to_dev(W), None, q, dev_status=st)
    q_ref = oracle.qkv_project_append(oc, x, W)
    assert np.array_equal(to_f64(q), q_ref)                               # exact arithmetic: bit for bit
    assert np.array_equal(gen.torch_to_bits(cache.k[layer]), oc.k) and np.array_equal(gen.torch_to_bits(cache.v[layer]), oc.v)
    assert cache.len[layer].cpu().tolist() == oc.len.tolist()
    assert st.item() == int(oc.status[0]) == bt.BT_DEV_OVERFLOW
    assert not cache.k[0].any() and not cache.len[0].any()               # the other layer is untouched


@pytest.mark.parametrize("B,H,hd,n,with_bias", [(133, 16, 64, 1, True), (70, 16, 128, 1, False), (40, 4, 64, 5, True),
                                                (2100, 3, 64, 3, True)])
def test_block_qkv_random_weights(bt, B, H, hd, n, with_bias):
    N, layer = 24, 0
    D = H * hd
    rng = np.random.default_rng(B)
    lens = rng.integers(0, N - n + 1, B).astype(np.int32)
    lens[:3] = [0, N - n, N - n + 1 if n <= N else N]                     # empty, exactly fitting, one row short
    cfg, cache, oc = _block_setup(bt, 730 + B, B, H, hd, N, lens, layers=1, layer=0)
    before_k, before_v = oc.k.copy(), oc.v.copy()
    x, W = rnd(730 + B, 3, (B, n, D)), rnd(730 + B, 4, (3 * D, D))
    bias = rnd(730 + B, 5, (3 * D,)) if with_bias else None
    q = torch.empty((B, H, n, hd), dtype=torch.bfloat16, device="cuda")
    st = status_word()
    bt.bt_block_qkv_project_append(cfg, cache, layer, to_dev(x), to_dev(W), None if bias is None else to_dev(bias), q, dev_status=st)
    q_ref = oracle.qkv_project_append(oc, x, W, bias)
    assert_close_proj(q, q_ref, "q of the block QKV projection")
    assert cache.len[layer].cpu().tolist() == oc.len.tolist() and st.item() == int(oc.status[0]) == bt.BT_DEV_OVERFLOW
    gk, gv = gen.torch_to_bits(cache.k[layer]), gen.torch_to_bits(cache.v[layer])
    for b in range(B):
        l = int(lens[b])
        if oc.len[b] == l:   # no room: nothing may have changed
            assert np.array_equal(gk[b], before_k[b]) and np.array_equal(gv[b], before_v[b])
            continue
        # outside the appended window: bit for bit what was there
        assert np.array_equal(gk[b, :, :l], before_k[b, :, :l]) and np.array_equal(gk[b, :, l + n:], before_k[b, :, l + n:])
        assert np.array_equal(gv[b, :, :l], before_v[b, :, :l]) and np.array_equal(gv[b, :, l + n:], before_v[b, :, l + n:])
    win = np.array([[l + i for i in range(n)] for l in lens])             # [B, n] rows of the window
    take = lambda a: np.stack([a[b][:, win[b] % N] for b in range(B)])
    ok = oc.len != lens
    for got, want, what in ((gk, oc.k, "K"), (gv, oc.v, "V")):
        g, r = widen(take(got))[ok], widen(take(want))[ok]
        err = np.abs(g - r)
        assert (err <= 2e-3 + 8e-3 * np.abs(r)).all(), f"{what} rows: max err {err.max():.3e}"   # within one bf16 step of the rounded float64 product
        assert (take(got)[ok] == take(want)[ok]).mean() > 0.97                                    # and nearly always the same bits


# ------------------------------------------------------------------ QKV projection into the local cache, then attention

@pytest.mark.parametrize("hd,P", [(64, 1), (64, 2), (128, 4)])
def test_local_qkv_projection_then_attend_only_over_two_blocks(bt, hd, P):
    """The token decoder with the projections in (section 2.4): at a block start the P prefix embeddings are
    projected (reset, rows 0..P-1 cached) and attended causally; every later token is projected, cached and
    attended.  Lengths and reset positions exact, outputs against the oracle's own projected cache."""
    B, H, L_B, layer = 37, 4, 4, 1
    D = H * hd
    cfg = bt.make_config(B, H, hd, L_B, P, 8, 2)
    lc = bt.LocalCache(cfg)
    lc.kv.copy_(to_dev(rnd(740, 9, tuple(lc.kv.shape))))
    oc = oracle.Cache(B, H, P + L_B, hd)
    W, bias = rnd(740 + hd, 4, (3 * D, D)), rnd(740 + hd, 5, (3 * D,))
    Wd, bd = to_dev(W), to_dev(bias)
    st = status_word()
    for t, (reset, n, len_after) in enumerate(oracle.token_step_schedule(L_B, P, 2 * L_B)):
        x = unit_rows(741 + hd, t, (B, n, D))
        q = torch.empty((B, H, n, hd), dtype=torch.bfloat16, device="cuda")
        out = torch.empty((B, H, n, hd), dtype=torch.bfloat16, device="cuda")
        bt.bt_local_qkv_project_append(cfg, lc, layer, to_dev(x), Wd, bd, q, reset_first=bool(reset), dev_status=st)
        bt.bt_token_decode_attn(cfg, lc, layer, q, None, None, out, n_q=n, dev_status=st)
        q_ref = oracle.qkv_project_append(oc, x, W, bias, reset_first=bool(reset))
        assert_close_proj(q, q_ref, f"q at token step {t}")
        ref = oracle.token_decode_attn(oc, oracle.round_to_bf16(q_ref), None, None)
        assert_close(out, ref, f"attention after projection, step {t}", p_bf16=True)
        lens = lc.len[layer].cpu().numpy()
        assert np.array_equal(lens, oc.len) and (lens == len_after).all()
        gk, gv = local_kv_split(lc.kv[layer])
        for g, r in ((gk, oc.k), (gv, oc.v)):
            err = np.abs(widen(g[:, :, :len_after]) - widen(r[:, :, :len_after]))
            assert (err <= 2e-3 + 8e-3 * np.abs(widen(r[:, :, :len_after]))).all()
    assert st.item() == 0 and not lc.len[0].any()


def test_local_qkv_projection_masked_reset_and_overflow(bt):
    B, H, hd, L_B, P, n = 6, 2, 64, 4, 2, 2
    D = H * hd
    cfg = bt.make_config(B, H, hd, L_B, P, 8, 1)
    lc = bt.LocalCache(cfg)
    oc = oracle.Cache(B, H, P + L_B, hd)
    lens0 = [0, 3, 4, 5, 6, 1]
    oc.k[...], oc.v[...], oc.len[...] = rnd(750, 1, oc.k.shape), rnd(750, 2, oc.v.shape), lens0
    kv = np.zeros(tuple(lc.kv[0].shape), np.uint16)
    kv[:, :, :, 0], kv[:, :, :, 1] = oc.k, oc.v
    lc.kv[0].copy_(to_dev(kv))
    lc.len[0].copy_(torch.from_numpy(oc.len.copy()).cuda())
    mask = np.array([0, 1, 0, 0, 1, 0], np.uint8)            # sequence 3 (5 + 2 > 6) has no room and is not reset
    x = rnd(750, 3, (B, n, D))
    W = bits(np.concatenate([np.eye(D), 2 * np.eye(D), -np.eye(D)]))
    q = torch.empty((B, H, n, hd), dtype=torch.bfloat16, device="cuda")
    st = status_word()
    bt.bt_local_qkv_project_append(cfg, lc, 0, to_dev(x), to_dev(W), None, q, reset_mask=torch.from_numpy(mask).cuda(),
                                   dev_status=st)
    q_ref = oracle.qkv_project_append(oc, x, W, reset_mask=mask)
    assert np.array_equal(to_f64(q), q_ref)
    assert lc.len[0].cpu().tolist() == oc.len.tolist() == [2, 2, 6, 5, 2, 3]
    gk, gv = local_kv_split(lc.kv[0])
    assert np.array_equal(gk, oc.k) and np.array_equal(gv, oc.v)
    assert st.item() == bt.BT_DEV_OVERFLOW == int(oc.status[0])


# ------------------------------------------------------------------ the block decoder's step with the projection in

@pytest.mark.parametrize("hd", [64, 128])
def test_block_step_project_then_attend(bt, hd):
    B, H, N = 21, 16, 70
    D = H * hd
    lens = (np.arange(B) * 3 % (N - 1)).astype(np.int32)
    cfg, cache, oc = _block_setup(bt, 760 + hd, B, H, hd, N, lens, layers=1, layer=0)
    ws = bt.alloc_workspace(cfg)
    W, bias = rnd(760 + hd, 4, (3 * D, D)), rnd(760 + hd, 5, (3 * D,))
    st = status_word()
    for step in range(2):
        x = unit_rows(761 + hd, step, (B, 1, D))
        q = torch.empty((B, H, 1, hd), dtype=torch.bfloat16, device="cuda")
        out = torch.empty((B, H, hd), dtype=torch.bfloat16, device="cuda")
        bt.bt_block_qkv_project_append(cfg, cache, 0, to_dev(x), to_dev(W), to_dev(bias), q, dev_status=st)
        bt.bt_block_decode_attn(cfg, cache, 0, q, out, ws, dev_status=st)
        q_ref = oracle.qkv_project_append(oc, x, W, bias)
        ref = oracle.block_decode_attn(oc, np.ascontiguousarray(oracle.round_to_bf16(q_ref)[:, :, 0]))
        assert_close_proj(q, q_ref, f"q at block step {step}")
        assert_close(out, ref, f"block decode after projection, step {step}", p_bf16=True)
        assert cache.len[0].cpu().tolist() == oc.len.tolist()
    assert st.item() == 0


# ------------------------------------------------------------------ the bench shapes, sampled

@pytest.mark.parametrize("B,H,hd,n", [(4096, 16, 64, 1), (256, 16, 64, 1), (512, 16, 128, 1), (32, 16, 128, 96)])
def test_qkv_projection_at_the_bench_shapes(bt, B, H, hd, n):
    """M = 4096 (token step), M = 256 (block step), head_dim 128, and a prompt's worth of rows per sequence:
    sampled sequences against the oracle, every length exact."""
    D, N = H * hd, 128
    cfg = bt.make_config(B, H, hd, 4, 1, N, 1)
    cache = bt.BlockCache(cfg)
    fill = lambda tid, shape: gen.normal_bf16_device(770 + hd, tid, shape, device="cuda")
    x, W, bias = fill(0, (B, n, D)), fill(1, (3 * D, D)), fill(2, (3 * D,))
    lens = torch.arange(B, dtype=torch.int32, device="cuda") % (N - n + 1)
    cache.len[0].copy_(lens)
    q = torch.empty((B, H, n, hd), dtype=torch.bfloat16, device="cuda")
    st = status_word()
    bt.bt_block_qkv_project_append(cfg, cache, 0, x, W, bias, q, dev_status=st)
    assert torch.equal(cache.len[0], lens + n) and st.item() == 0
    seqs = sorted({0, 1, B // 3, B - 2, B - 1})
    oc = oracle.Cache(len(seqs), H, N, hd)
    oc.len[...] = lens.cpu().numpy()[seqs]
    q_ref = oracle.qkv_project_append(oc, gen.torch_to_bits(x[seqs]), gen.torch_to_bits(W), gen.torch_to_bits(bias))
    assert_close_proj(q[seqs], q_ref, f"q at M={B * n}")
    gk, gv = gen.torch_to_bits(cache.k[0][seqs]), gen.torch_to_bits(cache.v[0][seqs])
    for g, r in ((gk, oc.k), (gv, oc.v)):
        err = np.abs(widen(g) - widen(r))
        assert (err <= 2e-3 + 8e-3 * np.abs(widen(r))).all()      # rows outside the window are zero on both sides


# ------------------------------------------------------------------ the prompt's path with the projection in

@pytest.mark.parametrize("hd,T", [(64, 200), (128, 130)])
def test_prompt_projection_then_prefill_from_the_cache(bt, hd, T):
    """The block decoder's prefill with the projection in front (sections 2.1, 2.3): the prompt's T block embeddings
    are projected in one call, the epilogue writes the T K,V rows of every sequence into the block cache, and the
    prefill attention reads K and V in place from the cache.  Against the oracle's projection + append + dense
    causal attention; lengths exact."""
    B, H, N = 3, 4, 256
    D = H * hd
    cfg = bt.make_config(B, H, hd, 4, 1, N, 1)
    cache = bt.BlockCache(cfg)
    x = unit_rows(780 + hd, 0, (B, T, D))
    W, bias = rnd(780 + hd, 1, (3 * D, D)), rnd(780 + hd, 2, (3 * D,))
    q = torch.empty((B, H, T, hd), dtype=torch.bfloat16, device="cuda")
    out = torch.empty((B, H, T, hd), dtype=torch.bfloat16, device="cuda")
    st = status_word()
    bt.bt_block_qkv_project_append(cfg, cache, 0, to_dev(x), to_dev(W), to_dev(bias), q, dev_status=st)
    bt.bt_block_prefill_attn(cfg, q, cache.k[0], cache.v[0], out, n_blocks=T, kv_seq_stride=N, dev_status=st)
    oc = oracle.Cache(B, H, N, hd)
    q_ref = oracle.qkv_project_append(oc, x, W, bias)
    assert_close_proj(q, q_ref, "q of the prompt projection")
    assert cache.len[0].cpu().tolist() == oc.len.tolist() == [T] * B and st.item() == 0
    ref = oracle.block_prefill_attn(oracle.round_to_bf16(q_ref), oc.k, oc.v, kv_seq_stride=N)
    assert_close(out, ref, "prefill attention over the projected cache", p_bf16=True)
