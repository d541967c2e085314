"""Pins for the CPU oracle: closed forms, invariants the paper fixes, a library routine
and brute force.  None of these call the CUDA path."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from workloads import gen

HD = 16


def bits(x):
    return gen.f32_to_bf16_bits(np.asarray(x, np.float32))


def widen(b):
    return gen.bf16_bits_to_f32(b).astype(np.float64)


def rnd(seed, tid, shape):
    return gen.normal_bf16_bits(seed, tid, shape)


# ---------------------------------------------------------------- closed forms

def test_single_row_returns_its_value_exactly():
    q, K, V = rnd(1, 0, (HD,)), rnd(1, 1, (1, HD)), rnd(1, 2, (1, HD))
    out, p = oracle.attend(q, K, V)
    assert p.tolist() == [1.0]
    assert np.array_equal(out, widen(V[0]))


def test_equal_keys_give_mean_of_values():
    q = rnd(2, 0, (HD,))
    K = np.repeat(rnd(2, 1, (1, HD)), 7, axis=0)
    V = rnd(2, 2, (7, HD))
    out, p = oracle.attend(q, K, V)
    np.testing.assert_allclose(p, np.full(7, 1 / 7), rtol=0, atol=1e-15)
    np.testing.assert_allclose(out, widen(V).mean(0), rtol=0, atol=1e-14)


def test_zero_query_gives_mean_of_values():
    q = np.zeros(HD, np.uint16)
    K, V = rnd(3, 1, (9, HD)), rnd(3, 2, (9, HD))
    out, _ = oracle.attend(q, K, V)
    np.testing.assert_allclose(out, widen(V).mean(0), rtol=0, atol=1e-14)


def test_two_rows_is_a_logistic_blend():
    # with two rows softmax reduces to the logistic function of the score difference
    q, K, V = rnd(4, 0, (HD,)), rnd(4, 1, (2, HD)), rnd(4, 2, (2, HD))
    scale = 0.37
    s = scale * (widen(K) @ widen(q))
    w0 = 1.0 / (1.0 + math.exp(-(s[0] - s[1])))
    out, _ = oracle.attend(q, K, V, scale=scale)
    np.testing.assert_allclose(out, widen(V[1]) + w0 * (widen(V[0]) - widen(V[1])), rtol=0, atol=1e-13)


def test_handmade_scores_one_two_three():
    # q = e0, keys with first coordinate 0, 1, 2 and scale = ln 2  ->  weights 1/7, 2/7, 4/7
    q = bits([1.0] + [0.0] * (HD - 1))
    K = np.zeros((3, HD), np.float32)
    K[:, 0] = [0.0, 1.0, 2.0]
    K[:, 1] = [5.0, -3.0, 2.0]  # orthogonal to q: must not matter
    V = np.zeros((3, HD), np.float32)
    V[:, 0] = [7.0, 14.0, 21.0]
    V[:, 3] = [1.0, 0.0, 0.0]
    out, p = oracle.attend(q, bits(K), bits(V), scale=math.log(2.0))
    np.testing.assert_allclose(p, [1 / 7, 2 / 7, 4 / 7], rtol=0, atol=1e-15)
    np.testing.assert_allclose(out[0], 1.0 + 4.0 + 12.0, rtol=0, atol=1e-13)
    np.testing.assert_allclose(out[3], 1 / 7, rtol=0, atol=1e-15)


def test_dominant_key_selects_its_value():
    q = bits(np.full(HD, 4.0))
    K = rnd(5, 1, (33, HD))
    V = rnd(5, 2, (33, HD))
    K[17] = bits(np.full(HD, 16.0))  # score 1024*scale, far above the rest
    out, p = oracle.attend(q, K, V, scale=1.0)
    assert p[17] > 1 - 1e-12
    np.testing.assert_allclose(out, widen(V[17]), rtol=0, atol=1e-9)


# ---------------------------------------------------------------- properties

@pytest.mark.parametrize("n", [1, 2, 5, 64, 513])
def test_probabilities_sum_to_one_and_hull(n):
    q, K, V = rnd(6, n, (HD,)), rnd(6, 100 + n, (n, HD)), rnd(6, 200 + n, (n, HD))
    out, p = oracle.attend(q, K, V)
    assert abs(p.sum() - 1.0) < 1e-12 and (p >= 0).all()
    Vf = widen(V)
    assert (out <= Vf.max(0) + 1e-12).all() and (out >= Vf.min(0) - 1e-12).all()


def test_permutation_invariance():
    n = 50
    q, K, V = rnd(7, 0, (HD,)), rnd(7, 1, (n, HD)), rnd(7, 2, (n, HD))
    perm = np.random.default_rng(0).permutation(n)
    a, _ = oracle.attend(q, K, V)
    b, _ = oracle.attend(q, K[perm], V[perm])
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-13)


def test_log_sum_exp_merge_of_two_halves_equals_whole():
    # the algebra a split of the row range relies on, checked against the unsplit definition
    n, cut = 40, 13
    q, K, V = rnd(8, 0, (HD,)), rnd(8, 1, (n, HD)), rnd(8, 2, (n, HD))
    scale = oracle.default_scale(HD)
    whole, _ = oracle.attend(q, K, V)
    parts = []
    for sl in (slice(0, cut), slice(cut, n)):
        o, _ = oracle.attend(q, K[sl], V[sl])
        s = scale * (widen(K[sl]) @ widen(q))
        parts.append((o, s.max() + math.log(np.exp(s - s.max()).sum())))
    (o1, l1), (o2, l2) = parts
    w1 = 1.0 / (1.0 + math.exp(l2 - l1))
    np.testing.assert_allclose(w1 * o1 + (1 - w1) * o2, whole, rtol=0, atol=1e-13)


def test_float32_twin_agrees():
    n = 300
    q, K, V = rnd(9, 0, (64,)), rnd(9, 1, (n, 64)), rnd(9, 2, (n, 64))
    a, pa = oracle.attend(q, K, V)
    b, pb = oracle.attend(q, K, V, f32=True)
    assert b.dtype == np.float32
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-5)
    np.testing.assert_allclose(pa, pb, rtol=0, atol=1e-6)


# ---------------------------------------------------------------- brute force, library routine

def brute_force(q, K, V, scale):
    """Pure-Python restatement with Python floats; only for tiny inputs."""
    n, hd = len(K), len(q)
    s = [scale * sum(q[d] * K[j][d] for d in range(hd)) for j in range(n)]
    m = max(s)
    e = [math.exp(x - m) for x in s]
    z = sum(e)
    return [sum(e[j] / z * V[j][d] for j in range(n)) for d in range(hd)]


@pytest.mark.parametrize("n,hd", [(1, 4), (3, 4), (6, 8), (11, 8)])
def test_brute_force_tiny(n, hd):
    q, K, V = rnd(10, n, (hd,)), rnd(10, 50 + n, (n, hd)), rnd(10, 90 + n, (n, hd))
    out, _ = oracle.attend(q, K, V, scale=0.5)
    ref = brute_force(widen(q).tolist(), widen(K).tolist(), widen(V).tolist(), 0.5)
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-13)


def sdpa64(q, k, v, causal):
    t = lambda b: torch.from_numpy(widen(b))
    return torch.nn.functional.scaled_dot_product_attention(t(q), t(k), t(v), is_causal=causal).numpy()


def test_prefill_matches_library_causal_attention():
    B, H, T, hd = 2, 3, 37, 32
    q, k, v = rnd(11, 0, (B, H, T, hd)), rnd(11, 1, (B, H, T, hd)), rnd(11, 2, (B, H, T, hd))
    np.testing.assert_allclose(oracle.block_prefill_attn(q, k, v), sdpa64(q, k, v, True), rtol=0, atol=1e-12)


def test_prefill_is_not_the_transposed_or_unmasked_variant():
    # a mistake the library pin must see: no mask, or mask on the wrong side
    B, H, T, hd = 1, 1, 9, 8
    q, k, v = rnd(12, 0, (B, H, T, hd)), rnd(12, 1, (B, H, T, hd)), rnd(12, 2, (B, H, T, hd))
    out = oracle.block_prefill_attn(q, k, v)
    assert np.abs(out - sdpa64(q, k, v, False)).max() > 1e-3
    # row 0 sees only block 0
    np.testing.assert_allclose(out[0, 0, 0], widen(v[0, 0, 0]), rtol=0, atol=0)
    # last row sees everything: equals the unmasked library result for that row
    np.testing.assert_allclose(out[0, 0, -1], sdpa64(q, k, v, False)[0, 0, -1], rtol=0, atol=1e-12)


def test_prefill_honours_kv_stride():
    B, H, T, hd, cap = 2, 2, 5, 8, 9
    q = rnd(13, 0, (B, H, T, hd))
    k, v = rnd(13, 1, (B, H, cap, hd)), rnd(13, 2, (B, H, cap, hd))
    a = oracle.block_prefill_attn(q, k, v)
    b = oracle.block_prefill_attn(q, np.ascontiguousarray(k[:, :, :T]), np.ascontiguousarray(v[:, :, :T]))
    assert np.array_equal(a, b)


# ---------------------------------------------------------------- invariants the paper fixes

def test_cached_decode_equals_full_recompute():
    """KV caching changes cost, not the function: step-by-step append + decode reproduces the
    rows of the dense causal prefill."""
    B, H, T, hd = 3, 2, 21, 16
    q, k, v = rnd(14, 0, (B, H, T, hd)), rnd(14, 1, (B, H, T, hd)), rnd(14, 2, (B, H, T, hd))
    full = oracle.block_prefill_attn(q, k, v)
    c = oracle.Cache(B, H, T, hd)
    for t in range(T):
        oracle.kv_append(c, k[:, :, t:t + 1], v[:, :, t:t + 1])
        assert (c.len == t + 1).all()
        out = oracle.block_decode_attn(c, np.ascontiguousarray(q[:, :, t]))
        assert np.array_equal(out, full[:, :, t])
    assert np.array_equal(c.k, k) and np.array_equal(c.v, v) and c.status[0] == 0


def test_densified_step_is_the_matching_rows_of_dense_causal_attention():
    """The densified block decoder's step (m sub-block rows and queries at once) changes the schedule,
    not the function: steps of m rows reproduce the rows of the dense causal prefill over all
    sub-block tokens; and m = 1 is the ordinary append + decode."""
    B, H, hd, m, steps = 2, 3, 16, 4, 5
    T = m * steps
    q, k, v = rnd(15, 0, (B, H, T, hd)), rnd(15, 1, (B, H, T, hd)), rnd(15, 2, (B, H, T, hd))
    full = oracle.block_prefill_attn(q, k, v)
    c = oracle.Cache(B, H, T, hd)
    for s_ in range(steps):
        sl = slice(s_ * m, (s_ + 1) * m)
        out = oracle.block_decode_step_multi(c, q[:, :, sl], k[:, :, sl], v[:, :, sl])
        assert (c.len == (s_ + 1) * m).all()
        assert np.array_equal(out, full[:, :, sl])
    assert np.array_equal(c.k, k) and np.array_equal(c.v, v) and c.status[0] == 0
    # m = 1: append then decode
    c1, c2 = oracle.Cache(B, H, 8, hd), oracle.Cache(B, H, 8, hd)
    for t in range(3):
        a_ = oracle.block_decode_step_multi(c1, q[:, :, t:t + 1], k[:, :, t:t + 1], v[:, :, t:t + 1])
        oracle.kv_append(c2, k[:, :, t:t + 1], v[:, :, t:t + 1])
        assert np.array_equal(a_[:, :, 0], oracle.block_decode_attn(c2, np.ascontiguousarray(q[:, :, t])))


def test_densified_step_without_room_appends_nothing():
    """All m rows or none: a sequence one row short of room is left as it is, flagged, and every query
    sees exactly its old rows (so the m outputs of one head differ only through their queries)."""
    B, H, hd, N, m = 2, 1, 16, 6, 4
    c = oracle.Cache(B, H, N, hd)
    c.k[...], c.v[...] = rnd(16, 1, (B, H, N, hd)), rnd(16, 2, (B, H, N, hd))
    c.len[...] = [2, 3]
    k0 = c.k.copy()
    q = np.repeat(rnd(16, 0, (B, H, 1, hd)), m, axis=2)   # the same query m times
    out = oracle.block_decode_step_multi(c, q, rnd(16, 3, (B, H, m, hd)), rnd(16, 4, (B, H, m, hd)))
    assert c.len.tolist() == [6, 3] and c.status[0] == 1          # BT_DEV_OVERFLOW
    assert np.array_equal(c.k[1], k0[1]) and not np.array_equal(c.k[0], k0[0])
    assert all(np.array_equal(out[1, :, i], out[1, :, 0]) for i in range(m))       # same rows, same query
    assert not np.array_equal(out[0, :, 1], out[0, :, 0])                            # causal: one more row each


def test_block_length_one_is_vanilla_causal_attention():
    """At L_B = 1 every token is its own block, so block-decoder attention over the block cache
    is token-level causal attention (the library routine, float64)."""
    B, H, L, hd = 2, 2, 24, 16
    q, k, v = rnd(15, 0, (B, H, L, hd)), rnd(15, 1, (B, H, L, hd)), rnd(15, 2, (B, H, L, hd))
    ref = sdpa64(q, k, v, True)
    c = oracle.Cache(B, H, L, hd)
    for t in range(L):
        oracle.kv_append(c, k[:, :, t:t + 1], v[:, :, t:t + 1])
        out = oracle.block_decode_attn(c, np.ascontiguousarray(q[:, :, t]))
        np.testing.assert_allclose(out, ref[:, :, t], rtol=0, atol=1e-12)


def test_ragged_lengths_and_rows_past_len_are_ignored():
    B, H, cap, hd = 4, 2, 12, 8
    c = oracle.Cache(B, H, cap, hd)
    c.k[...] = rnd(16, 1, c.k.shape)
    c.v[...] = rnd(16, 2, c.v.shape)
    c.len[...] = [1, 5, 12, 7]
    q = rnd(16, 0, (B, H, hd))
    out = oracle.block_decode_attn(c, q)
    for b in range(B):
        n = c.len[b]
        ref = sdpa64(q[b][:, None, :], c.k[b, :, :n], c.v[b, :, :n], False)[:, 0]
        np.testing.assert_allclose(out[b], ref, rtol=0, atol=1e-12)
    c2 = c.copy()
    for b in range(B):
        c2.k[b, :, c.len[b]:] = 0x7FC0  # NaN beyond the length
        c2.v[b, :, c.len[b]:] = 0x7FC0
    assert np.array_equal(oracle.block_decode_attn(c2, q), out)


def test_spike_row_at_the_length_boundary():
    """A key far above the rest flips the output to its value: inside the length it must win,
    one past the length it must be invisible (an off-by-one in the row range fails here)."""
    B, H, cap, hd, n = 1, 1, 40, 8, 31
    c = oracle.Cache(B, H, cap, hd)
    c.k[...] = rnd(17, 1, c.k.shape)
    c.v[...] = rnd(17, 2, c.v.shape)
    c.len[...] = n
    q = bits(np.full((B, H, hd), 3.0))
    base = oracle.block_decode_attn(c, q)
    spike_k, spike_v = bits(np.full(hd, 30.0)), bits(np.arange(hd) + 100.0)
    for row, visible in ((0, True), (n - 1, True), (n, False)):
        d = c.copy()
        d.k[0, 0, row], d.v[0, 0, row] = spike_k, spike_v
        out = oracle.block_decode_attn(d, q)
        if visible:
            np.testing.assert_allclose(out[0, 0], widen(spike_v), rtol=0, atol=1e-6)
        else:
            assert np.array_equal(out, base)


def test_append_overflow_and_empty_cache():
    c = oracle.Cache(2, 1, 3, 8)
    c.len[...] = [2, 3]
    k, v = rnd(18, 1, (2, 1, 1, 8)), rnd(18, 2, (2, 1, 1, 8))
    oracle.kv_append(c, k, v)
    assert c.len.tolist() == [3, 3] and c.status[0] == oracle.ST_OVERFLOW
    assert np.array_equal(c.k[0, 0, 2], k[0, 0, 0]) and not c.k[1].any()
    e = oracle.Cache(1, 1, 3, 8)
    out = oracle.block_decode_attn(e, rnd(18, 0, (1, 1, 8)))
    assert not out.any() and e.status[0] == oracle.ST_EMPTY


# ---------------------------------------------------------------- token decoder

def run_token_blocks(L_B, P, n_blocks, seed, B=2, H=2, hd=8, poison_between=False):
    """Drive the fused token step over n_blocks blocks following the schedule model."""
    c = oracle.Cache(B, H, P + L_B, hd)
    outs, lens = [], []
    for t, (reset, n_app, len_after) in enumerate(oracle.token_step_schedule(L_B, P, n_blocks * L_B)):
        q, k, v = (rnd(seed, 10 * t + i, (B, H, n_app, hd)) for i in range(3))
        if reset and poison_between:
            c.k[...] = rnd(seed + 99, t, c.k.shape)  # whatever the finished block left behind
            c.v[...] = 0x7FC0
        outs.append(oracle.token_decode_attn(c, q, k, v, reset_first=bool(reset)))
        assert (c.len == len_after).all()
        lens.append(len_after)
    return outs, lens, c


@pytest.mark.parametrize("L_B,P", [(4, 1), (4, 2), (1, 1), (8, 2), (2, 4)])
def test_token_decoder_never_crosses_a_block_boundary(L_B, P):
    a, lens, _ = run_token_blocks(L_B, P, 3, seed=20)
    b, _, _ = run_token_blocks(L_B, P, 3, seed=20, poison_between=True)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)
    assert max(lens) == P + L_B - 1


def test_token_step_equals_attention_over_prefix_plus_same_block_tokens():
    L_B, P, B, H, hd = 4, 2, 2, 2, 8
    c = oracle.Cache(B, H, P + L_B, hd)
    ks, vs = [], []
    for t, (reset, n_app, _) in enumerate(oracle.token_step_schedule(L_B, P, 2 * L_B)):
        q, k, v = (rnd(21, 10 * t + i, (B, H, n_app, hd)) for i in range(3))
        if reset:
            ks, vs = [], []
        ks.append(k)
        vs.append(v)
        out = oracle.token_decode_attn(c, q, k, v, reset_first=bool(reset))
        Kall, Vall = np.concatenate(ks, 2), np.concatenate(vs, 2)
        n = Kall.shape[2]
        for i in range(n_app):  # new row i sees rows 0 .. n - n_app + i
            m = n - n_app + i + 1
            ref = sdpa64(q[:, :, i:i + 1], Kall[:, :, :m], Vall[:, :, :m], False)
            np.testing.assert_allclose(out[:, :, i:i + 1], ref, rtol=0, atol=1e-12)


def test_token_attend_only_and_masked_reset():
    B, H, hd, cap = 3, 1, 8, 5
    c = oracle.Cache(B, H, cap, hd)
    for t in range(3):
        q, k, v = (rnd(22, 10 * t + i, (B, H, 1, hd)) for i in range(3))
        oracle.token_decode_attn(c, q, k, v)
    assert c.len.tolist() == [3, 3, 3]
    q = rnd(22, 77, (B, H, 1, hd))
    out = oracle.token_decode_attn(c, q, None, None)
    ref = sdpa64(q, c.k[:, :, :3], c.v[:, :, :3], False)
    np.testing.assert_allclose(out, ref, rtol=0, atol=1e-12)
    assert c.len.tolist() == [3, 3, 3]
    q, k, v = (rnd(22, 90 + i, (B, H, 1, hd)) for i in range(3))
    out = oracle.token_decode_attn(c, q, k, v, reset_mask=[0, 1, 0])
    assert c.len.tolist() == [4, 1, 4]
    np.testing.assert_array_equal(out[1, 0, 0], widen(v[1, 0, 0]))
    oracle.local_kv_reset(c, mask=[1, 0, 0])
    assert c.len.tolist() == [0, 1, 4]
    oracle.local_kv_reset(c)
    assert c.len.tolist() == [0, 0, 0]


def test_token_overflow_is_skipped_and_flagged():
    B, H, hd, cap = 2, 1, 8, 2
    c = oracle.Cache(B, H, cap, hd)
    c.len[...] = [1, 2]
    q, k, v = (rnd(23, i, (B, H, 1, hd)) for i in range(3))
    out = oracle.token_decode_attn(c, q, k, v)
    assert c.len.tolist() == [2, 2] and c.status[0] & oracle.ST_OVERFLOW
    assert not out[1].any() and not c.k[1].any()


def test_attend_only_over_the_last_rows_equals_the_appending_step():
    """k_new = None with n_q queries: they belong to the last n_q cached rows, query i sees rows
    0 .. len - n_q + i.  Pinned to the appending form of the same step, which the pins above fix."""
    B, H, hd, cap = 3, 2, 8, 9
    for n_q, start in ((1, 3), (2, 0), (4, 2), (4, 5)):
        a = oracle.Cache(B, H, cap, hd)
        a.k[...], a.v[...] = rnd(24, 1, a.k.shape), rnd(24, 2, a.v.shape)
        a.len[...] = start
        b = a.copy()
        q, k, v = (rnd(24, 10 * n_q + i, (B, H, n_q, hd)) for i in range(3))
        want = oracle.token_decode_attn(a, q, k, v)
        oracle.kv_append(b, k, v)
        got = oracle.token_decode_attn(b, q, None, None)
        assert np.array_equal(got, want) and b.len.tolist() == a.len.tolist() == [start + n_q] * B
        # and to the library routine: query i over the first start + i + 1 rows
        for i in range(n_q):
            m = start + i + 1
            np.testing.assert_allclose(got[:, :, i:i + 1], sdpa64(q[:, :, i:i + 1], b.k[:, :, :m], b.v[:, :, :m], False),
                                       rtol=0, atol=1e-12)
    # fewer rows than queries: the leading queries have nothing to see
    e = oracle.Cache(1, 1, 4, hd)
    e.k[...], e.v[...] = rnd(24, 5, e.k.shape), rnd(24, 6, e.v.shape)
    e.len[...] = 1
    out = oracle.token_decode_attn(e, rnd(24, 7, (1, 1, 2, hd)), None, None)
    assert not out[0, 0, 0].any() and np.array_equal(out[0, 0, 1], widen(e.v[0, 0, 0])) and e.status[0] & oracle.ST_EMPTY


# ---------------------------------------------------------------- projections either side of the path

def test_round_to_bf16_is_nearest_even():
    # ties: 1 + 2^-8 lies midway between 1 (even mantissa) and 1 + 2^-7; 1 + 3*2^-8 between 1 + 2^-7 (odd) and 1 + 2^-6
    cases = {1.0: 0x3F80, 1.0 + 2.0 ** -8: 0x3F80, 1.0 + 3 * 2.0 ** -8: 0x3F82, 1.0 + 2.0 ** -8 + 2.0 ** -30: 0x3F81,
             -2.5: 0xC020, 0.0: 0x0000, 255.5: 0x4380, 3.0e-5: int(bits([3.0e-5])[0])}
    for v, want in cases.items():
        assert int(oracle.round_to_bf16([v])[0]) == want, v
    # every float32 input: the independent float32 -> bf16 rounding of the input generators agrees
    x = np.concatenate([widen(rnd(30, 0, (4096,))) * s for s in (1.0, 37.0, 1e-3)]).astype(np.float32)
    x = (x.astype(np.float64) * (1.0 + 2.0 ** -10)).astype(np.float32)  # off the bf16 grid
    assert np.array_equal(oracle.round_to_bf16(x.astype(np.float64)), bits(x))


def test_linear_identity_one_hot_zero_input_and_library_product():
    M, K = 5, 12
    x = rnd(31, 0, (M, K))
    eye = bits(np.eye(K))
    assert np.array_equal(oracle.linear(x, eye), widen(x))                      # identity: rows come back exactly
    perm = np.random.default_rng(31).permutation(K)
    onehot = bits(2.0 * np.eye(K)[perm])                                        # output o = 2 * x[perm[o]]
    assert np.array_equal(oracle.linear(x, onehot), 2.0 * widen(x)[:, perm])
    W, b = rnd(31, 1, (7, K)), rnd(31, 2, (7,))
    assert np.array_equal(oracle.linear(bits(np.zeros((M, K))), W, b), np.tile(widen(b), (M, 1)))   # zero input: the bias
    ref = widen(x) @ widen(W).T + widen(b)                                      # numpy's float64 product
    np.testing.assert_allclose(oracle.linear(x, W, b), ref, rtol=0, atol=1e-12)
    np.testing.assert_allclose(oracle.linear(x, W), ref - widen(b), rtol=0, atol=1e-12)
    np.testing.assert_allclose(oracle.linear(x, W, b, f32=True), ref, rtol=0, atol=2e-5)
    # a non-square, non-symmetric case told apart from its transpose: W[o][k] = 1 only at (0, 1)
    W2 = np.zeros((3, 2)); W2[0, 1] = 1.0
    y = oracle.linear(bits([[5.0, 7.0]]), bits(W2))
    assert y.tolist() == [[7.0, 0.0, 0.0]]


def test_prefix_projection_layout():
    """Output feature p*D + d is dimension d of prefix token p (section 2.4: the context embedding is
    projected into P prefix token embeddings)."""
    B, D, P = 3, 8, 2
    ctx = rnd(32, 0, (B, D))
    W = np.zeros((P * D, D))
    W[:D] = np.eye(D)                 # prefix token 0 = the context embedding
    W[D:] = -np.eye(D)[::-1]          # prefix token 1 = its negated mirror image
    out = oracle.prefix_project(ctx, bits(W), None, P)
    assert out.shape == (B, P, D)
    assert np.array_equal(out[:, 0], widen(ctx)) and np.array_equal(out[:, 1], -widen(ctx)[:, ::-1])
    b = rnd(32, 1, (P * D,))
    np.testing.assert_allclose(oracle.prefix_project(ctx, bits(W), b, P), out + widen(b).reshape(1, P, D), rtol=0, atol=1e-12)


def _qkv_case(seed, B, n, H, hd, cap, lens):
    D = H * hd
    c = oracle.Cache(B, H, cap, hd)
    c.k[...], c.v[...] = rnd(seed, 1, c.k.shape), rnd(seed, 2, c.v.shape)
    c.len[...] = lens
    return c, rnd(seed, 3, (B, n, D)), D


def test_qkv_projection_with_identity_blocks_caches_the_input_rows():
    """W = [I; 2I; -I]: q is x regrouped by head, the K rows are 2x and the V rows -x, bit for bit, at
    rows len .. len+n-1 of each head's slab; a sequence without room keeps everything."""
    B, n, H, hd, cap = 4, 3, 2, 4, 6
    lens = [0, 2, 3, 4]                      # the last one has no room for 3 more rows
    c, x, D = _qkv_case(33, B, n, H, hd, cap, lens)
    before = c.copy()
    W = bits(np.concatenate([np.eye(D), 2 * np.eye(D), -np.eye(D)]))
    q = oracle.qkv_project_append(c, x, W)
    xr = x.reshape(B, n, H, hd).transpose(0, 2, 1, 3)          # [B,H,n,hd]
    assert np.array_equal(q, widen(xr))
    assert c.len.tolist() == [3, 5, 6, 4] and c.status[0] == oracle.ST_OVERFLOW
    for b in range(3):
        l = lens[b]
        assert np.array_equal(c.k[b, :, l:l + n], bits(2.0 * widen(xr[b]))) and np.array_equal(c.v[b, :, l:l + n], bits(-widen(xr[b])))
        assert np.array_equal(c.k[b, :, :l], before.k[b, :, :l]) and np.array_equal(c.k[b, :, l + n:], before.k[b, :, l + n:])
    assert np.array_equal(c.k[3], before.k[3]) and np.array_equal(c.v[3], before.v[3])


def test_project_then_append_equals_append_of_projected_rows():
    B, n, H, hd, cap = 3, 2, 3, 8, 7
    c, x, D = _qkv_case(34, B, n, H, hd, cap, [0, 5, 1])
    W, bias = rnd(34, 4, (3 * D, D)), rnd(34, 5, (3 * D,))
    ref = c.copy()
    q = oracle.qkv_project_append(c, x, W, bias)
    y = (widen(x).reshape(B * n, D) @ widen(W).T + widen(bias)).reshape(B, n, 3, H, hd)   # numpy's float64 product
    np.testing.assert_allclose(q, y[:, :, 0].transpose(0, 2, 1, 3), rtol=0, atol=1e-12)
    kn, vn = (np.ascontiguousarray(y[:, :, j].transpose(0, 2, 1, 3)) for j in (1, 2))
    oracle.kv_append(ref, oracle.round_to_bf16(kn), oracle.round_to_bf16(vn))
    # (the two float64 sums may differ in the last place, which can move a value across a rounding boundary)
    for got, want in ((c.k, ref.k), (c.v, ref.v)):
        d = np.abs(got.astype(np.int32) - want.astype(np.int32))
        assert d.max() <= 1 and (d > 0).mean() < 1e-3
    assert np.array_equal(c.len, ref.len) and c.len.tolist() == [2, 7, 3]
    # exact arithmetic (small integers): no rounding anywhere, so the rows are fixed bit for bit
    rng = np.random.default_rng(34)
    xi, Wi = bits(rng.integers(-1, 2, (B, n, D))), bits(rng.integers(-1, 3, (3 * D, D)))
    c2, r2 = oracle.Cache(B, H, cap, hd), oracle.Cache(B, H, cap, hd)
    oracle.qkv_project_append(c2, xi, Wi)
    yi = (widen(xi).reshape(B * n, D) @ widen(Wi).T).reshape(B, n, 3, H, hd)
    oracle.kv_append(r2, *(bits(np.ascontiguousarray(yi[:, :, j].transpose(0, 2, 1, 3))) for j in (1, 2)))
    assert np.array_equal(c2.k, r2.k) and np.array_equal(c2.v, r2.v) and c2.len.tolist() == [n] * B


def test_qkv_projection_reset_is_the_block_boundary_reset():
    B, n, H, hd, cap = 4, 2, 2, 4, 5
    c, x, D = _qkv_case(35, B, n, H, hd, cap, [3, 4, 0, 5])
    W = rnd(35, 4, (3 * D, D))
    a, b = c.copy(), c.copy()
    mask = [1, 0, 0, 1]
    qa = oracle.qkv_project_append(a, x, W, reset_mask=mask)
    oracle.local_kv_reset(b, mask)
    qb = oracle.qkv_project_append(b, x, W)
    assert np.array_equal(qa, qb) and np.array_equal(a.k, b.k) and np.array_equal(a.v, b.v)
    assert a.len.tolist() == b.len.tolist() == [2, 4, 2, 2] and a.status[0] == oracle.ST_OVERFLOW  # sequence 1: 4 + 2 > 5
    e = c.copy()
    oracle.qkv_project_append(e, x, W, reset_first=True)
    assert e.len.tolist() == [2, 2, 2, 2] and e.status[0] == 0
    # after a reset the rows land at index 0 .. n-1, as for the masked sequences above
    assert np.array_equal(e.k[0, :, :n], a.k[0, :, :n]) and np.array_equal(e.v[3, :, :n], a.v[3, :, :n])


def test_projected_step_equals_appending_step_on_projected_rows():
    """The path with the projections in: project + cache, then attend-only over the cache, gives what the
    fused append-and-attend step gives when handed the projected (rounded) rows."""
    B, n, H, hd, cap = 2, 2, 2, 8, 6
    c, x, D = _qkv_case(36, B, n, H, hd, cap, [1, 3])
    W = rnd(36, 4, (3 * D, D))
    a = c.copy()
    q = oracle.qkv_project_append(c, x, W)
    qb = oracle.round_to_bf16(q)
    got = oracle.token_decode_attn(c, qb, None, None)
    l0 = a.len.copy()
    kn = np.stack([c.k[b, :, l0[b]:l0[b] + n] for b in range(B)])
    vn = np.stack([c.v[b, :, l0[b]:l0[b] + n] for b in range(B)])
    want = oracle.token_decode_attn(a, qb, kn, vn)
    assert np.array_equal(got, want)


# ---------------------------------------------------------------- schedule model + byte model

def golden():
    vals = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "paper_counting_examples.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if "=" in line:
                k, v = line.split("=")
                vals[k.strip()] = int(v)
    return vals


def test_schedule_model():
    g = golden()
    s = oracle.token_step_schedule(4, 2, 8)
    assert [x[2] for x in s] == [2, 3, 4, 5, 2, 3, 4, 5]
    assert max(x[2] for x in s) == g["local_attn_len_LB4_P2"]
    assert [x[0] for x in s] == [1, 0, 0, 0, 1, 0, 0, 0]
    ev = oracle.generation_schedule(4, 1, 128, 2048)
    assert ev[0] == ("prefill", 32)
    assert sum(e[0] == "token" for e in ev) == 2048
    blocks = [e[1] for e in ev if e[0] == "block"]
    assert blocks == list(range(33, 33 + 512))
    # L_B = 1: one block step per token, local cache never beyond the prefix
    ev1 = oracle.generation_schedule(1, 1, 128, 16)
    assert all(e[3] == 1 and e[1] == 1 for e in ev1 if e[0] == "token")


def test_byte_model_matches_the_papers_counting_examples():
    from workloads import traffic
    g = golden()
    per_tok = traffic.kv_bytes_per_token(g["llama7b_layers"], g["llama7b_model_dim"])
    assert per_tok == g["llama7b_kv_bytes_per_token"]
    assert per_tok * 2048 * 16 == g["llama7b_kv_bytes_L2048_B16"]
    # block-decoder KV reads over a generation shrink by L_B^2 (size / L_B, frequency / L_B)
    def kv_reads(L_B, L=2048, B=1, H=16, hd=64):
        return sum(B * H * n * 2 * hd * 2 for n in range(1, L // L_B + 1))
    r = kv_reads(1) / kv_reads(4)
    assert abs(r / 16 - 1) < 0.01
    # token-decoder KV reads: L_B^2-ish per block over L/L_B blocks vs L^2  ->  ~ L / L_B
    L, L_B = 2048, 4
    vanilla = sum(range(1, L + 1))
    local = (L // L_B) * sum(range(1, L_B + 1))
    assert abs((vanilla / local) / (L / L_B) - 1) < 0.25
