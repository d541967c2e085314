"""Decode-heavy generation (benchmark configs[4]: the L_B sweep) through the harness driver: every
token step and block step of a small generation against the oracle at L_B = 1, 2, 4, 8, and the
full-size run (batch 512, prompt 128, 2048 generated tokens) at L_B = 4 with lengths, cache rows and
sampled outputs checked."""
import numpy as np
import pytest
import torch

import oracle
from oracle import schedule
from workloads import configs, gen

from util import assert_close, local_kv_split

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bt():
    import paper_2406_02657_b200 as bt
    assert torch.cuda.is_available()
    return bt


def _fill(seed):
    return lambda tid, shape: gen.normal_bf16_device(seed, tid, shape, device="cuda")


@pytest.mark.parametrize("L_B", [1, 2, 4, 8])
def test_small_generation_every_step_against_the_oracle(bt, L_B):
    from paper_2406_02657_b200 import harness
    prompt, G = 32, 48
    w = configs.scaled(configs.sweep(L_B), batch=5, heads=3, n_layers=2, max_blocks=(prompt + G) // L_B,
                       prompt_blocks=prompt // L_B, prompt_tokens=prompt, gen_tokens=G)
    run = harness.GenerationRun(w, fill=_fill(4200 + L_B), ring=2)
    B, H, hd, T = w.batch, w.heads, w.head_dim, w.prompt_blocks
    bits = gen.torch_to_bits
    run.start()
    torch.cuda.synchronize()
    ob = {l: oracle.Cache(B, H, w.max_blocks, hd) for l in range(w.n_layers)}
    ol = {l: oracle.Cache(B, H, w.local_cap, hd) for l in range(w.n_layers)}
    for l in range(w.n_layers):
        assert_close(run.pout[l], oracle.block_prefill_attn(bits(run.pq[l]), bits(run.pk[l]), bits(run.pv[l])), f"prefill layer {l}", p_bf16=True)
        oracle.kv_append(ob[l], bits(run.pk[l]), bits(run.pv[l]))
    events = schedule.generation_schedule(L_B, w.prefix_len, prompt, G)
    assert events[0] == ("prefill", T)
    ev = iter(events[1:])
    for g in range(G // L_B):
        r = g % run.ring
        # the driver issues the whole block; replay it step by step here to compare after every launch
        for j in range(L_B):
            kind, reset, n_app, len_after = next(ev)
            assert kind == "token" and n_app == 1  # prefix length 1: the prefix row is the block's first row
            for l in range(w.n_layers):
                bt.bt_token_decode_attn(run.cfg, run.local, l, run.tq[r, j, l], run.tk[r, j, l], run.tv[r, j, l], run.tout[l],
                                        n_q=1, reset_first=(j == 0), dev_status=run.status)
                ref = oracle.token_decode_attn(ol[l], bits(run.tq[r, j, l]), bits(run.tk[r, j, l]), bits(run.tv[r, j, l]),
                                               reset_first=bool(reset))
                assert_close(run.tout[l], ref, f"L_B {L_B} block {g} token step {j} layer {l}")
            assert (run.local.len == len_after).all()
        kind, n_after = next(ev)
        assert kind == "block"
        for l in range(w.n_layers):
            bt.bt_block_kv_append(run.cfg, run.block, l, run.bk[r, l], run.bv[r, l], n_new=1, dev_status=run.status)
            bt.bt_block_decode_attn(run.cfg, run.block, l, run.bq[r, l], run.bout[l], run.ws, dev_status=run.status)
            oracle.kv_append(ob[l], bits(run.bk[r, l]), bits(run.bv[r, l]))
            ref = oracle.block_decode_attn(ob[l], bits(run.bq[r, l][:, :, 0]))
            assert_close(run.bout[l][:, :, 0], ref, f"L_B {L_B} block step {g} layer {l}")
        assert (run.block.len == n_after).all()
    for l in range(w.n_layers):
        assert np.array_equal(bits(run.block.k[l]), ob[l].k) and np.array_equal(bits(run.block.v[l]), ob[l].v)
        gk, gv = local_kv_split(run.local.kv[l])
        n = int(ol[l].len[0])
        assert np.array_equal(gk[:, :, :n], ol[l].k[:, :, :n]) and np.array_equal(gv[:, :, :n], ol[l].v[:, :, :n])
    assert run.status.item() == 0
    # the driver's own loop (eager, then graph replays) must end in the same state
    for use_graph in (False, True):
        if use_graph:
            run.capture()
        run.generate()
        torch.cuda.synchronize()
        assert run.status.item() == 0
        assert (run.block.len == w.max_blocks).all() and (run.local.len == w.prefix_len + L_B - 1).all()
        for l in range(w.n_layers):
            assert np.array_equal(bits(run.block.k[l]), ob[l].k) and np.array_equal(bits(run.block.v[l]), ob[l].v)


def test_full_size_generation_l_b_4(bt):
    from paper_2406_02657_b200 import harness
    w = configs.sweep(4)
    run = harness.GenerationRun(w, fill=_fill(w.seed))
    run.capture()
    run.generate()
    torch.cuda.synchronize()
    assert run.status.item() == 0
    T, nb = w.prompt_blocks, w.gen_tokens // w.block_len
    assert (run.block.len == T + nb).all() and T + nb == w.max_blocks == 544
    assert (run.local.len == w.prefix_len + w.block_len - 1).all()
    last = (nb - 1) % run.ring
    bits = gen.torch_to_bits
    for l in (0, w.n_layers - 1):
        # cache rows are the prompt rows, then the ring's rows in turn, bit for bit (sampled)
        assert torch.equal(run.block.k[l, :, :, :T], run.pk[l])
        for g in (0, 1, 5, nb - 2, nb - 1):
            assert torch.equal(run.block.v[l, :, :, T + g], run.bv[g % run.ring, l, :, :, 0])
        seqs = [0, 255, 511]
        c = oracle.Cache(len(seqs), w.heads, w.max_blocks, w.head_dim)
        c.k[...] = bits(run.block.k[l][seqs])
        c.v[...] = bits(run.block.v[l][seqs])
        c.len[...] = w.max_blocks
        ref = oracle.block_decode_attn(c, bits(run.bq[last, l][seqs][:, :, 0]))
        assert_close(run.bout[l][seqs][:, :, 0], ref, f"last block step, layer {l}")
        # last token step of the last block: local cache holds the block's first L_B rows
        lc = oracle.Cache(len(seqs), w.heads, w.local_cap, w.head_dim)
        for j in range(w.block_len):
            ref = oracle.token_decode_attn(lc, bits(run.tq[last, j, l][seqs]), bits(run.tk[last, j, l][seqs]),
                                           bits(run.tv[last, j, l][seqs]), reset_first=(j == 0))
        assert_close(run.tout[l][seqs], ref, f"last token step, layer {l}")
