"""GPU parity at the full workload sizes, in the launch configuration bench.py times (the harness
drivers): the CUDA path runs the whole workload, the oracle recomputes sampled sequences from
exactly the bytes the GPU used (copied back), and everything integer (lengths, appended rows) is
checked bit-exactly over the full size."""
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


def _fill(w):
    return lambda tid, shape: gen.normal_bf16_device(w.seed, tid, shape, device="cuda")


def test_block_decode_step_full_size(bt):
    """benchmark configs[1]: batch 256, 16 heads, head_dim 64, 512 rows after the append, 12 layers."""
    from paper_2406_02657_b200 import harness
    w = configs.BLOCK_DECODE
    run = harness.BlockDecodeStep(w, fill=_fill(w))
    k_before = {l: gen.torch_to_bits(run.cache.k[l, :, :, w.ctx_blocks - 1]) for l in (0, 5)}  # the row the append overwrites
    run.step()
    torch.cuda.synchronize()
    assert run.status.item() == 0
    assert (run.cache.len == w.ctx_blocks).all()  # every (layer, sequence) advanced by exactly one row
    # the appended rows are the new rows, bit for bit, over the whole batch
    for l in range(w.n_layers):
        assert torch.equal(run.cache.k[l, :, :, w.ctx_blocks - 1], run.k_new[l, :, :, 0])
        assert torch.equal(run.cache.v[l, :, :, w.ctx_blocks - 1], run.v_new[l, :, :, 0])
    assert not np.array_equal(k_before[0], gen.torch_to_bits(run.k_new[0, :, :, 0]))  # the check above is not vacuous
    # sampled sequences, every head, first / middle / last layer: outputs against the oracle
    seqs = [0, 1, 97, 128, 254, 255]
    for l in (0, 5, w.n_layers - 1):
        c = oracle.Cache(len(seqs), w.heads, w.max_blocks, w.head_dim)
        c.k[...] = gen.torch_to_bits(run.cache.k[l][seqs])
        c.v[...] = gen.torch_to_bits(run.cache.v[l][seqs])
        c.len[...] = w.ctx_blocks
        ref = oracle.block_decode_attn(c, gen.torch_to_bits(run.q[l][seqs][:, :, 0]))
        assert_close(run.out[l][seqs][:, :, 0], ref, f"full-size block decode layer {l}")


@pytest.mark.parametrize("batch", [64, 1])
def test_block_decode_step_long_context(bt, batch):
    """The 16K-token context (4096 block rows): the bench batch, unsplit, and a single sequence, whose
    row ranges are split across the GPU and merged inside the launch."""
    from paper_2406_02657_b200 import harness
    w = configs.scaled(configs.BLOCK_DECODE_16K, batch=batch, n_layers=2)
    run = harness.BlockDecodeStep(w, fill=_fill(w))
    assert (bt.bt_decode_splits(run.cfg) > 1) == (batch == 1)
    for _ in range(2):   # twice on the same workspace
        run.rewind()
        run.out.zero_()
        run.step()
        torch.cuda.synchronize()
        assert run.status.item() == 0 and (run.cache.len == w.ctx_blocks).all()
        assert torch.equal(run.cache.k[:, :, :, w.ctx_blocks - 1], run.k_new[:, :, :, 0])
        assert torch.equal(run.cache.v[:, :, :, w.ctx_blocks - 1], run.v_new[:, :, :, 0])
        seqs = sorted({0, batch // 2, batch - 1})
        for l in range(w.n_layers):
            c = oracle.Cache(len(seqs), w.heads, w.max_blocks, w.head_dim)
            c.k[...] = gen.torch_to_bits(run.cache.k[l][seqs])
            c.v[...] = gen.torch_to_bits(run.cache.v[l][seqs])
            c.len[...] = w.ctx_blocks
            ref = oracle.block_decode_attn(c, gen.torch_to_bits(run.q[l][seqs][:, :, 0]))
            assert_close(run.out[l][seqs][:, :, 0], ref, f"16K-context block decode, batch {batch}, layer {l}")


def test_dense_decode_step_full_size(bt):
    """The densified block decoder at the bench shape: batch 256, 16 heads, 2048 rows after a step that
    appends 4 rows and runs 4 queries per (sequence, head); two of the 12 layers, twice."""
    from paper_2406_02657_b200 import harness
    w = configs.scaled(configs.DENSE_DECODE, n_layers=2)
    m = w.block_len
    run = harness.DenseDecodeStep(w, fill=_fill(w))
    seqs = [0, 101, 255]
    for _ in range(2):
        run.rewind()
        run.out.zero_()
        torch.cuda.synchronize()
        before = {l: (gen.torch_to_bits(run.cache.k[l][seqs]), gen.torch_to_bits(run.cache.v[l][seqs])) for l in range(w.n_layers)}
        run.step()
        torch.cuda.synchronize()
        assert run.status.item() == 0 and (run.cache.len == w.ctx_blocks).all()
        assert torch.equal(run.cache.k[:, :, :, w.ctx_blocks - m:], run.k_new)   # the appended rows, whole batch
        assert torch.equal(run.cache.v[:, :, :, w.ctx_blocks - m:], run.v_new)
        for l in range(w.n_layers):
            c = oracle.Cache(len(seqs), w.heads, w.max_blocks, w.head_dim)
            c.k[...], c.v[...] = before[l]
            c.len[...] = w.ctx_blocks - m
            ref = oracle.block_decode_step_multi(c, *(gen.torch_to_bits(x[l][seqs]) for x in (run.q, run.k_new, run.v_new)))
            assert_close(run.out[l][seqs], ref, f"full-size dense decode layer {l}", p_bf16=True)
            assert np.array_equal(gen.torch_to_bits(run.cache.k[l][seqs]), c.k)


def test_block_decode_step_through_host_buffers(bt):
    """The e2e path of bench.py: the same step driven from pinned host buffers through
    bt_block_decode_step_host (per-layer calls on several streams) gives the device-resident step's
    outputs bit for bit, and the same cache."""
    from paper_2406_02657_b200 import harness
    w = configs.scaled(configs.BLOCK_DECODE, batch=64, n_layers=5)
    run = harness.BlockDecodeStep(w, fill=_fill(w))
    run.step()
    torch.cuda.synchronize()
    want_out, want_k = run.out.clone(), run.cache.k.clone()
    run.rewind()
    run.cache.k[:, :, :, w.ctx_blocks - 1].zero_()   # the row the step appends
    run.out.zero_()
    run.step_host()
    torch.cuda.synchronize()
    assert run.status.item() == 0 and (run.cache.len == w.ctx_blocks).all()
    assert torch.equal(run.out, want_out) and torch.equal(run.cache.k, want_k)
    assert torch.equal(run._host["out"], want_out.cpu())   # and the host copy of the result
    # the same step as one CUDA-graph replay (copies included), as bench.py times it
    run.capture_host()
    run.cache.k[:, :, :, w.ctx_blocks - 1].zero_()
    run.out.zero_()
    run._host["out"].zero_()
    run.replay_host()
    torch.cuda.synchronize()
    assert run.status.item() == 0 and (run.cache.len == w.ctx_blocks).all()
    assert torch.equal(run.out, want_out) and torch.equal(run.cache.k, want_k)
    assert torch.equal(run._host["out"], want_out.cpu())


def test_token_decode_full_size_two_blocks(bt):
    """benchmark configs[2]: 4096 sequences, 12 layers, local cache 1 prefix + up to L_B rows; two
    blocks of consecutive token steps, lengths against the integer schedule model at full size."""
    from paper_2406_02657_b200 import harness
    w = configs.TOKEN_DECODE
    run = harness.TokenDecodeRun(w, fill=_fill(w))
    seqs = [0, 5, 2047, 4095]
    layers = (0, w.n_layers - 1)
    ocache = {l: oracle.Cache(len(seqs), w.heads, w.local_cap, w.head_dim) for l in layers}
    n_steps = 2 * w.block_len
    sched = schedule.token_step_schedule(w.block_len, w.prefix_len, n_steps)
    for t in range(n_steps):
        r = t % run.ring
        run.token_step()
        torch.cuda.synchronize()
        reset, n_app, len_after = sched[t]
        assert (run.cache.len == len_after).all(), f"step {t}: lengths differ from the schedule model"
        for l in layers:
            q, k, v = (gen.torch_to_bits(x[r, l][seqs]) for x in (run.q, run.k_new, run.v_new))
            ref = oracle.token_decode_attn(ocache[l], q, k, v, reset_first=bool(reset))
            assert_close(run.out[l][seqs], ref, f"full-size token step {t} layer {l}")
            assert np.array_equal(ocache[l].len, np.full(len(seqs), len_after, np.int32))
            gk, gv = local_kv_split(run.cache.kv[l][seqs])
            n = len_after
            assert np.array_equal(gk[:, :, :n], ocache[l].k[:, :, :n]) and np.array_equal(gv[:, :, :n], ocache[l].v[:, :, :n])
    assert run.status.item() == 0


def test_token_decode_full_batch_prefix_length_two(bt):
    """The paper's main setting P = 2 at the full batch: a block starts with a two-row causal prefix step."""
    from paper_2406_02657_b200 import harness
    w = configs.scaled(configs.TOKEN_DECODE, prefix_len=2, n_layers=2)
    run = harness.TokenDecodeRun(w, fill=_fill(w))
    seqs = [0, 7, 2048, 4095]
    ocache = {l: oracle.Cache(len(seqs), w.heads, w.local_cap, w.head_dim) for l in range(w.n_layers)}
    n_steps = 2 * w.block_len
    sched = schedule.token_step_schedule(w.block_len, w.prefix_len, n_steps)
    for t in range(n_steps):
        r = t % run.ring
        first = t % w.block_len == 0
        run.token_step()
        torch.cuda.synchronize()
        reset, n_app, len_after = sched[t]
        assert n_app == (w.prefix_len if first else 1)
        assert (run.cache.len == len_after).all(), f"step {t}: lengths differ from the schedule model"
        src = (run.q, run.k_new, run.v_new, run.out) if first else (run.q1, run.k1, run.v1, run.out1)
        for l in range(w.n_layers):
            q, k, v = (gen.torch_to_bits(x[r, l][seqs]) for x in src[:3])
            ref = oracle.token_decode_attn(ocache[l], q, k, v, reset_first=bool(reset))
            assert_close(src[3][l][seqs], ref, f"P=2 token step {t} layer {l}")
            gk, gv = local_kv_split(run.cache.kv[l][seqs])
            assert np.array_equal(gk[:, :, :len_after], ocache[l].k[:, :, :len_after])
            assert np.array_equal(gv[:, :, :len_after], ocache[l].v[:, :, :len_after])
    assert run.status.item() == 0


def test_block_prefill_full_size(bt):
    """benchmark configs[3]: batch 32, 512 prompt blocks, 16 heads, head_dim 128, 12 layers."""
    from paper_2406_02657_b200 import harness
    w = configs.BLOCK_PREFILL
    run = harness.PrefillRun(w, fill=_fill(w))
    run.out.fill_(float("nan"))
    run.step()
    torch.cuda.synchronize()
    assert torch.isfinite(run.out.float()).all()  # every row of every layer was written
    for l, b, h in ((0, 0, 0), (0, 31, 15), (6, 13, 7), (11, 31, 0), (11, 5, 15)):
        q, k, v = (gen.torch_to_bits(x[l, b:b + 1, h:h + 1]) for x in (run.q, run.k, run.v))
        ref = oracle.block_prefill_attn(q, k, v)
        assert_close(run.out[l, b:b + 1, h:h + 1], ref, f"full-size prefill layer {l} b {b} h {h}", p_bf16=True)


def test_block_prefill_8k_prompt_full_size(bt):
    """The 8K-prompt case (2048 prompt blocks, batch 8, 16 heads, head_dim 128), two of the 12 layers:
    every row written, sampled (sequence, head) pairs against the oracle."""
    from paper_2406_02657_b200 import harness
    w = configs.scaled(configs.BLOCK_PREFILL_8K, n_layers=2)
    run = harness.PrefillRun(w, fill=_fill(w))
    run.out.fill_(float("nan"))
    run.step()
    torch.cuda.synchronize()
    assert torch.isfinite(run.out.float()).all()
    for l, b, h in ((0, 0, 0), (0, 7, 15), (1, 3, 8), (1, 7, 0)):
        q, k, v = (gen.torch_to_bits(x[l, b:b + 1, h:h + 1]) for x in (run.q, run.k, run.v))
        ref = oracle.block_prefill_attn(q, k, v)
        assert_close(run.out[l, b:b + 1, h:h + 1], ref, f"8K-prompt prefill layer {l} b {b} h {h}", p_bf16=True)


def test_block_prefill_many_items_ragged_last_tile(bt):
    """A launch too large for the host-made item table (768 (sequence, head) pairs x 7 pairs of query tiles), so
    the CTAs walk the items round robin, with a prompt that ends half way into its last query tile (1600 blocks =
    12.5 tiles): every row written, sampled (sequence, head) pairs against the oracle."""
    from paper_2406_02657_b200 import harness
    w = configs.scaled(configs.BLOCK_PREFILL, batch=48, prompt_blocks=1600, max_blocks=1600, n_layers=1)
    run = harness.PrefillRun(w, fill=_fill(w))
    run.out.fill_(float("nan"))
    run.step()
    torch.cuda.synchronize()
    assert torch.isfinite(run.out.float()).all()
    for l, b, h in ((0, 0, 0), (0, 47, 15), (0, 23, 9)):
        q, k, v = (gen.torch_to_bits(x[l, b:b + 1, h:h + 1]) for x in (run.q, run.k, run.v))
        ref = oracle.block_prefill_attn(q, k, v)
        assert_close(run.out[l, b:b + 1, h:h + 1], ref, f"many-item prefill b {b} h {h}", p_bf16=True)
