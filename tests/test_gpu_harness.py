"""The workload drivers bench.py times: each one captured as a CUDA graph and replayed at a small size, so
that a driver that cannot capture or replay is caught here and not in a benchmark run."""
import pytest
import torch

from workloads import configs, gen

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def harness():
    from paper_2406_02657_b200 import harness
    assert torch.cuda.is_available()
    return harness


def _fill(w):
    return lambda tid, shape: gen.normal_bf16_device(w.seed, tid, shape, device="cuda")


def test_block_and_dense_decode_drivers(harness):
    w = configs.scaled(configs.BLOCK_DECODE, batch=8, n_layers=2)
    run = harness.BlockDecodeStep(w, fill=_fill(w))
    run.capture()
    run.replay(), run.replay_attn(), run.replay_timed()
    run.capture_host()
    run.replay_host()
    torch.cuda.synchronize()
    assert run.status.item() == 0 and (run.cache.len == w.ctx_blocks).all()
    d = configs.scaled(configs.DENSE_DECODE, batch=8, n_layers=2)
    run = harness.DenseDecodeStep(d, fill=_fill(d))
    run.capture()
    run.replay(), run.replay()
    torch.cuda.synchronize()
    assert run.status.item() == 0 and (run.cache.len == d.ctx_blocks).all()


def test_token_prefill_and_generation_drivers(harness):
    for P in (1, 2, 8):
        w = configs.scaled(configs.TOKEN_DECODE, batch=64, n_layers=2, prefix_len=P)
        run = harness.TokenDecodeRun(w, fill=_fill(w))
        run.capture()
        run.replay(), run.replay()
        torch.cuda.synchronize()
        assert run.status.item() == 0 and (run.cache.len == P + w.block_len - 1).all()
    w = configs.scaled(configs.BLOCK_PREFILL, batch=2, n_layers=2)
    run = harness.PrefillRun(w, fill=_fill(w))
    run.capture()
    run.replay(), run.replay_timed()
    torch.cuda.synchronize()
    assert torch.isfinite(run.out.float()).all()
    g = configs.scaled(configs.sweep(4), batch=16, n_layers=2, gen_tokens=64, max_blocks=(128 + 64) // 4)
    run = harness.GenerationRun(g, fill=_fill(g))
    run.capture()
    run.generate()
    torch.cuda.synchronize()
    assert run.status.item() == 0 and (run.block.len == g.max_blocks).all()


def test_projection_drivers(harness):
    for name, kind in (("qkv_project_token", "qkv_token"), ("qkv_project_block", "qkv_block"), ("prefix_project", "prefix")):
        w = configs.scaled(configs.BY_NAME[name], batch=160, n_layers=2)
        run = harness.ProjectRun(w, kind, fill=_fill(w), sets=2)
        run.capture()
        run.replay(), run.replay()
        torch.cuda.synchronize()
        assert run.status.item() == 0
    w = configs.scaled(configs.TOKEN_DECODE_PROJECTED, batch=160, n_layers=2)
    run = harness.ProjectedTokenRun(w, fill=_fill(w))
    run.capture()
    run.replay(), run.replay()
    torch.cuda.synchronize()
    assert run.status.item() == 0 and (run.cache.len == w.prefix_len + w.block_len - 1).all()
