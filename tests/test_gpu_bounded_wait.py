"""The bounded waits of the kernels, shown to give up on a live GPU without anything in flight, and
the recovery rule for a workspace whose arrival counters a timed-out launch may have left non-zero."""
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


def test_bounded_waits_run_out_and_raise_timeout(bt):
    """bt_selftest_bounded_wait runs the decode kernels' poll-bounded wait and the prefill kernel's
    time-bounded wait on barriers nothing completes: both must give up, BT_DEV_TIMEOUT must be raised,
    a wait on a completed barrier must still succeed, and the context must stay usable."""
    st = status_word()
    report = torch.full((4,), 77, dtype=torch.int32, device="cuda")
    for _ in range(2):
        st.zero_()
        bt.bt_selftest_bounded_wait(report, st)
        torch.cuda.synchronize()
        r = report.cpu().numpy().view(np.uint32)
        assert r[0] == 1, "the poll-bounded wait did not give up"
        assert r[1] == 1, "the time-bounded wait did not give up"
        assert r[2] == 1, "a wait on a completed barrier failed"
        assert 150_000 <= r[3] < 50_000_000, f"time-bounded wait took {r[3]} ns (limit 0.2 ms)"
        assert st.item() == bt.BT_DEV_TIMEOUT
    # without a report buffer
    st.zero_()
    bt.bt_selftest_bounded_wait(None, st)
    assert st.item() == bt.BT_DEV_TIMEOUT
    # the context is intact: an ordinary call still works
    assert torch.ones(4, device="cuda").sum().item() == 4.0


@pytest.mark.parametrize("splits", [1, 3])
def test_workspace_init_restores_counters_left_by_a_timed_out_launch(bt, splits):
    """A launch that raised BT_DEV_TIMEOUT may leave arrival counts behind; the documented recovery is
    bt_workspace_init.  Leftovers are planted by hand (garbage in every counter), the workspace is
    initialised again, and a fused step must then give the oracle's result and exact lengths."""
    B, H, hd, N = 5, 3, 64, 200
    cfg = bt.make_config(B, H, hd, 4, 1, N, 1, decode_splits=splits)
    lens = np.array([199, 0, 64, 130, 17], np.int32)
    k, v = gen.normal_bf16_bits(611, 1, (B, H, N, hd)), gen.normal_bf16_bits(611, 2, (B, H, N, hd))
    q, kn, vn = (gen.normal_bf16_bits(611, 3 + i, (B, H, 1, hd)) for i in range(3))
    cache = bt.BlockCache(cfg)
    cache.k[0].copy_(to_dev(k))
    cache.v[0].copy_(to_dev(v))
    cache.len[0].copy_(torch.from_numpy(lens).cuda())
    ws = bt.alloc_workspace(cfg)
    ws.view(torch.int32).fill_(0x01010101)        # counters (and partials) as a dead launch might leave them
    bt.bt_workspace_init(cfg, ws)
    n_counters = B * H + B
    assert not ws.view(torch.int32)[-n_counters:].any()
    st = status_word()
    out = torch.empty((B, H, hd), dtype=torch.bfloat16, device="cuda")
    bt.bt_block_decode_step(cfg, cache, 0, to_dev(q), to_dev(kn), to_dev(vn), out, ws, dev_status=st)
    oc = oracle.Cache(B, H, N, hd)
    oc.k[...], oc.v[...], oc.len[...] = k, v, lens
    oracle.kv_append(oc, kn, vn)
    assert_close(out, oracle.block_decode_attn(oc, np.ascontiguousarray(q[:, :, 0])), "step after re-initialisation")
    assert cache.len[0].cpu().tolist() == oc.len.tolist() and st.item() == 0
    assert not ws.view(torch.int32)[-n_counters:].any()   # and the launch left them at zero again
