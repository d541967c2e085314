"""The C-ABI library loads, exports what include/bt.h declares, and rejects bad arguments
before launching anything (no GPU needed: every call here returns before a launch)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "bt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bt_[a-z0-9_]+)\s*\(", text)))


@pytest.fixture(scope="module")
def bt():
    import paper_2406_02657_b200 as bt
    return bt


def test_library_exports_every_declared_symbol(bt):
    names = declared_symbols()
    assert len(names) >= 11
    for n in names:
        assert hasattr(bt.lib(), n), f"{n} declared in bt.h but not exported"
        assert hasattr(bt, n) or n in ("bt_status_string",), f"{n} has no python binding"


def test_version_and_status_strings(bt):
    assert bt.bt_version() >= 100
    assert bt.status_string(0) == "BT_OK" and bt.status_string(4) == "BT_ERR_CAPACITY"


def test_split_choice_and_workspace(bt):
    big = bt.make_config(256, 16, 64, 4, 1, 512, 12)
    counters = lambda B, H: (B * H + B) * 4   # arrival counters: one per (b,h), one per sequence
    assert bt.bt_decode_splits(big) == 1 and bt.bt_workspace_bytes(big) == counters(256, 16)
    tiny = bt.make_config(4, 8, 64, 4, 1, 64, 2)
    s = bt.bt_decode_splits(tiny)
    assert s > 1 and bt.bt_workspace_bytes(tiny) == s * 4 * 8 * 68 * 4 + counters(4, 8)
    forced = bt.make_config(4, 8, 64, 4, 1, 64, 2, decode_splits=7)
    assert bt.bt_decode_splits(forced) == 7
    # the choice aims at about 512 work items of at least 128 rows (short caches: up to 4 parts of >= 16 rows)
    for (B, H, N), want in {(1, 16, 8192): 32, (1, 16, 2048): 16, (8, 16, 8192): 4, (16, 16, 4096): 2,
                            (64, 16, 4096): 1, (4, 8, 64): 4, (2, 2, 20): 1}.items():
        assert bt.bt_decode_splits(bt.make_config(B, H, 64, 4, 1, N, 1)) == want, (B, H, N)
    bad = bt.make_config(4, 8, 48, 4, 1, 64, 2)
    assert bt.bt_decode_splits(bad) == 0 and bt.bt_workspace_bytes(bad) == 0


def test_host_detectable_errors_return_before_launch(bt):
    L = bt.lib()
    fake = ctypes.c_void_p(0x1000)  # never dereferenced: each call below fails validation first
    cfg = bt.make_config(4, 8, 64, 4, 1, 64, 2)
    bc = bt.binding.bt_block_cache(0x1000, 0x1000, 0x1000)
    lc = bt.binding.bt_local_cache(0x1000, 0x1000)
    ref = ctypes.byref
    # null config / bad shapes
    assert L.bt_block_kv_append(None, ref(bc), 0, fake, fake, 1, None, None) == bt.BT_ERR_NULL
    assert L.bt_block_kv_append(ref(cfg), ref(bc), 2, fake, fake, 1, None, None) == bt.BT_ERR_SHAPE
    assert L.bt_block_kv_append(ref(cfg), ref(bc), -1, fake, fake, 1, None, None) == bt.BT_ERR_SHAPE
    assert L.bt_block_kv_append(ref(cfg), ref(bc), 0, None, fake, 1, None, None) == bt.BT_ERR_NULL
    assert L.bt_block_kv_append(ref(cfg), ref(bc), 0, fake, fake, 0, None, None) == bt.BT_ERR_SHAPE
    assert L.bt_block_kv_append(ref(cfg), ref(bc), 0, fake, fake, 65, None, None) == bt.BT_ERR_CAPACITY
    nullc = bt.binding.bt_block_cache(0, 0x1000, 0x1000)
    assert L.bt_block_kv_append(ref(cfg), ref(nullc), 0, fake, fake, 1, None, None) == bt.BT_ERR_NULL
    # unsupported head_dim / too many heads
    bad = bt.make_config(4, 8, 96, 4, 1, 64, 2)
    assert L.bt_block_decode_attn(ref(bad), ref(bc), 0, fake, fake, None, 0, None, None) == bt.BT_ERR_UNSUPPORTED
    many = bt.make_config(4, 64, 64, 4, 1, 64, 2)
    assert L.bt_block_decode_attn(ref(many), ref(bc), 0, fake, fake, None, 0, None, None) == bt.BT_ERR_UNSUPPORTED
    neg = bt.make_config(0, 8, 64, 4, 1, 64, 2)
    assert L.bt_block_decode_attn(ref(neg), ref(bc), 0, fake, fake, None, 0, None, None) == bt.BT_ERR_SHAPE
    # workspace too small when the row range is split
    assert L.bt_block_decode_attn(ref(cfg), ref(bc), 0, fake, fake, None, 0, None, None) == bt.BT_ERR_WORKSPACE
    assert L.bt_block_decode_attn(ref(cfg), ref(bc), 0, fake, fake, fake, 16, None, None) == bt.BT_ERR_WORKSPACE
    # the fused step needs one always; the initialiser checks its size too
    assert L.bt_block_decode_step(ref(cfg), ref(bc), 0, fake, fake, fake, fake, None, 0, None, None) == bt.BT_ERR_WORKSPACE
    assert L.bt_block_decode_step(ref(cfg), ref(bc), 0, fake, None, fake, fake, fake, 1 << 20, None, None) == bt.BT_ERR_NULL
    assert L.bt_workspace_init(ref(cfg), fake, 16, None) == bt.BT_ERR_WORKSPACE
    assert L.bt_workspace_init(ref(cfg), None, 1 << 20, None) == bt.BT_ERR_NULL
    assert L.bt_block_decode_attn(ref(cfg), ref(bc), 0, None, fake, fake, 1 << 20, None, None) == bt.BT_ERR_NULL
    # local cache
    assert L.bt_local_kv_reset(ref(cfg), None, 0, None, None) == bt.BT_ERR_NULL
    assert L.bt_local_kv_append(ref(cfg), ref(lc), 0, fake, fake, 6, None, None) == bt.BT_ERR_CAPACITY
    assert L.bt_token_decode_attn(ref(cfg), ref(lc), 0, fake, fake, None, 1, 0, None, fake, None, None) == bt.BT_ERR_NULL
    assert L.bt_token_decode_attn(ref(cfg), ref(lc), 0, fake, None, None, 6, 0, None, fake, None, None) == bt.BT_ERR_CAPACITY
    assert L.bt_token_decode_attn(ref(cfg), ref(lc), 0, fake, fake, fake, 6, 0, None, fake, None, None) == bt.BT_ERR_CAPACITY
    assert L.bt_token_decode_attn(ref(cfg), ref(lc), 0, fake, fake, fake, 0, 0, None, fake, None, None) == bt.BT_ERR_SHAPE
    assert L.bt_token_decode_attn(ref(cfg), ref(lc), 0, fake, fake, fake, 1, 0, None, None, None, None) == bt.BT_ERR_NULL
    # prefill
    assert L.bt_block_prefill_attn(ref(cfg), fake, fake, fake, 0, 8, fake, None, None) == bt.BT_ERR_SHAPE
    assert L.bt_block_prefill_attn(ref(cfg), fake, fake, fake, 16, 8, fake, None, None) == bt.BT_ERR_SHAPE
    assert L.bt_block_prefill_attn(ref(cfg), fake, None, fake, 8, 8, fake, None, None) == bt.BT_ERR_NULL
    # projections
    assert L.bt_prefix_project(ref(cfg), fake, None, None, fake, None, None) == bt.BT_ERR_NULL
    assert L.bt_prefix_project(ref(bad), fake, fake, None, fake, None, None) == bt.BT_ERR_UNSUPPORTED
    assert L.bt_block_qkv_project_append(ref(cfg), ref(bc), 0, fake, 65, fake, None, fake, None, None) == bt.BT_ERR_CAPACITY
    assert L.bt_block_qkv_project_append(ref(cfg), ref(bc), 0, fake, 0, fake, None, fake, None, None) == bt.BT_ERR_SHAPE
    assert L.bt_block_qkv_project_append(ref(cfg), ref(nullc), 0, fake, 1, fake, None, fake, None, None) == bt.BT_ERR_NULL
    assert L.bt_block_qkv_project_append(ref(cfg), ref(bc), 2, fake, 1, fake, None, fake, None, None) == bt.BT_ERR_SHAPE
    assert L.bt_local_qkv_project_append(ref(cfg), ref(lc), 0, fake, 6, fake, None, 0, None, fake, None, None) == bt.BT_ERR_CAPACITY
    assert L.bt_local_qkv_project_append(ref(cfg), ref(lc), 0, fake, 1, None, None, 0, None, fake, None, None) == bt.BT_ERR_NULL
    assert L.bt_local_qkv_project_append(ref(cfg), ref(lc), 0, fake, 1, fake, ctypes.c_void_p(0x1002), 0, None, fake, None, None) \
        == bt.BT_ERR_UNSUPPORTED
    # host-driven step
    assert L.bt_block_decode_step_host(ref(cfg), ref(bc), 0, None, fake, fake, fake, fake, fake, fake, fake,
                                       None, 0, None, None) == bt.BT_ERR_NULL


def test_misaligned_pointers_are_refused_before_launch(bt):
    """The kernels use 16-byte loads, stores and copies: a pointer off a 16-byte boundary (a 2-byte-aligned
    bf16 view, say) would fault on the device, so every entry point refuses it on the host.  Fake
    addresses: nothing is launched, nothing is dereferenced."""
    L = bt.lib()
    ref = ctypes.byref
    ok, odd, odd4 = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x1002), ctypes.c_void_p(0x1008)
    cfg = bt.make_config(4, 8, 64, 4, 1, 64, 2, decode_splits=1)
    split = bt.make_config(4, 8, 64, 4, 1, 64, 2, decode_splits=2)
    bc = bt.binding.bt_block_cache(0x1000, 0x1000, 0x1000)
    lc = bt.binding.bt_local_cache(0x1000, 0x1000)
    U = bt.BT_ERR_UNSUPPORTED
    big = 1 << 20
    for bad in (odd, odd4):
        assert L.bt_block_kv_append(ref(cfg), ref(bc), 0, bad, ok, 1, None, None) == U
        assert L.bt_block_kv_append(ref(cfg), ref(bc), 0, ok, bad, 1, None, None) == U
        assert L.bt_block_decode_attn(ref(cfg), ref(bc), 0, bad, ok, None, 0, None, None) == U
        assert L.bt_block_decode_attn(ref(cfg), ref(bc), 0, ok, bad, None, 0, None, None) == U
        assert L.bt_block_decode_attn(ref(split), ref(bc), 0, ok, ok, bad, big, None, None) == U
        assert L.bt_block_decode_attn_noalloc(ref(cfg), ref(bc), 0, bad, ok, None, None) == U
        assert L.bt_block_decode_step(ref(cfg), ref(bc), 0, ok, bad, ok, ok, ok, big, None, None) == U
        assert L.bt_block_decode_step(ref(cfg), ref(bc), 0, ok, ok, ok, ok, bad, big, None, None) == U
        assert L.bt_block_decode_step_multi(ref(cfg), ref(bc), 0, ok, ok, bad, 2, ok, ok, big, None, None) == U
        assert L.bt_block_decode_step_host(ref(cfg), ref(bc), 0, ok, ok, ok, ok, ok, bad, ok, ok, ok, big, None, None) == U
        assert L.bt_local_kv_append(ref(cfg), ref(lc), 0, bad, ok, 1, None, None) == U
        assert L.bt_token_decode_attn(ref(cfg), ref(lc), 0, bad, ok, ok, 1, 0, None, ok, None, None) == U
        assert L.bt_token_decode_attn(ref(cfg), ref(lc), 0, ok, ok, ok, 1, 0, None, bad, None, None) == U
        assert L.bt_block_prefill_attn(ref(cfg), ok, bad, ok, 8, 8, ok, None, None) == U
        assert L.bt_workspace_init(ref(cfg), bad, big, None) == U
    for k, v, ln in ((0x1002, 0x1000, 0x1000), (0x1000, 0x1008, 0x1000), (0x1000, 0x1000, 0x1002)):
        mis = bt.binding.bt_block_cache(k, v, ln)
        assert L.bt_block_decode_attn(ref(cfg), ref(mis), 0, ok, ok, None, 0, None, None) == U
        assert L.bt_block_kv_append(ref(cfg), ref(mis), 0, ok, ok, 1, None, None) == U
    for kv, ln in ((0x1004, 0x1000), (0x1000, 0x1001)):
        mis = bt.binding.bt_local_cache(kv, ln)
        assert L.bt_token_decode_attn(ref(cfg), ref(mis), 0, ok, ok, ok, 1, 0, None, ok, None, None) == U
    assert L.bt_local_kv_reset(ref(cfg), ref(bt.binding.bt_local_cache(0x1000, 0x1002)), 0, None, None) == U
    # a misaligned status word (uint32) is refused too
    assert L.bt_block_decode_attn(ref(cfg), ref(bc), 0, ok, ok, None, 0, ctypes.c_void_p(0x1002), None) == U
    # the prefill never changes kernels on its own: the CUDA-core kernel must be asked for, and wants aligned pointers too
    plain = bt.make_config(4, 8, 64, 4, 1, 64, 2, prefill_plain=1)
    assert L.bt_block_prefill_attn(ref(plain), ok, odd, ok, 8, 8, ok, None, None) == U


def test_refused_calls_enqueue_nothing(bt):
    """The two entry points that enqueue something before their kernel (host copies; the memset of the
    shared scratch) judge every argument first: a NULL cache comes back as BT_ERR_NULL although the
    copy sources / the scratch would have been usable."""
    L = bt.lib()
    ref = ctypes.byref
    ok = ctypes.c_void_p(0x1000)
    cfg = bt.make_config(4, 8, 64, 4, 1, 64, 2)
    assert bt.bt_decode_splits(cfg) > 1
    for k, v, ln in ((0, 0x1000, 0x1000), (0x1000, 0, 0x1000), (0x1000, 0x1000, 0)):
        nullc = bt.binding.bt_block_cache(k, v, ln)
        assert L.bt_block_decode_step_host(ref(cfg), ref(nullc), 0, ok, ok, ok, ok, ok, ok, ok, ok, ok, 1 << 20, None, None) \
            == bt.BT_ERR_NULL
        assert L.bt_block_decode_attn_noalloc(ref(cfg), ref(nullc), 0, ok, ok, None, None) == bt.BT_ERR_NULL
    bc = bt.binding.bt_block_cache(0x1000, 0x1000, 0x1000)
    assert L.bt_block_decode_step_host(ref(cfg), None, 0, ok, ok, ok, ok, ok, ok, ok, ok, ok, 1 << 20, None, None) == bt.BT_ERR_NULL
    assert L.bt_block_decode_step_host(ref(cfg), ref(bc), 0, ok, ok, ok, ok, ok, ok, ok, ok, None, 0, None, None) == bt.BT_ERR_WORKSPACE
    assert L.bt_block_decode_step_host(ref(cfg), ref(bc), 5, ok, ok, ok, ok, ok, ok, ok, ok, ok, 1 << 20, None, None) == bt.BT_ERR_SHAPE
    assert L.bt_block_decode_attn_noalloc(ref(cfg), ref(bc), 0, None, ok, None, None) == bt.BT_ERR_NULL
    assert L.bt_block_decode_attn_noalloc(ref(cfg), ref(bc), 7, ok, ok, None, None) == bt.BT_ERR_SHAPE
    assert L.bt_selftest_bounded_wait(None, None, None) == bt.BT_ERR_NULL


def test_oracle_is_not_imported_by_the_product():
    pkg = os.path.join(ROOT, "paper_2406_02657_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src, f"{f} mentions the oracle"
