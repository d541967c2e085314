"""Thin ctypes binding of libbt.so: argument marshalling only.

Function names and argument order mirror ``include/bt.h``.  Tensors are torch CUDA
tensors (torch is used for device memory and streams only); every step of the
attention path runs inside the library's kernels.  There is no fallback: if the
shared library is missing and cannot be built, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

BT_OK, BT_ERR_NULL, BT_ERR_SHAPE, BT_ERR_UNSUPPORTED, BT_ERR_CAPACITY, BT_ERR_WORKSPACE, BT_ERR_CUDA = range(7)
BT_DEV_OK, BT_DEV_OVERFLOW, BT_DEV_EMPTY, BT_DEV_TIMEOUT = 0, 1, 2, 4

EXPORTS = [
    "bt_version", "bt_status_string", "bt_decode_splits", "bt_workspace_bytes", "bt_block_kv_append",
    "bt_block_decode_attn", "bt_local_kv_reset", "bt_local_kv_append", "bt_token_decode_attn",
    "bt_block_prefill_attn", "bt_block_decode_step_host", "bt_block_decode_attn_noalloc",
    "bt_workspace_init", "bt_block_decode_step", "bt_block_decode_step_multi", "bt_selftest_bounded_wait",
    "bt_prefix_project", "bt_block_qkv_project_append", "bt_local_qkv_project_append",
]


class bt_config(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("block_len", ctypes.c_int32), ("prefix_len", ctypes.c_int32), ("max_blocks", ctypes.c_int32),
                ("n_layers", ctypes.c_int32), ("decode_splits", ctypes.c_int32), ("softmax_scale", ctypes.c_float),
                ("prefill_plain", ctypes.c_int32)]


class bt_block_cache(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("len", ctypes.c_void_p)]


class bt_local_cache(ctypes.Structure):
    _fields_ = [("kv", ctypes.c_void_p), ("len", ctypes.c_void_p)]


class BtError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


def _load() -> ctypes.CDLL:
    path = _build.LIB
    if not os.path.exists(path) or not _build.up_to_date():
        path = _build.build()  # raises if nvcc is unavailable: no silent fallback
    lib = ctypes.CDLL(path)
    vp, i32, u64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    cfgp = ctypes.POINTER(bt_config)
    lib.bt_version.restype = ctypes.c_int
    lib.bt_status_string.restype = ctypes.c_char_p
    lib.bt_status_string.argtypes = [ctypes.c_int]
    lib.bt_decode_splits.restype = ctypes.c_int
    lib.bt_decode_splits.argtypes = [cfgp]
    lib.bt_workspace_bytes.restype = ctypes.c_size_t
    lib.bt_workspace_bytes.argtypes = [cfgp]
    lib.bt_block_kv_append.argtypes = [cfgp, ctypes.POINTER(bt_block_cache), i32, vp, vp, i32, vp, vp]
    lib.bt_block_decode_attn.argtypes = [cfgp, ctypes.POINTER(bt_block_cache), i32, vp, vp, vp, u64, vp, vp]
    lib.bt_workspace_init.argtypes = [cfgp, vp, u64, vp]
    lib.bt_block_decode_step.argtypes = [cfgp, ctypes.POINTER(bt_block_cache), i32, vp, vp, vp, vp, vp, u64, vp, vp]
    lib.bt_block_decode_step_multi.argtypes = [cfgp, ctypes.POINTER(bt_block_cache), i32, vp, vp, vp, i32, vp, vp, u64, vp, vp]
    lib.bt_local_kv_reset.argtypes = [cfgp, ctypes.POINTER(bt_local_cache), i32, vp, vp]
    lib.bt_local_kv_append.argtypes = [cfgp, ctypes.POINTER(bt_local_cache), i32, vp, vp, i32, vp, vp]
    lib.bt_token_decode_attn.argtypes = [cfgp, ctypes.POINTER(bt_local_cache), i32, vp, vp, vp, i32, i32, vp, vp, vp, vp]
    lib.bt_block_prefill_attn.argtypes = [cfgp, vp, vp, vp, i32, ctypes.c_int64, vp, vp, vp]
    lib.bt_block_decode_step_host.argtypes = [cfgp, ctypes.POINTER(bt_block_cache), i32, vp, vp, vp, vp,
                                              vp, vp, vp, vp, vp, u64, vp, vp]
    lib.bt_block_decode_attn_noalloc.argtypes = [cfgp, ctypes.POINTER(bt_block_cache), i32, vp, vp, vp, vp]
    lib.bt_selftest_bounded_wait.argtypes = [vp, vp, vp]
    lib.bt_prefix_project.argtypes = [cfgp, vp, vp, vp, vp, vp, vp]
    lib.bt_block_qkv_project_append.argtypes = [cfgp, ctypes.POINTER(bt_block_cache), i32, vp, i32, vp, vp, vp, vp, vp]
    lib.bt_local_qkv_project_append.argtypes = [cfgp, ctypes.POINTER(bt_local_cache), i32, vp, i32, vp, vp, i32, vp, vp, vp, vp]
    for name in EXPORTS[4:]:
        getattr(lib, name).restype = ctypes.c_int
    return lib


_lib = _load()


def lib() -> ctypes.CDLL:
    return _lib


def status_string(code: int) -> str:
    return _lib.bt_status_string(int(code)).decode()


def _ptr(t):
    if t is None:
        return None
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, torch.cuda.Stream):
        return ctypes.c_void_p(stream.cuda_stream)
    return ctypes.c_void_p(int(stream))


def _check(code: int, where: str):
    if code != BT_OK:
        raise BtError(code, where)


def make_config(batch, heads, head_dim, block_len, prefix_len, max_blocks, n_layers, decode_splits=0,
                softmax_scale=0.0, prefill_plain=0) -> bt_config:
    return bt_config(batch, heads, head_dim, block_len, prefix_len, max_blocks, n_layers, decode_splits,
                     softmax_scale, prefill_plain)


class BlockCache:
    """Caller-owned block KV cache: k, v bf16 [layers,B,H,N_max,hd], len int32 [layers,B]."""

    def __init__(self, cfg: bt_config, device="cuda", k=None, v=None, length=None):
        shape = (cfg.n_layers, cfg.batch, cfg.heads, cfg.max_blocks, cfg.head_dim)
        self.k = torch.zeros(shape, dtype=torch.bfloat16, device=device) if k is None else k
        self.v = torch.zeros(shape, dtype=torch.bfloat16, device=device) if v is None else v
        self.len = torch.zeros((cfg.n_layers, cfg.batch), dtype=torch.int32, device=device) if length is None else length
        assert self.k.shape == shape and self.v.shape == shape and self.k.is_contiguous() and self.v.is_contiguous()
        self.c = bt_block_cache(self.k.data_ptr(), self.v.data_ptr(), self.len.data_ptr())


class LocalCache:
    """Caller-owned local KV cache: kv bf16 [layers,B,H,P+L_B,2,hd], len int32 [layers,B]."""

    def __init__(self, cfg: bt_config, device="cuda"):
        cap = cfg.prefix_len + cfg.block_len
        self.kv = torch.zeros((cfg.n_layers, cfg.batch, cfg.heads, cap, 2, cfg.head_dim), dtype=torch.bfloat16,
                              device=device)
        self.len = torch.zeros((cfg.n_layers, cfg.batch), dtype=torch.int32, device=device)
        self.c = bt_local_cache(self.kv.data_ptr(), self.len.data_ptr())


def bt_version() -> int:
    return _lib.bt_version()


def bt_decode_splits(cfg) -> int:
    return _lib.bt_decode_splits(ctypes.byref(cfg))


def bt_workspace_bytes(cfg) -> int:
    return _lib.bt_workspace_bytes(ctypes.byref(cfg))


def bt_workspace_init(cfg, workspace, stream=None):
    _check(_lib.bt_workspace_init(ctypes.byref(cfg), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                  _stream(stream)), "bt_workspace_init")


def alloc_workspace(cfg, device="cuda"):
    """A workspace for the decode calls of this config, initialised (counters zeroed) and ready."""
    n = bt_workspace_bytes(cfg)
    ws = torch.empty((max(n, 4) + 3) // 4, dtype=torch.float32, device=device)
    bt_workspace_init(cfg, ws)
    return ws


def bt_block_kv_append(cfg, cache: BlockCache, layer, k_new, v_new, n_new=None, dev_status=None, stream=None):
    n_new = k_new.shape[2] if n_new is None else n_new
    _check(_lib.bt_block_kv_append(ctypes.byref(cfg), ctypes.byref(cache.c), layer, _ptr(k_new), _ptr(v_new),
                                   n_new, _ptr(dev_status), _stream(stream)), "bt_block_kv_append")


def bt_block_decode_attn(cfg, cache: BlockCache, layer, q, out, workspace=None, dev_status=None, stream=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.bt_block_decode_attn(ctypes.byref(cfg), ctypes.byref(cache.c), layer, _ptr(q), _ptr(out),
                                     _ptr(workspace), ws_bytes, _ptr(dev_status), _stream(stream)),
           "bt_block_decode_attn")


def bt_block_decode_step(cfg, cache: BlockCache, layer, q, k_new, v_new, out, workspace, dev_status=None, stream=None):
    """Append the new block's row and attend over the cache including it, in one launch."""
    _check(_lib.bt_block_decode_step(ctypes.byref(cfg), ctypes.byref(cache.c), layer, _ptr(q), _ptr(k_new), _ptr(v_new),
                                     _ptr(out), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                     _ptr(dev_status), _stream(stream)), "bt_block_decode_step")


def bt_block_decode_step_multi(cfg, cache: BlockCache, layer, q, k_new, v_new, out, workspace, n_q=None, dev_status=None,
                               stream=None):
    """Append n_q rows and run n_q queries (query i sees the cache and new rows 0..i), one launch."""
    n_q = q.shape[2] if n_q is None else n_q
    _check(_lib.bt_block_decode_step_multi(ctypes.byref(cfg), ctypes.byref(cache.c), layer, _ptr(q), _ptr(k_new), _ptr(v_new),
                                           n_q, _ptr(out), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                           _ptr(dev_status), _stream(stream)), "bt_block_decode_step_multi")


BT_STATIC_WORKSPACE_BYTES = 2 << 20


def bt_block_decode_attn_noalloc(cfg, cache: BlockCache, layer, q, out, dev_status=None, stream=None):
    """bt_block_decode_attn with the split scratch inside the library (no workspace argument): for
    callers that cannot allocate device memory.  Rejects configs whose scratch would exceed
    BT_STATIC_WORKSPACE_BYTES; calls on one device share the scratch, so do not overlap them."""
    _check(_lib.bt_block_decode_attn_noalloc(ctypes.byref(cfg), ctypes.byref(cache.c), layer, _ptr(q), _ptr(out),
                                             _ptr(dev_status), _stream(stream)), "bt_block_decode_attn_noalloc")


def bt_prefix_project(cfg, ctx, w_prefix, bias, prefix_out, dev_status=None, stream=None):
    """Context embedding [B,D] -> P prefix token embeddings [B,P,D]."""
    _check(_lib.bt_prefix_project(ctypes.byref(cfg), _ptr(ctx), _ptr(w_prefix), _ptr(bias), _ptr(prefix_out),
                                  _ptr(dev_status), _stream(stream)), "bt_prefix_project")


def bt_block_qkv_project_append(cfg, cache: BlockCache, layer, x, w_qkv, bias, q_out, n_rows=None, dev_status=None, stream=None):
    """QKV projection of x [B,n,D]; Q -> q_out [B,H,n,hd], K and V rows appended to the block cache."""
    n_rows = x.shape[1] if n_rows is None else n_rows
    _check(_lib.bt_block_qkv_project_append(ctypes.byref(cfg), ctypes.byref(cache.c), layer, _ptr(x), n_rows, _ptr(w_qkv),
                                            _ptr(bias), _ptr(q_out), _ptr(dev_status), _stream(stream)),
           "bt_block_qkv_project_append")


def bt_local_qkv_project_append(cfg, cache: LocalCache, layer, x, w_qkv, bias, q_out, n_rows=None, reset_first=False,
                                reset_mask=None, dev_status=None, stream=None):
    """QKV projection of x [B,n,D]; Q -> q_out [B,H,n,hd], K and V rows appended to the local cache
    (after the optional block-boundary reset)."""
    n_rows = x.shape[1] if n_rows is None else n_rows
    _check(_lib.bt_local_qkv_project_append(ctypes.byref(cfg), ctypes.byref(cache.c), layer, _ptr(x), n_rows, _ptr(w_qkv),
                                            _ptr(bias), 1 if reset_first else 0, _ptr(reset_mask), _ptr(q_out),
                                            _ptr(dev_status), _stream(stream)), "bt_local_qkv_project_append")


def bt_selftest_bounded_wait(report, dev_status, stream=None):
    """Run the library's two bounded-wait routines on barriers nothing completes (test support)."""
    _check(_lib.bt_selftest_bounded_wait(_ptr(report), _ptr(dev_status), _stream(stream)), "bt_selftest_bounded_wait")


def bt_local_kv_reset(cfg, cache: LocalCache, layer, seq_mask=None, stream=None):
    _check(_lib.bt_local_kv_reset(ctypes.byref(cfg), ctypes.byref(cache.c), layer, _ptr(seq_mask), _stream(stream)),
           "bt_local_kv_reset")


def bt_local_kv_append(cfg, cache: LocalCache, layer, k_new, v_new, n_new=None, dev_status=None, stream=None):
    n_new = k_new.shape[2] if n_new is None else n_new
    _check(_lib.bt_local_kv_append(ctypes.byref(cfg), ctypes.byref(cache.c), layer, _ptr(k_new), _ptr(v_new),
                                   n_new, _ptr(dev_status), _stream(stream)), "bt_local_kv_append")


def bt_token_decode_attn(cfg, cache: LocalCache, layer, q, k_new, v_new, out, n_q=None, reset_first=False,
                         reset_mask=None, dev_status=None, stream=None):
    n_q = q.shape[2] if n_q is None else n_q
    _check(_lib.bt_token_decode_attn(ctypes.byref(cfg), ctypes.byref(cache.c), layer, _ptr(q), _ptr(k_new),
                                     _ptr(v_new), n_q, 1 if reset_first else 0, _ptr(reset_mask), _ptr(out),
                                     _ptr(dev_status), _stream(stream)), "bt_token_decode_attn")


def bt_block_prefill_attn(cfg, q, k, v, out, n_blocks=None, kv_seq_stride=None, dev_status=None, stream=None):
    n_blocks = q.shape[2] if n_blocks is None else n_blocks
    kv_seq_stride = n_blocks if kv_seq_stride is None else kv_seq_stride
    _check(_lib.bt_block_prefill_attn(ctypes.byref(cfg), _ptr(q), _ptr(k), _ptr(v), n_blocks, kv_seq_stride,
                                      _ptr(out), _ptr(dev_status), _stream(stream)), "bt_block_prefill_attn")


def bt_block_decode_step_host(cfg, cache: BlockCache, layer, q_host, k_new_host, v_new_host, out_host, q_dev, k_dev,
                              v_dev, out_dev, workspace=None, dev_status=None, stream=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(_lib.bt_block_decode_step_host(ctypes.byref(cfg), ctypes.byref(cache.c), layer, _ptr(q_host),
                                          _ptr(k_new_host), _ptr(v_new_host), _ptr(out_host), _ptr(q_dev),
                                          _ptr(k_dev), _ptr(v_dev), _ptr(out_dev), _ptr(workspace), ws_bytes,
                                          _ptr(dev_status), _stream(stream)), "bt_block_decode_step_host")
