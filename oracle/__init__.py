"""CPU oracle (test infrastructure, not product code).

Builds ``bt_oracle.c`` with gcc into two shared objects' worth of symbols (float64
primary, float32 twin) and wraps them with ctypes over numpy arrays.  bf16 data
is carried as ``uint16`` bit patterns.  Nothing here imports the CUDA package.

Only the tests, the smoke check and the benchmark's cpu_baseline / reference legs
may import this package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

from .schedule import generation_schedule, token_step_schedule  # noqa: F401

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bt_oracle.c")
_SO = os.path.join(_HERE, "libbt_oracle.so")
_lock = threading.Lock()
_lib = None

ST_OVERFLOW = 1
ST_EMPTY = 2


def build(force: bool = False) -> str:
    """Compile the C oracle (both precisions) into one shared library."""
    with _lock:
        if not force and os.path.exists(_SO) and os.path.getmtime(_SO) >= os.path.getmtime(_SRC):
            return _SO
        objs = []
        for real, suffix in (("double", ""), ("float", "_f32")):
            obj = os.path.join(_HERE, f"bt_oracle{suffix or '_f64'}.o")
            subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-std=c11", "-Wall",
                                   f"-DREAL={real}", f"-DSUFFIX={suffix}", "-c", _SRC, "-o", obj])
            objs.append(obj)
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-shared", "-fopenmp", "-o", tmp] + objs + ["-lm"])
        os.replace(tmp, _SO)
        return _SO


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def n_threads() -> int:
    """Threads the OpenMP loops of the oracle will use."""
    v = os.environ.get("OMP_NUM_THREADS")
    return int(v) if v else (os.cpu_count() or 1)


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _real(f32):
    return (np.float32, "_f32") if f32 else (np.float64, "")


def default_scale(hd: int) -> float:
    return 1.0 / float(np.sqrt(hd))


def attend(q, K, V, scale=None, f32=False):
    """Softmax attention of one query [hd] over rows K,V [n,hd]; returns (out[hd], probs[n])."""
    q, K, V = _u16(q), _u16(K), _u16(V)
    n, hd = K.shape
    dt, sfx = _real(f32)
    out = np.zeros(hd, dt)
    probs = np.zeros(max(n, 1), dt)
    getattr(lib(), "bto_attend" + sfx)(_p(q), _p(K), _p(V), ctypes.c_int(n), ctypes.c_int(hd),
                                       ctypes.c_double(scale if scale is not None else default_scale(hd)),
                                       _p(out), _p(probs))
    return out, probs[:n]


class Cache:
    """One layer's KV cache as the oracle sees it: K, V [B,H,cap,hd] (bf16 bits) + len[B]."""

    def __init__(self, B, H, cap, hd):
        self.B, self.H, self.cap, self.hd = B, H, cap, hd
        self.k = np.zeros((B, H, cap, hd), np.uint16)
        self.v = np.zeros((B, H, cap, hd), np.uint16)
        self.len = np.zeros(B, np.int32)
        self.status = np.zeros(1, np.uint32)

    def copy(self):
        c = Cache(self.B, self.H, self.cap, self.hd)
        c.k[...] = self.k
        c.v[...] = self.v
        c.len[...] = self.len
        c.status[...] = self.status
        return c


def kv_append(c: Cache, k_new, v_new):
    """Append rows [B,H,n_new,hd] at len..len+n_new-1 (block cache or local cache)."""
    k_new, v_new = _u16(k_new), _u16(v_new)
    n_new = k_new.shape[2]
    assert k_new.shape == (c.B, c.H, n_new, c.hd) and v_new.shape == k_new.shape
    lib().bto_kv_append(c.B, c.H, c.hd, c.cap, _p(c.k), _p(c.v), _p(c.len), _p(k_new), _p(v_new),
                        ctypes.c_int(n_new), _p(c.status))


def block_decode_attn(c: Cache, q, scale=None, f32=False):
    """One query per (b,h) over rows < len[b]; q [B,H,hd] -> out [B,H,hd]."""
    q = _u16(q)
    assert q.shape == (c.B, c.H, c.hd)
    dt, sfx = _real(f32)
    out = np.zeros((c.B, c.H, c.hd), dt)
    getattr(lib(), "bto_block_decode_attn" + sfx)(
        c.B, c.H, c.hd, c.cap, _p(c.k), _p(c.v), _p(c.len), _p(q),
        ctypes.c_double(scale if scale is not None else default_scale(c.hd)), _p(out), _p(c.status))
    return out


def local_kv_reset(c: Cache, mask=None):
    m = None if mask is None else np.ascontiguousarray(mask, np.uint8)
    lib().bto_local_kv_reset(c.B, _p(c.len), _p(m))


def token_decode_attn(c: Cache, q, k_new, v_new, reset_first=False, reset_mask=None, scale=None, f32=False):
    """Fused token-decoder step: reset? -> append n_q rows -> causal attention inside the block.
    k_new = v_new = None: nothing is appended, the n_q queries belong to the last n_q cached rows."""
    q = _u16(q)
    n_q = q.shape[2]
    assert q.shape == (c.B, c.H, n_q, c.hd)
    if k_new is not None:
        k_new, v_new = _u16(k_new), _u16(v_new)
        assert k_new.shape == q.shape and v_new.shape == q.shape
    m = None if reset_mask is None else np.ascontiguousarray(reset_mask, np.uint8)
    dt, sfx = _real(f32)
    out = np.zeros((c.B, c.H, n_q, c.hd), dt)
    getattr(lib(), "bto_token_decode_attn" + sfx)(
        c.B, c.H, c.hd, c.cap, _p(c.k), _p(c.v), _p(c.len), _p(q), _p(k_new), _p(v_new),
        ctypes.c_int(n_q), ctypes.c_int(1 if reset_first else 0), _p(m),
        ctypes.c_double(scale if scale is not None else default_scale(c.hd)), _p(out), _p(c.status))
    return out


def block_decode_step_multi(c: Cache, q, k_new, v_new, scale=None, f32=False):
    """Decode step of the densified block decoder (appendix "Discussion and future works"): a block
    is L_B sub-block tokens, so a step appends m rows and runs m queries, query i seeing every cached
    row and the new rows 0..i.  q, k_new, v_new [B,H,m,hd] -> out [B,H,m,hd].

    Written as the definition: the m rows are appended (all of them or, for a sequence without room,
    none, as kv_append does), then query i is a plain decode over the first len_before + i + 1 rows.
    A sequence that had no room keeps its rows and every query attends over them."""
    q = _u16(q)
    m = q.shape[2]
    assert q.shape == (c.B, c.H, m, c.hd)
    before = c.len.copy()
    kv_append(c, k_new, v_new)
    after = c.len.copy()
    dt, _ = _real(f32)
    out = np.zeros((c.B, c.H, m, c.hd), dt)
    for i in range(m):
        c.len[...] = np.where(after > before, before + i + 1, before)
        out[:, :, i] = block_decode_attn(c, np.ascontiguousarray(q[:, :, i]), scale=scale, f32=f32)
    c.len[...] = after
    return out


def block_prefill_attn(q, k, v, scale=None, f32=False, kv_seq_stride=None):
    """Dense causal attention over T blocks; q [B,H,T,hd]; k,v [B,H,stride,hd] -> out [B,H,T,hd]."""
    q, k, v = _u16(q), _u16(k), _u16(v)
    B, H, T, hd = q.shape
    stride = k.shape[2] if kv_seq_stride is None else kv_seq_stride
    assert k.shape == (B, H, stride, hd) and v.shape == k.shape and stride >= T
    dt, sfx = _real(f32)
    out = np.zeros((B, H, T, hd), dt)
    getattr(lib(), "bto_block_prefill_attn" + sfx)(
        B, H, T, hd, _p(q), _p(k), _p(v), ctypes.c_longlong(stride),
        ctypes.c_double(scale if scale is not None else default_scale(hd)), _p(out))
    return out


def linear(x, W, bias=None, f32=False):
    """y = W x + b over rows: x [M,K], W [N,K] (row o = weights of output feature o), bias [N] -> [M,N]."""
    x, W = _u16(x), _u16(W)
    M, K = x.shape
    N = W.shape[0]
    assert W.shape == (N, K)
    if bias is not None:
        bias = _u16(bias)
        assert bias.shape == (N,)
    dt, sfx = _real(f32)
    y = np.zeros((M, N), dt)
    getattr(lib(), "bto_linear" + sfx)(M, K, N, _p(x), _p(W), _p(bias), _p(y))
    return y


def round_to_bf16(v):
    """Nearest bf16 (ties to even) of float64 values, as uint16 bits."""
    f = lib().bto_round_to_bf16
    f.restype, f.argtypes = ctypes.c_uint16, [ctypes.c_double]
    a = np.asarray(v, np.float64)
    return np.array([f(float(t)) for t in a.ravel()], np.uint16).reshape(a.shape)


def prefix_project(ctx, W, bias, P, f32=False):
    """Context embedding -> P prefix token embeddings (section 2.4; appendix on token-decoder variants,
    "Prefix"): ctx [B,D], W [P*D,D], bias [P*D] or None -> [B,P,D] (output feature p*D + d is
    dimension d of prefix token p)."""
    B, D = ctx.shape
    assert W.shape == (P * D, D)
    return linear(ctx, W, bias, f32=f32).reshape(B, P, D)


def qkv_project_append(c: Cache, x, W, bias=None, reset_first=False, reset_mask=None, f32=False):
    """y = W x + b for x [B,n,D]; returns q [B,H,n,hd] (not rounded) and appends the K and V parts,
    rounded to bf16, to the cache (block or local) as kv_append would, after the optional reset."""
    x, W = _u16(x), _u16(W)
    B, n, D = x.shape
    assert B == c.B and D == c.H * c.hd and W.shape == (3 * D, D)
    if bias is not None:
        bias = _u16(bias)
        assert bias.shape == (3 * D,)
    m = None if reset_mask is None else np.ascontiguousarray(reset_mask, np.uint8)
    dt, sfx = _real(f32)
    q = np.zeros((B, c.H, n, c.hd), dt)
    getattr(lib(), "bto_qkv_project_append" + sfx)(
        B, n, c.H, c.hd, c.cap, _p(x), _p(W), _p(bias), _p(c.k), _p(c.v), _p(c.len),
        ctypes.c_int(1 if reset_first else 0), _p(m), _p(q), _p(c.status))
    return q
