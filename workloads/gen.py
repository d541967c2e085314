"""Seeded synthetic inputs shared by the tests, the oracle runs and the CUDA runs.

This module only *draws numbers*: i.i.d. N(0,1) values rounded to bf16, keyed by
(seed, tensor id).  It holds none of the attention arithmetic, so both the CPU
oracle and the CUDA path can be fed the same bytes from here without sharing any
of the method's code.

Two generators exist because of size:

* ``normal_bf16_bits`` (host, numpy): a counter-based generator.  Element ``i`` of
  tensor ``tid`` under ``seed`` is a pure function of ``(seed, tid, i)``:
  splitmix64 of the counter gives two uniforms, Box-Muller in float64 gives a
  normal deviate, which is rounded to float32 and then to bf16 (nearest even).
  Used for every case the oracle computes in full.
* ``normal_bf16_device`` (torch CUDA generator): for multi-GiB caches that would
  take minutes on the host.  The bytes then live on the GPU; tests copy the
  sampled slices back to the host and hand exactly those bytes to the oracle.

bf16 values travel as ``uint16`` bit patterns on the numpy side.
"""
from __future__ import annotations

import numpy as np

_MASK64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def _splitmix64(x: np.ndarray) -> np.ndarray:
    """One round of the splitmix64 output function on a uint64 array."""
    x = (x + np.uint64(0x9E3779B97F4A7C15)) & _MASK64
    z = x
    z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _MASK64
    z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _MASK64
    return z ^ (z >> np.uint64(31))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round to nearest, ties to even); returns uint16 bits."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (b >> np.uint32(16)) & np.uint32(1)
    r = b + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) exactly to float32."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16_bits(seed: int, tid: int, shape, chunk: int = 1 << 22) -> np.ndarray:
    """N(0,1) samples rounded to bf16, as uint16 bit patterns of the given shape."""
    n = int(np.prod(shape)) if len(shape) else 1
    out = np.empty(n, dtype=np.uint16)
    with np.errstate(over="ignore"):
        key = _splitmix64(np.array([(int(seed) << 20) ^ int(tid)], dtype=np.uint64))[0]
        for lo in range(0, n, chunk):
            hi = min(n, lo + chunk)
            ctr = np.arange(lo, hi, dtype=np.uint64)
            a = _splitmix64((ctr * np.uint64(2)) ^ key)
            b = _splitmix64((ctr * np.uint64(2) + np.uint64(1)) ^ key)
            # 53-bit uniforms; u1 in (0,1], u2 in [0,1)
            u1 = ((a >> np.uint64(11)).astype(np.float64) + 1.0) * (1.0 / 9007199254740992.0)
            u2 = (b >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)
            z = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
            out[lo:hi] = f32_to_bf16_bits(z.astype(np.float32))
    return out.reshape(shape)


# ---- torch side (imported lazily so that the numpy part has no torch dependency) ----

def bits_to_torch(bits: np.ndarray, device="cpu"):
    """uint16 bf16 bit patterns -> torch.bfloat16 tensor (same bytes)."""
    import torch

    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t.to(device) if str(device) != "cpu" else t


def torch_to_bits(t) -> np.ndarray:
    """torch.bfloat16 tensor (any device) -> uint16 bit patterns on the host."""
    import torch

    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16).copy()


def normal_bf16_device(seed: int, tid: int, shape, device="cuda"):
    """N(0,1) bf16 tensor drawn with torch's seeded generator on ``device``.

    For buffers too large to draw on the host.  Drawn in slabs along dim 0 so the
    float32 temporary stays small.
    """
    import torch

    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1000003 + int(tid)) & 0x7FFFFFFFFFFFFFFF)
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    n = flat.numel()
    slab = 1 << 26
    for lo in range(0, n, slab):
        hi = min(n, lo + slab)
        flat[lo:hi] = torch.randn(hi - lo, generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)
    return out
