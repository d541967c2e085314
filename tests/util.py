"""Helpers shared by the GPU parity tests (marshalling between numpy bf16 bits and torch)."""
import numpy as np
import torch

from workloads import gen

ATOL, RTOL = 1e-2, 2e-2          # the stated bar: |g - r| <= 1e-2 + 2e-2 |r|
TIGHT_ATOL, TIGHT_RTOL = 1e-4, 4e-3  # what bf16 rounding of an fp32-accumulated result should meet


def to_dev(bits):
    return gen.bits_to_torch(bits).cuda()


def to_f64(t):
    """bf16 CUDA tensor -> float64 numpy (exact widening)."""
    return gen.bf16_bits_to_f32(gen.torch_to_bits(t)).astype(np.float64)


# The tensor-core prefill feeds the softmax numerators to the second product as bf16 (8-bit
# mantissa, like K and V).  Each term p_j v_j then carries up to 2^-9 relative error, so the
# output error is bounded by 2^-9 * sum_j p_j |v_j| <= 2^-9 * max|v| (about 5 for N(0,1) values),
# independent of how small the output itself is, plus the bf16 rounding of the output.
P_BF16_ATOL, P_BF16_RTOL = 6e-3, 8e-3


def assert_close(gpu_bf16, ref, what="", p_bf16=False):
    g = to_f64(gpu_bf16).reshape(ref.shape)
    assert np.isfinite(g).all(), f"{what}: non-finite output"
    err = np.abs(g - ref)
    bound = ATOL + RTOL * np.abs(ref)
    assert (err <= bound).all(), f"{what}: max err {err.max():.3e} beyond the stated tolerance"
    tight = (P_BF16_ATOL + P_BF16_RTOL * np.abs(ref)) if p_bf16 else (TIGHT_ATOL + TIGHT_RTOL * np.abs(ref))
    assert (err <= tight).all(), f"{what}: max err {err.max():.3e} beyond bf16 rounding ({(err - tight).max():.3e} over)"
    return err.max()


def status_word():
    return torch.zeros(1, dtype=torch.int32, device="cuda")


def local_kv_split(kv_t):
    """local cache tensor [..., C, 2, hd] (one layer: [B,H,C,2,hd]) -> K bits, V bits [B,H,C,hd]."""
    bits = gen.torch_to_bits(kv_t)
    return np.ascontiguousarray(bits[..., 0, :]), np.ascontiguousarray(bits[..., 1, :])


# The projections accumulate K products in fp32 on the tensor cores and round once to bf16: half a bf16
# ulp (2^-9 relative) plus the accumulation error, which grows with sum_k |x_k w_k| (about 0.64 K for
# N(0,1) inputs) times a few fp32 ulps - 2e-3 covers K up to 2048.
PROJ_ATOL, PROJ_RTOL = 2e-3, 4e-3


def assert_close_proj(gpu_bf16, ref, what=""):
    g = to_f64(gpu_bf16).reshape(ref.shape)
    assert np.isfinite(g).all(), f"{what}: non-finite output"
    err = np.abs(g - ref)
    assert (err <= ATOL + RTOL * np.abs(ref)).all(), f"{what}: max err {err.max():.3e} beyond the stated tolerance"
    tight = PROJ_ATOL + PROJ_RTOL * np.abs(ref)
    assert (err <= tight).all(), f"{what}: max err {err.max():.3e} beyond fp32-accumulate + bf16 rounding"
    return err.max()
