"""Algorithmic byte and FLOP counts of the attention path (cost model only).

These are the numbers the roofline fractions are quoted against: the bytes an
ideal implementation must move once, with bf16 (2-byte) storage.  The formulas
are checked against the paper's own counting examples (KV bytes per token of a
7B model; L_B**2 and L/L_B reductions) in the CPU tests.
"""
from __future__ import annotations

BF16 = 2


def kv_bytes_per_token(n_layers: int, model_dim: int, elem_bytes: int = BF16) -> int:
    """K and V of one position over all layers."""
    return n_layers * 2 * model_dim * elem_bytes


def block_decode_layer_bytes(B: int, H: int, hd: int, ctx_len: int, with_append: bool = True) -> int:
    """One layer of one block-decoder decode step: read K,V rows 0..ctx_len-1, q in, out out,
    and (if fused in the step) the appended row read once and written once."""
    kv = B * H * ctx_len * 2 * hd * BF16
    qo = 2 * B * H * hd * BF16
    app = (2 * 2 * B * H * hd * BF16) if with_append else 0
    return kv + qo + app


def dense_decode_layer_bytes(B: int, H: int, hd: int, rows_after: int, m: int) -> int:
    """One layer of one densified block-decoder step: the rows_after - m cached rows (K and V) read,
    m queries in and m outputs out, the m new K,V rows read once and written once."""
    row = hd * BF16
    return B * H * ((rows_after - m) * 2 * row + 2 * m * row + 2 * 2 * m * row)


def token_decode_layer_bytes(B: int, H: int, hd: int, rows_before: int, n_new: int = 1) -> int:
    """One layer of one token-decoder step: q, k_new, v_new in; out out; the new rows written
    to the local cache; rows_before cached rows (K and V) read."""
    row = hd * BF16
    fixed = (3 * n_new + n_new + 2 * n_new) * row      # q,k,v reads + out write + K,V row writes
    return B * H * (fixed + rows_before * 2 * row)


def prefill_layer_bytes(B: int, H: int, T: int, hd: int) -> int:
    """Q, K, V read once and the output written once."""
    return 4 * B * H * T * hd * BF16


def prefill_layer_flops(B: int, H: int, T: int, hd: int) -> int:
    """Causal attention: T(T+1)/2 (query, key) pairs, each 2*hd flops for the score and 2*hd
    for the weighted sum."""
    return B * H * (T * (T + 1) // 2) * 4 * hd


def generation_bytes(B: int, H: int, hd: int, n_layers: int, block_len: int, prompt_tokens: int, gen_tokens: int) -> dict:
    """Whole decode-heavy generation: prompt prefill + bulk append, then per generated block L_B token
    steps (step j reads j cached rows) and one block step over T + g + 1 rows.  Returns the parts."""
    T = prompt_tokens // block_len
    G = gen_tokens // block_len
    prefill = n_layers * (prefill_layer_bytes(B, H, T, hd) + 2 * 2 * B * H * T * hd * BF16)
    token = n_layers * G * sum(token_decode_layer_bytes(B, H, hd, j) for j in range(block_len))
    block = n_layers * sum(block_decode_layer_bytes(B, H, hd, T + g + 1, True) for g in range(G))
    return {"prefill": prefill, "token": token, "block": block, "total": prefill + token + block}


def linear_flops(M: int, N: int, K: int) -> int:
    """y = W x + b over M rows: one multiply-add per (row, output feature, input feature)."""
    return 2 * M * N * K


def linear_bytes(M: int, N: int, K: int) -> int:
    """x [M,K] and W [N,K] read once, bias [N] read once, y [M,N] written once (wherever its parts go)."""
    return (M * K + N * K + N + M * N) * BF16
