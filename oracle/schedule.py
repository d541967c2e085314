"""Pure-integer model of when the caches grow and reset (test infrastructure).

Generation with a Block Transformer (Figure 1; sections 2.3, 2.4; appendix E.2):
the prompt's T = prompt_len / L_B blocks are prefilled through the block decoder
(one block-cache row each); the token decoder prefills nothing.  Then, per
generated block: L_B token-decoder steps, followed by one block-decoder step that
appends the finished block's row and attends over all rows.

Token step j (0-based) inside a block:
  j == 0: the local cache is reset and the P prefix rows projected from the
          context embedding are appended; the last prefix position predicts the
          block's first token;
  j >= 1: the row of the token produced by step j-1 is appended.
After step j the local cache holds P + j rows, so at most P + L_B - 1 rows are
ever attended (the attention map is 5 long for L_B = 4, P = 2) and the last
token of a block is never fed to the token decoder.
"""
from __future__ import annotations

from typing import List, Tuple


def token_step_schedule(block_len: int, prefix_len: int, n_steps: int) -> List[Tuple[int, int, int]]:
    """For token steps 0..n_steps-1: (reset?, rows appended, local length after)."""
    out = []
    for t in range(n_steps):
        j = t % block_len
        out.append((1 if j == 0 else 0, prefix_len if j == 0 else 1, prefix_len + j))
    return out


def generation_schedule(block_len: int, prefix_len: int, prompt_len: int, gen_tokens: int):
    """Event list for one generation.

    Events: ("prefill", T) | ("token", reset, n_append, local_len_after)
            | ("block", block_len_after).
    ``prompt_len`` and ``gen_tokens`` must be multiples of ``block_len`` (callers pad).
    """
    assert prompt_len % block_len == 0 and gen_tokens % block_len == 0
    T = prompt_len // block_len
    ev = [("prefill", T)]
    n = T
    for _g in range(gen_tokens // block_len):
        for j in range(block_len):
            ev.append(("token", 1 if j == 0 else 0, prefix_len if j == 0 else 1, prefix_len + j))
        n += 1
        ev.append(("block", n))
    return ev
