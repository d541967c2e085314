"""Named workload shapes (plain data, no arithmetic of the method).

The shapes follow the paper's model table (12+12 layers, 16 heads, model dim 1024
with head_dim 64, or 2048 with head_dim 128), its block length L_B = 4 and its
two serving settings: prefill-heavy (2048 prompt / 128 generated) and
decode-heavy (128 / 2048), with every prompt padded to the same length.
"""
from __future__ import annotations

from dataclasses import dataclass, replace


@dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    heads: int
    head_dim: int
    block_len: int          # L_B
    prefix_len: int         # P
    n_layers: int
    max_blocks: int         # block-cache capacity N_max (rows)
    ctx_blocks: int = 0     # block-cache length after the append (decode configs)
    prompt_blocks: int = 0  # T (prefill configs)
    prompt_tokens: int = 0
    gen_tokens: int = 0
    seed: int = 1000

    @property
    def local_cap(self) -> int:
        return self.prefix_len + self.block_len


# config 1: tiny single decode step, every entry point, checked against full recompute
TINY = Workload("tiny", batch=4, heads=8, head_dim=64, block_len=4, prefix_len=1, n_layers=2,
                max_blocks=64, ctx_blocks=64, prompt_blocks=64, seed=1001)

# config 2: block-decoder decode step (2048-token context -> 512 block entries), 12 layers
BLOCK_DECODE = Workload("block_decode", batch=256, heads=16, head_dim=64, block_len=4, prefix_len=1,
                        n_layers=12, max_blocks=512, ctx_blocks=512, seed=1002)

# config 2b: the same step at a context eight times longer (16K tokens -> 4096 block entries; the paper's
# long-context comparison raises the context four- and eightfold), batch sized to a 13 GB cache
BLOCK_DECODE_16K = Workload("block_decode_16k", batch=64, heads=16, head_dim=64, block_len=4, prefix_len=1,
                            n_layers=12, max_blocks=4096, ctx_blocks=4096, seed=1012)

# the densified block decoder the paper proposes as future work: a block is L_B sub-block tokens, so the
# cache holds one row per token (2048 rows for the 2048-token context) and a step appends L_B rows and
# runs L_B queries
DENSE_DECODE = Workload("dense_decode", batch=256, heads=16, head_dim=64, block_len=4, prefix_len=1,
                        n_layers=12, max_blocks=2048, ctx_blocks=2048, seed=1022)

# config 3: token-decoder local decode, 4096 sequences, local cache 1 prefix + up to L_B tokens
TOKEN_DECODE = Workload("token_decode", batch=4096, heads=16, head_dim=64, block_len=4, prefix_len=1,
                        n_layers=12, max_blocks=1, gen_tokens=4096, seed=1003)

# config 4: block-decoder prefill, 2048-token prompt -> 512 blocks, head_dim 128
BLOCK_PREFILL = Workload("block_prefill", batch=32, heads=16, head_dim=128, block_len=4, prefix_len=1,
                         n_layers=12, max_blocks=512, prompt_blocks=512, prompt_tokens=2048, seed=1004)

# config 4b: the 8K-prompt case (2048 blocks), where the tensor pipe rather than HBM binds
BLOCK_PREFILL_8K = Workload("block_prefill_8k", batch=8, heads=16, head_dim=128, block_len=4, prefix_len=1,
                            n_layers=12, max_blocks=2048, prompt_blocks=2048, prompt_tokens=8192, seed=1014)


# the linear maps either side of the path, at the shapes of configs 3 and 2: one token step of the token decoder
# (4096 rows), one block step of the block decoder (256 rows), model dim 1024, distinct weights per layer
QKV_PROJECT_TOKEN = Workload("qkv_project_token", batch=4096, heads=16, head_dim=64, block_len=4, prefix_len=1,
                             n_layers=12, max_blocks=1, seed=1033)
QKV_PROJECT_BLOCK = Workload("qkv_project_block", batch=256, heads=16, head_dim=64, block_len=4, prefix_len=1,
                             n_layers=12, max_blocks=512, ctx_blocks=512, seed=1032)
TOKEN_DECODE_PROJECTED = Workload("token_decode_projected", batch=4096, heads=16, head_dim=64, block_len=4, prefix_len=1,
                                  n_layers=12, max_blocks=1, seed=1035)
PREFIX_PROJECT = Workload("prefix_project", batch=4096, heads=16, head_dim=64, block_len=4, prefix_len=2,
                          n_layers=12, max_blocks=1, seed=1034)


def sweep(block_len: int) -> Workload:
    """config 5: decode-heavy generation (128-token prompt, 2048 generated) at one block length."""
    prompt, gen = 128, 2048
    return Workload(f"sweep_LB{block_len}", batch=512, heads=16, head_dim=64, block_len=block_len,
                    prefix_len=1, n_layers=12, max_blocks=(prompt + gen) // block_len,
                    prompt_blocks=prompt // block_len, prompt_tokens=prompt, gen_tokens=gen,
                    seed=1005)


def scaled(w: Workload, **kw) -> Workload:
    """A smaller copy of a workload for tests (same structure, fewer sequences/layers)."""
    return replace(w, **kw)


BY_NAME = {w.name: w for w in (TINY, BLOCK_DECODE, BLOCK_DECODE_16K, DENSE_DECODE, TOKEN_DECODE, BLOCK_PREFILL, BLOCK_PREFILL_8K,
                               QKV_PROJECT_TOKEN, QKV_PROJECT_BLOCK, PREFIX_PROJECT, TOKEN_DECODE_PROJECTED)}
