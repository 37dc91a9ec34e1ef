"""Named synthetic workloads.

Shapes follow the models the paper evaluates (App. B "Models"): a
LlamaGen-like 16384-entry codebook with 8-dim codes and 16x16 / 32x32 token
grids, and a Chameleon-family 65536-token vocabulary whose image tokens map to
an 8192 x 256 codebook.  Logits are Gaussian stand-ins for model outputs; the
drafter rows are noisy copies of the target rows so that acceptance rates are
neither 0 nor 1.  The paper's data sets and model weights are not used.
"""

from dataclasses import dataclass
from typing import Optional


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    index: int              # seeds are 1000 * index + step
    batch: int              # B sequences verified per call
    n_nodes: int            # N tree nodes including the root
    vocab: int              # V logits per row
    dtype: str              # "f32" or "bf16" logits
    cfg_scale: Optional[float]   # classifier-free guidance g, None = no uncond rows
    temperature: float
    top_k: int              # truncation before softmax on both sides, 0 = off
    logit_std: float
    draft_mix: float        # drafter = draft_mix * target + N(0, draft_noise^2)
    draft_noise: float
    codebook_size: int      # L
    codebook_dim: int       # d
    codebook_dtype: str
    code_offset: int        # token t has latent code t - code_offset
    k: int                  # latent neighbours per token
    lam: float              # multiplicative bound lambda
    steps: int              # decode steps of one image in the modelled run


CONFIGS = {
    "c1_tiny": WorkloadConfig("c1_tiny", 1, 1, 26, 16384, "f32", 7.5, 1.0, 0, 1.5,
                              1.0, 0.5, 16384, 8, "f32", 0, 50, 2.0, 256),
    "c2_llamagen512": WorkloadConfig("c2_llamagen512", 2, 8, 60, 16384, "f32", 7.5, 1.0,
                                     1000, 1.2, 1.0, 0.5, 16384, 8, "f32", 0, 100, 3.0, 1024),
    "c3_lumina": WorkloadConfig("c3_lumina", 3, 4, 60, 65536, "f32", 3.0, 1.0, 0, 1.5,
                                1.0, 0.5, 8192, 256, "bf16", 4096, 100, 3.0, 2400),
    "c4_batch64": WorkloadConfig("c4_batch64", 4, 64, 80, 65536, "bf16", None, 1.0, 0, 1.0,
                                 0.7, 0.7, 8192, 256, "bf16", 4096, 200, 3.0, 20),
}

# neighbour-table sweep (config 5): every (L, d, k) combination, bf16 codes,
# 5 % of the rows are exact copies of other rows
SWEEP_L = (4096, 16384, 65536)
SWEEP_D = (8, 64, 256)
SWEEP_K = (10, 50, 200)
SWEEP_DUP_FRAC = 0.05
