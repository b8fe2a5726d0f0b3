"""Seeded synthetic inputs shared by the oracle-side tests and the GPU-side tests / benchmark.

Holds no arithmetic of the method: only "draw N(mean, std) from a seeded CPU generator, cast to the
storage dtype".  Seeds follow  3905*1000 + 10*config + tensor_ordinal.
"""
from __future__ import annotations

import numpy as np
import torch


def seed_for(config: int, ordinal: int) -> int:
    return 3905 * 1000 + 10 * config + ordinal


def normal(shape, mean: float, std: float, dtype: torch.dtype, config: int, ordinal: int) -> torch.Tensor:
    """N(mean, std) drawn in fp32 from torch's CPU generator, then rounded (RNE) to `dtype`."""
    g = torch.Generator(device="cpu").manual_seed(seed_for(config, ordinal))
    t = torch.randn(tuple(shape), generator=g, dtype=torch.float32) * std + mean
    return t.to(dtype).contiguous()


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact conversion of stored fp32 / bf16 values to fp64 for the oracle."""
    return t.detach().to("cpu").to(torch.float64).numpy()


def llama_weights(hidden: int, ffn: int, config: int = 5, dtype=torch.bfloat16, first_ordinal: int = 1, kv_hidden: int | None = None):
    """Random-init block weights, all [in, out]: N(0, 0.02); norm gains N(1, 0.1). kv_hidden = width of the key / value
    projections (n_kv_heads * d_head; = hidden unless the block is grouped-query)."""
    o = first_ordinal
    w = {}
    kvh = hidden if kv_hidden is None else kv_hidden
    for name, shape in (("wq", (hidden, hidden)), ("wk", (hidden, kvh)), ("wv", (hidden, kvh)),
                        ("wo", (hidden, hidden)), ("w1", (hidden, ffn)), ("w3", (hidden, ffn)),
                        ("w2", (ffn, hidden))):
        w[name] = normal(shape, 0.0, 0.02, dtype, config, o)
        o += 1
    for name in ("g1", "g2"):
        w[name] = normal((hidden,), 1.0, 0.1, dtype, config, o)
        o += 1
    return w
