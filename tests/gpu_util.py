"""Helpers for the GPU parity tests: move seeded tensors into relations with the ORACLE's packing (so
the GPU's own relayout is never trusted to prepare its own inputs), read relations back, compare."""
from __future__ import annotations

import numpy as np
import torch

import paper_2609_03905_b200 as ja
from oracle import blocked


def np_bits(t: torch.Tensor) -> np.ndarray:
    """Raw storage of a CPU tensor as a numpy array (bf16 -> uint16 bit patterns)."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def from_bits(a: np.ndarray, dtype: torch.dtype) -> torch.Tensor:
    if dtype == torch.bfloat16:
        return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16)
    return torch.from_numpy(a.copy())


def to_f64(a: np.ndarray, dtype: torch.dtype) -> np.ndarray:
    return from_bits(a, dtype).to(torch.float64).numpy()


def upload(dense: torch.Tensor, splits) -> ja.Relation:
    """dense CPU tensor -> relation on the GPU, packed on the host by the oracle's key-table code."""
    payload = blocked.pack(np_bits(dense), splits)
    t = from_bits(payload, dense.dtype).cuda()
    return ja.Relation(list(dense.shape), splits, dense.dtype, t)


def empty_like_tiling(extents, splits, dtype, fill=None) -> ja.Relation:
    r = ja.Relation(extents, splits, dtype)
    if fill is not None:
        r.payload.fill_(fill)
    return r


def download(rel: ja.Relation) -> np.ndarray:
    """relation -> dense fp64 numpy tensor, unpacked on the host by the oracle's key-table code."""
    torch.cuda.synchronize()
    bits = np_bits(rel.payload.cpu())
    dense_bits = blocked.unpack(bits, rel.extents, rel.splits)
    return to_f64(dense_bits, rel.dtype)


def download_bits(rel: ja.Relation) -> np.ndarray:
    torch.cuda.synchronize()
    return np_bits(rel.payload.cpu())


def relfro(got: np.ndarray, ref: np.ndarray) -> float:
    assert got.shape == ref.shape, (got.shape, ref.shape)
    assert np.isfinite(got).all(), "non-finite values in the GPU result"
    den = np.linalg.norm(ref.reshape(-1))
    return float(np.linalg.norm((got - ref).reshape(-1)) / (den if den > 0 else 1.0))


def check_status():
    assert ja.ja_stream_status(torch.cuda.current_stream().cuda_stream) == 0, "device status word set (bounded wait expired)"


TOL = {torch.float32: 1e-5, torch.bfloat16: 2e-2}
