"""Helpers for the GPU parity tests: move seeded tensors into relations with the ORACLE's packing (so
the GPU's own relayout is never trusted to prepare its own inputs), read relations back, compare."""
from __future__ import annotations

import weakref

import numpy as np
import torch

import paper_2609_03905_b200 as ja
from oracle import blocked


def np_bits(t: torch.Tensor) -> np.ndarray:
    """Raw storage of a CPU tensor as a numpy array (bf16, f16 -> uint16 bit patterns)."""
    t = t.detach().cpu().contiguous()
    if t.dtype in (torch.bfloat16, torch.float16):
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def from_bits(a: np.ndarray, dtype: torch.dtype) -> torch.Tensor:
    if dtype in (torch.bfloat16, torch.float16):
        return torch.from_numpy(a.view(np.int16).copy()).view(dtype)
    return torch.from_numpy(a.copy())


def to_f64(a: np.ndarray, dtype: torch.dtype) -> np.ndarray:
    return from_bits(a, dtype).to(torch.float64).numpy()


# Every payload the tests allocate sits between two 256-byte guard zones filled with a sentinel (the stand-in for a memory
# checker, which is closed on this machine): a kernel that writes one cell before or past a relation's payload changes a guard,
# and download() / check_status() look at the guards of every live guarded relation.
GUARD_BYTES = 256
_SENTINEL = 0x5A
_guarded = weakref.WeakSet()


def _guarded_relation(extents, splits, dtype, init: torch.Tensor | None = None) -> ja.Relation:
    dt_code = {torch.bfloat16: ja.JA_BF16, torch.float16: ja.JA_F16, torch.float32: ja.JA_F32}[dtype]
    nbytes = ja.ja_relation_bytes([int(e) for e in extents], [list(map(int, sp)) for sp in splits], dt_code)
    nbytes = (nbytes + 127) // 128 * 128
    raw = torch.full((nbytes + 2 * GUARD_BYTES,), _SENTINEL, dtype=torch.uint8, device="cuda")
    assert raw.data_ptr() % 128 == 0
    inner = raw[GUARD_BYTES: GUARD_BYTES + nbytes].view(dtype)
    if init is None:
        inner.zero_()
    else:
        inner.zero_()
        inner[: init.numel()].copy_(init)
    r = ja.Relation(list(extents), splits, dtype, inner)
    r._raw = raw
    _guarded.add(r)
    return r


def check_guards(rel=None):
    for r in ([rel] if rel is not None else list(_guarded)):
        raw = getattr(r, "_raw", None)
        if raw is None:
            continue
        front, back = raw[:GUARD_BYTES], raw[-GUARD_BYTES:]
        assert bool((front == _SENTINEL).all()) and bool((back == _SENTINEL).all()), \
            f"a kernel wrote outside the payload of a relation with extents {r.extents}"


def upload(dense: torch.Tensor, splits) -> ja.Relation:
    """dense CPU tensor -> relation on the GPU, packed on the host by the oracle's key-table code."""
    payload = blocked.pack(np_bits(dense), splits)
    return _guarded_relation(list(dense.shape), splits, dense.dtype, from_bits(payload, dense.dtype).cuda())


def empty_like_tiling(extents, splits, dtype, fill=None) -> ja.Relation:
    r = _guarded_relation(extents, splits, dtype)
    if fill is not None:
        r.payload.fill_(fill)
    return r


def download(rel: ja.Relation) -> np.ndarray:
    """relation -> dense fp64 numpy tensor, unpacked on the host by the oracle's key-table code."""
    torch.cuda.synchronize()
    check_guards(rel)
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
    torch.cuda.synchronize()
    check_guards()
    assert ja.ja_stream_status(torch.cuda.current_stream().cuda_stream) == 0, "device status word set (bounded wait expired)"


# relative Frobenius error against the fp64 oracle: ten half-ulps of the storage type (bf16 2^-9, f16 2^-12)
TOL = {torch.float32: 1e-5, torch.bfloat16: 2e-2, torch.float16: 2.5e-3}
