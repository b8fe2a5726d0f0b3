"""Small conveniences over the binding for callers that hold relation payloads in torch tensors:
allocation of a payload buffer of the right size, handle lifetime, and the current stream.
No arithmetic and no data movement happens here (packing a dense tensor into a relation is itself
a ja_repartition from the one-block tiling)."""
from __future__ import annotations

import torch

from . import binding as B

_DT = {torch.float32: B.JA_F32, torch.bfloat16: B.JA_BF16, torch.float16: B.JA_F16}


def equal_splits(extent: int, n: int):
    """Near-equal intervals: interval s of n is [floor(s*E/n), floor((s+1)*E/n))."""
    return [(s * extent) // n for s in range(n + 1)]


def current_stream() -> int:
    return torch.cuda.current_stream().cuda_stream


class Relation:
    """A tensor relation whose payload lives in a torch CUDA tensor (flat, 128-byte aligned)."""

    def __init__(self, extents, splits, dtype=torch.bfloat16, payload: torch.Tensor | None = None, device="cuda"):
        self.extents = [int(e) for e in extents]
        self.splits = [[int(x) for x in s] for s in splits]
        self.dtype = dtype
        nbytes = B.ja_relation_bytes(self.extents, self.splits, _DT[dtype])
        if payload is None:
            payload = torch.zeros(nbytes // dtype.itemsize, dtype=dtype, device=device)
        assert payload.is_cuda and payload.is_contiguous() and payload.dtype == dtype
        assert payload.numel() * dtype.itemsize >= nbytes
        self.payload = payload
        self.nbytes = nbytes
        self.handle = B.ja_relation_create(self.extents, self.splits, _DT[dtype], payload.data_ptr(),
                                           payload.numel() * dtype.itemsize)

    def view_as(self, extents, splits) -> "Relation":
        """Another relation handle over the SAME payload (a reshape of the tensor whose block layout coincides)."""
        return Relation(extents, splits, self.dtype, self.payload)

    def close(self):
        if getattr(self, "handle", None):
            B.ja_relation_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Spec:
    def __init__(self, einsum: str, parts: dict, fn="mul", fn_params=(), agg="sum"):
        self.einsum, self.parts = einsum, parts
        self.handle = B.ja_spec_create(einsum, parts, fn, fn_params, agg)

    def execute(self, inputs, output, stream: int | None = None):
        """output: one relation, or a list of relations for multi-output specs (attention: [O, lse])."""
        outs = output if isinstance(output, (list, tuple)) else [output]
        B.ja_execute(self.handle, [r.handle for r in inputs], [r.handle for r in outs],
                     current_stream() if stream is None else stream)

    def execute_join(self, inputs, partials: Relation, stream: int | None = None):
        B.ja_execute_join(self.handle, [r.handle for r in inputs], partials.handle, current_stream() if stream is None else stream)

    def close(self):
        if getattr(self, "handle", None):
            B.ja_spec_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def repartition(src: Relation, dst: Relation, stream: int | None = None):
    B.ja_repartition(src.handle, dst.handle, current_stream() if stream is None else stream)


def repartition_agg(partials: Relation, agg: str, dst: Relation, stream: int | None = None):
    B.ja_repartition_agg(partials.handle, agg, dst.handle, current_stream() if stream is None else stream)


def attention_combine(o_parts, lse_parts, o: Relation, lse: Relation | None = None, stream: int | None = None):
    """Partial attention results over disjoint key ranges -> one result (the online-softmax aggregation as its own step)."""
    B.ja_attention_combine([r.handle for r in o_parts], [r.handle for r in lse_parts], o.handle, lse.handle if lse is not None else None,
                           current_stream() if stream is None else stream)


def partial_relation(copies: int, extents, splits, dtype) -> Relation:
    """Empty partial relation [c, x...]: the copy index in front, cut into its unit intervals."""
    return Relation([copies] + list(extents), [list(range(copies + 1))] + [list(s) for s in splits], dtype)


def from_dense(dense: torch.Tensor, splits) -> Relation:
    """Pack a dense row-major CUDA tensor into a relation: ja_repartition from the one-block tiling."""
    dense = dense.contiguous()
    one = Relation(list(dense.shape), [[0, e] for e in dense.shape], dense.dtype, _aligned_flat(dense))
    dst = Relation(list(dense.shape), splits, dense.dtype)
    repartition(one, dst)
    torch.cuda.current_stream().synchronize()
    one.close()
    return dst


def to_dense(rel: Relation) -> torch.Tensor:
    """Recompose a relation into a dense row-major tensor: ja_repartition to the one-block tiling."""
    one = Relation(rel.extents, [[0, e] for e in rel.extents], rel.dtype)
    repartition(rel, one)
    torch.cuda.current_stream().synchronize()
    n = 1
    for e in rel.extents:
        n *= e
    out = one.payload[:n].reshape(rel.extents).clone()
    one.close()
    return out


def _aligned_flat(t: torch.Tensor) -> torch.Tensor:
    flat = t.reshape(-1)
    pad = (-flat.numel() * flat.element_size()) % 128
    if pad or flat.data_ptr() % 128:
        buf = torch.zeros(flat.numel() + pad // flat.element_size(), dtype=t.dtype, device=t.device)
        buf[: flat.numel()] = flat
        return buf
    return flat
