"""TEST INFRASTRUCTURE ONLY -- engine T2: Definition 3.7 ("Implementation") taken literally.

Given an einsum signature and, for every named index, a list of split points
(Section 3.3: the intervals handed to an abstract operator), build the join-agg
spec J = {F_1..F_p} with one function specification per combination of
intervals, run the concrete operator on every joined tuple of projected
sub-tensors, aggregate partial outputs that share an output type, recompose.

The same module produces, independently of the GPU library, the integer
bookkeeping that the library must reproduce bit for bit: key tables of a tensor
relation, the tuple list of a spec, the cost-model counts of Section 4.3 and the
overlay atoms of Section 5.3.

Canonical orders (the paper leaves a spec a *set*): index letters in order of
first appearance in the signature (inputs left to right, then output); function
specifications row-major over the interval grid in that letter order (last
letter fastest); blocks of a relation row-major over the relation's own index
order; atoms row-major over the overlay grid.
"""
from __future__ import annotations

import itertools

import numpy as np

from . import core

ALIGN = 128  # bytes: every block of a relation payload starts on a 128-byte boundary


def equal_splits(extent: int, n: int):
    """Near-equal intervals: interval s of n is [floor(s*E/n), floor((s+1)*E/n))."""
    return [(s * extent) // n for s in range(n + 1)]


def check_splits(extent: int, splits) -> None:
    """Tiling condition in one dimension (Definition 3.2): cover [0, extent) with disjoint non-empty intervals."""
    s = list(splits)
    if len(s) < 2 or s[0] != 0 or s[-1] != extent or any(b <= a for a, b in zip(s, s[1:])):
        raise ValueError(f"splits {s} do not tile [0, {extent})")


class Spec:
    """The join-agg spec J for one interval decomposition (Definition 3.6 / Section 3.3)."""

    def __init__(self, einsum: str, parts: dict, band=None, induced=None, segments=None):
        """band = (k_letter, q_letter): the selection k <= q lifted to blocks -- a cell of the interval grid is
        a function specification only if some key position of its k interval is <= some query position of its
        q interval (attention with the key index split inside a sequence).
        induced = (h_letter, g_letter, group): h is not shardable by itself (Example 3.10, grouped-query attention):
        its intervals are those of g scaled by `group`, and a function specification pairs interval m of g with
        interval m of h only.
        segments = (k_letter, q_letter, ends): packed sequences ending at `ends` (Example 3.10): attention never
        crosses a sequence boundary, so a cell is a function specification only if its q and k intervals lie in
        the same sequence; both indices may be split at sequence ends (and, in the extended form, inside)."""
        self.einsum = einsum
        self.ins, self.out, self.letters = core.parse_einsum(einsum)
        self.parts = {c: list(parts[c]) for c in self.letters}
        for c in self.letters:
            check_splits(self.parts[c][-1], self.parts[c])
        self.nb = {c: len(self.parts[c]) - 1 for c in self.letters}
        self.extent = {c: self.parts[c][-1] for c in self.letters}
        grid = [range(self.nb[c]) for c in self.letters]
        self.cells = list(itertools.product(*grid))  # row-major, last letter fastest
        if band is not None:
            ik, iq = self.letters.index(band[0]), self.letters.index(band[1])
            self.cells = [c for c in self.cells
                          if self.parts[band[0]][c[ik]] <= self.parts[band[1]][c[iq] + 1] - 1]
        if induced is not None:
            h, g, group = induced
            if self.parts[h] != [group * x for x in self.parts[g]]:
                raise ValueError(f"intervals of '{h}' must be those of '{g}' scaled by {group}")
            ih, ig = self.letters.index(h), self.letters.index(g)
            self.cells = [c for c in self.cells if c[ih] == c[ig]]
        if segments is not None:
            kl, ql, ends = segments
            for l in (kl, ql):
                if any(e not in self.parts[l] for e in ends):
                    raise ValueError(f"index '{l}' may only be cut so that every sequence end is a split point")
            seq_of = lambda x: sum(1 for e in ends if e <= x)   # sequence that position x belongs to
            ik, iq = self.letters.index(kl), self.letters.index(ql)
            self.cells = [c for c in self.cells
                          if seq_of(self.parts[kl][c[ik]]) == seq_of(self.parts[ql][c[iq]])]
        self.p = len(self.cells)

    # -- per-operand helpers (operand = index into self.ins, or -1 for the output) --------------
    def term(self, operand: int) -> str:
        return self.out if operand < 0 else self.ins[operand]

    def block_coords(self, cell, operand: int):
        return tuple(cell[self.letters.index(c)] for c in self.term(operand))

    def flat_key(self, coords, operand: int) -> int:
        k = 0
        for c, x in zip(self.term(operand), coords):
            k = k * self.nb[c] + x
        return k

    def bounds(self, coords, operand: int):
        lo = [self.parts[c][x] for c, x in zip(self.term(operand), coords)]
        hi = [self.parts[c][x + 1] for c, x in zip(self.term(operand), coords)]
        return lo, hi

    # -- tables -----------------------------------------------------------------------------------
    def tuples(self):
        """in_keys int32 [p, n_in], out_keys int32 [p]: flat block keys of every function specification."""
        ink = np.zeros((self.p, len(self.ins)), dtype=np.int32)
        outk = np.zeros(self.p, dtype=np.int32)
        for t, cell in enumerate(self.cells):
            for k in range(len(self.ins)):
                ink[t, k] = self.flat_key(self.block_coords(cell, k), k)
            outk[t] = self.flat_key(self.block_coords(cell, -1), -1)
        return ink, outk

    def operand_tiling(self, operand: int):
        """(nblocks per dim, list of split-point lists) = in_k(J) or out(J) as a grid."""
        t = self.term(operand)
        return [self.nb[c] for c in t], [self.parts[c] for c in t]

    def multiplicity(self):
        """m per distinct output type, indexed by flat output key."""
        _, outk = self.tuples()
        n_out = int(np.prod([self.nb[c] for c in self.out])) if self.out else 1
        return np.bincount(outk, minlength=n_out)

    def cost_terms(self):
        """Section 4.3: join sub-cost  sum_F sum_k |I(T^(i_k))|  and aggregation sub-cost
        sum over distinct output types of (m - 1) |I(T^(o))|."""
        join = 0
        for cell in self.cells:
            for k in range(len(self.ins)):
                lo, hi = self.bounds(self.block_coords(cell, k), k)
                join += int(np.prod([h - l for l, h in zip(lo, hi)])) if lo else 1
        aggc = 0
        m = self.multiplicity()
        out_grid = [range(self.nb[c]) for c in self.out]
        for coords in itertools.product(*out_grid):
            lo, hi = self.bounds(coords, -1)
            card = int(np.prod([h - l for l, h in zip(lo, hi)])) if lo else 1
            aggc += (int(m[self.flat_key(coords, -1)]) - 1) * card
        return join, aggc


def relation_keys(extents, splits, elsize: int):
    """Key table of a tensor relation: for every block, in row-major key order, its block
    coordinates, its tensor type (lower / upper bound vectors -- the key of the paper) and the
    byte offset of its dense row-major payload.  Blocks lie back to back, each 128-byte aligned."""
    rank = len(extents)
    for e, s in zip(extents, splits):
        check_splits(e, s)
    grid = [range(len(s) - 1) for s in splits]
    coords, lower, upper, offsets = [], [], [], []
    off = 0
    for c in itertools.product(*grid):
        lo = [splits[d][c[d]] for d in range(rank)]
        hi = [splits[d][c[d] + 1] for d in range(rank)]
        coords.append(list(c)); lower.append(lo); upper.append(hi); offsets.append(off)
        nbytes = int(np.prod([h - l for l, h in zip(lo, hi)])) * elsize
        off += (nbytes + ALIGN - 1) // ALIGN * ALIGN
    return (np.array(coords, dtype=np.int32).reshape(-1, rank), np.array(lower, dtype=np.int64).reshape(-1, rank),
            np.array(upper, dtype=np.int64).reshape(-1, rank), np.array(offsets, dtype=np.int64), off)


def pack(dense: np.ndarray, splits, elsize: int | None = None) -> np.ndarray:
    """Dense tensor -> relation payload (flat array of the same dtype, alignment gaps zero)."""
    elsize = elsize or dense.dtype.itemsize
    _, lower, upper, offsets, total = relation_keys(dense.shape, splits, elsize)
    out = np.zeros(total // elsize, dtype=dense.dtype)
    for lo, hi, off in zip(lower, upper, offsets):
        blk = dense[tuple(slice(l, h) for l, h in zip(lo, hi))]
        out[off // elsize: off // elsize + blk.size] = blk.reshape(-1)
    return out


def unpack(payload: np.ndarray, extents, splits, elsize: int | None = None) -> np.ndarray:
    """Relation payload -> dense tensor (the Recompose step of Definition 3.7)."""
    elsize = elsize or payload.dtype.itemsize
    _, lower, upper, offsets, _ = relation_keys(extents, splits, elsize)
    out = np.zeros(extents, dtype=payload.dtype)
    for lo, hi, off in zip(lower, upper, offsets):
        shape = [h - l for l, h in zip(lo, hi)]
        n = int(np.prod(shape))
        out[tuple(slice(l, h) for l, h in zip(lo, hi))] = payload[off // elsize: off // elsize + n].reshape(shape)
    return out


def overlay_atoms(src_splits, dst_splits):
    """Section 5.3: per dimension, the union of the bounds of every block of the producer tiling and
    of the consumer tiling; the cells of the resulting grid are the atoms.  Returns the overlay split
    points and, per atom in row-major order, (lower, upper, flat source block, flat destination block)."""
    rank = len(src_splits)
    over = [sorted(set(src_splits[d]) | set(dst_splits[d])) for d in range(rank)]

    def owner(splits_d, x):  # index of the interval of splits_d containing x
        return int(np.searchsorted(np.asarray(splits_d), x, side="right") - 1)

    atoms = []
    for cell in itertools.product(*[range(len(o) - 1) for o in over]):
        lo = [over[d][cell[d]] for d in range(rank)]
        hi = [over[d][cell[d] + 1] for d in range(rank)]
        sb = db = 0
        for d in range(rank):
            sb = sb * (len(src_splits[d]) - 1) + owner(src_splits[d], lo[d])
            db = db * (len(dst_splits[d]) - 1) + owner(dst_splits[d], lo[d])
        atoms.append((lo, hi, sb, db))
    return over, atoms


def repartition(payload: np.ndarray, extents, src_splits, dst_splits) -> np.ndarray:
    """decompose + recompose (Section 5.3): copy every atom from its source block to its destination block."""
    es = payload.dtype.itemsize
    _, slo, _, soff, _ = relation_keys(extents, src_splits, es)
    _, dlo, dup, doff, dtotal = relation_keys(extents, dst_splits, es)
    _, sl2, sup, _, _ = relation_keys(extents, src_splits, es)
    out = np.zeros(dtotal // es, dtype=payload.dtype)
    _, atoms = overlay_atoms(src_splits, dst_splits)
    for lo, hi, sb, db in atoms:
        sshape = [int(u - l) for l, u in zip(slo[sb], sup[sb])]
        dshape = [int(u - l) for l, u in zip(dlo[db], dup[db])]
        sblk = payload[soff[sb] // es: soff[sb] // es + int(np.prod(sshape))].reshape(sshape)
        dblk = out[doff[db] // es: doff[db] // es + int(np.prod(dshape))].reshape(dshape)
        s_sl = tuple(slice(l - b, h - b) for l, h, b in zip(lo, hi, slo[sb]))
        d_sl = tuple(slice(l - b, h - b) for l, h, b in zip(lo, hi, dlo[db]))
        dblk[d_sl] = sblk[s_sl]
    return out


def t2_join_agg(einsum: str, parts: dict, inputs, fn="mul", agg="sum", params=()):
    """Definition 3.7 verbatim.  (1) Join: for each F project every input and run f[F] (the scalar
    engine restricted to F's boxes).  (2) Aggregate: (+)-combine, in ascending order of F, the partial
    outputs that share an output type.  (3) Recompose: place each aggregated block by its bounds."""
    spec = Spec(einsum, parts)
    arrs = [np.asarray(a, dtype=np.float64) for a in inputs]
    partial = {}
    for cell in spec.cells:
        proj = []
        for k in range(len(spec.ins)):
            lo, hi = spec.bounds(spec.block_coords(cell, k), k)
            proj.append(arrs[k][tuple(slice(l, h) for l, h in zip(lo, hi))])
        ext = {c: spec.parts[c][x + 1] - spec.parts[c][x] for c, x in zip(spec.letters, cell)}
        part = core.join_agg(einsum, proj, fn=fn, agg=agg, params=params, extents=ext)
        okey = spec.block_coords(cell, -1)
        if okey not in partial:
            partial[okey] = part
        elif agg == "sum":
            partial[okey] = partial[okey] + part
        elif agg == "max":
            partial[okey] = np.maximum(partial[okey], part)
        else:
            raise ValueError("two function specifications share an output type but there is no aggregation")
    out = np.full([spec.extent[c] for c in spec.out], np.nan)
    for okey, blk in partial.items():
        lo, hi = spec.bounds(okey, -1)
        out[tuple(slice(l, h) for l, h in zip(lo, hi))] = blk
    assert not np.isnan(out).any(), "output types do not tile the output (tiling condition)"
    return out


# ---------------------------------------------------------------------------------------------------
# Producers compiled "through their join" and the aggregating relayout that consumes them
# (Section 5.1: the unaggregated partial blocks of a producer stay where they were computed and the
# consumer aggregates them as it brings them where they are needed; Section 5.3: decompose every
# copy into atoms, (+)-aggregate the m copies of each atom, recompose the consumer's blocks).
# ---------------------------------------------------------------------------------------------------
def join_partials(einsum: str, parts: dict, inputs, fn="mul", agg="sum", params=(), dtype=None):
    """Step (1) of Definition 3.7 alone.  Returns the dense tensor P[c, out...]: for every output type,
    copy c is the output of the c-th function specification (ascending F) that has this output type.
    Every output type must have the same multiplicity m.  Each partial block is rounded once to
    `dtype` (its store); the per-specification reduction over the indices inside the block uses `agg`."""
    spec = Spec(einsum, parts)
    mult = spec.multiplicity()
    m = int(mult.reshape(-1)[0])
    if not (mult == m).all():
        raise ValueError("output types have different multiplicities")
    arrs = [np.asarray(a, dtype=np.float64) for a in inputs]
    out = np.full([m] + [spec.extent[c] for c in spec.out], np.nan)
    seen = {}
    for cell in spec.cells:
        proj = []
        for k in range(len(spec.ins)):
            lo, hi = spec.bounds(spec.block_coords(cell, k), k)
            proj.append(arrs[k][tuple(slice(l, h) for l, h in zip(lo, hi))])
        ext = {c: spec.parts[c][x + 1] - spec.parts[c][x] for c, x in zip(spec.letters, cell)}
        part = core.join_agg(einsum, proj, fn=fn, agg=agg, params=params, extents=ext)
        okey = spec.block_coords(cell, -1)
        c = seen.get(okey, 0)
        seen[okey] = c + 1
        lo, hi = spec.bounds(okey, -1)
        out[(c,) + tuple(slice(l, h) for l, h in zip(lo, hi))] = part
    assert not np.isnan(out).any()
    return core.round_to(out, dtype) if dtype in ("f32", "bf16", "f16") else out


def partial_splits(m: int, splits):
    """Tiling of a partial relation: the copy index in front, cut into its m unit intervals."""
    return [list(range(m + 1))] + [list(s) for s in splits]


def aggregate_repartition(partials: np.ndarray, src_splits, dst_splits, agg="sum", dtype=None) -> np.ndarray:
    """Section 5.3 on one processor.  `partials` is the dense fp64 tensor P[c, x...] of a partial
    relation whose blocks are (copy c) x (block of src_splits).  decompose: every copy of every
    producer block is sliced into the atoms of the overlay of src_splits and dst_splits; aggregate:
    the m copies of an atom are (+)-combined in ascending copy order; recompose: the aggregated atoms
    of a consumer block are concatenated.  One rounding to `dtype` at the consumer's store.  Returns
    the dense tensor (the caller packs it with dst_splits)."""
    P = np.asarray(partials, dtype=np.float64)
    m = P.shape[0]
    out = np.full(P.shape[1:], np.nan)
    _, atoms = overlay_atoms(src_splits, dst_splits)
    for lo, hi, _sb, _db in atoms:
        sl = tuple(slice(l, h) for l, h in zip(lo, hi))
        acc = P[(0,) + sl].copy()
        for c in range(1, m):
            if agg == "sum":
                acc = acc + P[(c,) + sl]
            elif agg == "max":
                acc = np.maximum(acc, P[(c,) + sl])
            else:
                raise ValueError("an atom has several copies but there is no aggregation")
        out[sl] = acc
    assert not np.isnan(out).any()
    return core.round_to(out, dtype) if dtype in ("f32", "bf16", "f16") else out
