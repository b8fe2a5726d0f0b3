"""TEST INFRASTRUCTURE ONLY -- the literal relational reading of a join-agg.

Engine T0: every tensor is materialised as a relation of (key columns, scalar
value) tuples (paper Section 1, degenerate case of a tensor relation), the
inputs are combined with NATURAL JOINs on their shared index columns, the
scalar function g is applied to every joined tuple and the result is grouped by
the output index columns with the aggregation operator.  Plus a brute-force
einsum checker (pure Python loops over every index assignment, no relations).
"""
from __future__ import annotations

import itertools
import math

import numpy as np

from .core import parse_einsum


class Relation:
    """cols: tuple of index letters; keys: int64 [n, len(cols)]; vals: list of float64 [n] value columns."""

    def __init__(self, cols, keys, vals):
        self.cols, self.keys, self.vals = tuple(cols), keys, list(vals)

    def __len__(self):
        return self.keys.shape[0]


def to_relation(arr, letters: str) -> Relation:
    arr = np.asarray(arr, dtype=np.float64)
    assert len(set(letters)) == len(letters) == arr.ndim
    grids = np.indices(arr.shape, dtype=np.int64).reshape(arr.ndim, -1).T
    return Relation(letters, np.ascontiguousarray(grids), [arr.reshape(-1).copy()])


def _composite(keys, col_ids, radix):
    comp = np.zeros(keys.shape[0], dtype=np.int64)
    for c, r in zip(col_ids, radix):
        comp = comp * r + keys[:, c]
    return comp


def natural_join(R: Relation, S: Relation, extent: dict) -> Relation:
    """Sort-merge equi-join on the columns R and S share (cartesian product if none)."""
    shared = [c for c in R.cols if c in S.cols]
    radix = [extent[c] for c in shared]
    rk = _composite(R.keys, [R.cols.index(c) for c in shared], radix)
    sk = _composite(S.keys, [S.cols.index(c) for c in shared], radix)
    order = np.argsort(sk, kind="stable")
    sk_sorted = sk[order]
    lo = np.searchsorted(sk_sorted, rk, side="left")
    hi = np.searchsorted(sk_sorted, rk, side="right")
    cnt = hi - lo
    r_rows = np.repeat(np.arange(len(R), dtype=np.int64), cnt)
    starts = np.repeat(lo, cnt)
    within = np.arange(cnt.sum(), dtype=np.int64) - np.repeat(np.cumsum(cnt) - cnt, cnt)
    s_rows = order[starts + within]
    extra = [c for c in S.cols if c not in R.cols]
    keys = np.concatenate([R.keys[r_rows]] + [S.keys[s_rows][:, [S.cols.index(c)]] for c in extra], axis=1)
    vals = [v[r_rows] for v in R.vals] + [v[s_rows] for v in S.vals]
    return Relation(R.cols + tuple(extra), keys, vals)


def _g(fn: str, v, p):
    if fn == "mul":
        r = v[0]
        for x in v[1:]:
            r = r * x
        return r
    if fn == "ident":
        return v[0]
    if fn == "square":
        return v[0] * v[0]
    if fn == "add":
        r = v[0]
        for x in v[1:]:
            r = r + x
        return r
    if fn == "silu_mul":
        return v[0] / (1.0 + np.exp(-v[0])) * v[1]
    if fn == "rms_scale":
        return v[0] * (1.0 / np.sqrt(v[1] / p[1] + p[0])) * v[2]
    if fn == "exp_sub":
        return np.exp(v[0] - v[1])
    if fn == "exp_sub_div":
        return np.exp(v[0] - v[1]) / v[2]
    raise ValueError(fn)


def t0_join_agg(einsum: str, inputs, fn="mul", agg="sum", params=(), pred=None) -> np.ndarray:
    """Materialising tuple engine: join, select, map g, group by, fold in ascending key order."""
    ins, rhs, letters = parse_einsum(einsum)
    extent = {}
    for term, a in zip(ins, inputs):
        for ch, n in zip(term, np.shape(a)):
            extent[ch] = n
    rels = [to_relation(a, t) for a, t in zip(inputs, ins)]
    J = rels[0]
    for S in rels[1:]:
        J = natural_join(J, S, extent)
    if pred is not None:  # selection sigma_{lo <= hi}
        keep = J.keys[:, J.cols.index(pred[0])] <= J.keys[:, J.cols.index(pred[1])]
        J = Relation(J.cols, J.keys[keep], [v[keep] for v in J.vals])
    g = _g(fn, J.vals, params)
    out_shape = [extent[c] for c in rhs]
    okey = _composite(J.keys, [J.cols.index(c) for c in rhs], out_shape)
    agg_cols = [c for c in letters if c not in rhs]
    akey = _composite(J.keys, [J.cols.index(c) for c in agg_cols], [extent[c] for c in agg_cols])
    order = np.lexsort((akey, okey))  # group by output key, ascending aggregated key inside a group
    okey, g = okey[order], g[order]
    n_out = int(np.prod(out_shape)) if out_shape else 1
    if agg == "sum":
        out = np.zeros(n_out)
        np.add.at(out, okey, g)       # unbuffered: folds sequentially in the sorted order
    elif agg == "max":
        out = np.full(n_out, -np.inf)
        np.maximum.at(out, okey, g)
    else:
        assert not agg_cols and len(np.unique(okey)) == len(okey)
        out = np.full(n_out, np.nan)
        out[okey] = g
    return out.reshape(out_shape)


def brute_einsum(einsum: str, inputs, fn="mul", agg="sum", params=(), pred=None) -> np.ndarray:
    """Nested loops over every assignment of every index letter: out[o] (+)= g(...). Tiny inputs only."""
    ins, rhs, letters = parse_einsum(einsum)
    arrs = [np.asarray(a, dtype=np.float64) for a in inputs]
    extent = {}
    for term, a in zip(ins, arrs):
        for ch, n in zip(term, a.shape):
            extent[ch] = n
    out_shape = tuple(extent[c] for c in rhs)
    ident = {"sum": 0.0, "max": -math.inf, "none": math.nan}[agg]
    out = np.full(out_shape, ident, dtype=np.float64)
    for assign in itertools.product(*[range(extent[c]) for c in letters]):
        env = dict(zip(letters, assign))
        if pred is not None and not env[pred[0]] <= env[pred[1]]:
            continue
        v = [float(a[tuple(env[c] for c in term)]) for a, term in zip(arrs, ins)]
        if fn == "mul":
            g = math.prod(v)
        elif fn == "ident":
            g = v[0]
        elif fn == "square":
            g = v[0] * v[0]
        elif fn == "add":
            g = sum(v[1:], v[0])
        elif fn == "silu_mul":
            g = v[0] / (1.0 + math.exp(-v[0])) * v[1]
        elif fn == "rms_scale":
            g = v[0] * (1.0 / math.sqrt(v[1] / params[1] + params[0])) * v[2]
        elif fn == "exp_sub":
            g = math.exp(v[0] - v[1])
        elif fn == "exp_sub_div":
            g = math.exp(v[0] - v[1]) / v[2]
        else:
            raise ValueError(fn)
        o = tuple(env[c] for c in rhs)
        if agg == "sum":
            out[o] = out[o] + g
        elif agg == "max":
            out[o] = max(out[o], g)
        else:
            out[o] = g
    return out
