"""TEST INFRASTRUCTURE ONLY -- loader and thin numpy wrappers for the C oracle.

The oracle evaluates join-agg specs in the degenerate relational form of the
paper (Section 1: key = one cell, sub-tensor = one scalar; Definition 3.7) in
fp64.  Nothing here is imported by the GPU library or its Python binding.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ja_oracle.c")
_LIB = os.path.join(_HERE, "libja_oracle.so")

MAX_IDX = 12

FN = {"mul": 0, "ident": 1, "square": 2, "add": 3, "silu_mul": 4, "rms_scale": 5, "exp_sub": 6,
      "exp_sub_div": 7}
AGG = {"none": 0, "sum": 1, "max": 2}


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP) if the shared object is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB)
        L.orc_round_bf16.restype = ctypes.c_double
        L.orc_round_bf16.argtypes = [ctypes.c_double]
        L.orc_round_f32.restype = ctypes.c_double
        L.orc_round_f32.argtypes = [ctypes.c_double]
        L.orc_num_threads.restype = ctypes.c_int
        L.orc_join_agg.restype = ctypes.c_int
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def round_to(a, dtype: str) -> np.ndarray:
    """Round fp64 values to the nearest value of `dtype` ('f32' | 'bf16' | 'f16'), ties to even; result stays fp64."""
    out = _f64(a).copy()
    lib().orc_round_array(_ptr(out), ctypes.c_int64(out.size), ctypes.c_int({"f32": 0, "bf16": 1, "f16": 2}[dtype]))
    return out


def parse_einsum(einsum: str):
    """'ij,jk->ik' -> (list of input index strings, output index string, letters in order of first appearance)."""
    lhs, rhs = einsum.replace(" ", "").split("->")
    ins = lhs.split(",")
    letters = []
    for term in ins + [rhs]:
        for ch in term:
            if ch not in letters:
                letters.append(ch)
    return ins, rhs, letters


def join_agg(einsum: str, inputs, fn: str = "mul", agg: str = "sum", params=(), pred=None,
             extents: dict | None = None) -> np.ndarray:
    """Engine T1: scalar-keyed natural join of the input relations on their shared index
    letters, g applied per joined tuple, GROUP BY the output letters with `agg`.

    pred = (lo_letter, hi_letter) keeps only tuples with value(lo) <= value(hi).
    """
    ins, rhs, letters = parse_einsum(einsum)
    arrs = [_f64(a) for a in inputs]
    ext = dict(extents or {})
    for term, a in zip(ins, arrs):
        assert a.ndim == len(term), (term, a.shape)
        for ch, n in zip(term, a.shape):
            assert ext.setdefault(ch, n) == n, f"extent clash on {ch}"
    n_idx = len(letters)
    extent = (ctypes.c_int64 * n_idx)(*[ext[ch] for ch in letters])
    n_in = len(ins)
    in_rank = (ctypes.c_int * n_in)(*[len(t) for t in ins])
    in_idx = (ctypes.c_int * (n_in * MAX_IDX))()
    for k, term in enumerate(ins):
        for d, ch in enumerate(term):
            in_idx[k * MAX_IDX + d] = letters.index(ch)
    data = (ctypes.c_void_p * n_in)(*[a.ctypes.data for a in arrs])
    out_idx = (ctypes.c_int * max(1, len(rhs)))(*[letters.index(ch) for ch in rhs])
    out = np.empty([ext[ch] for ch in rhs], dtype=np.float64)
    p = _f64(list(params) if len(params) else [0.0])
    lo, hi = (-1, -1) if pred is None else (letters.index(pred[0]), letters.index(pred[1]))
    rc = lib().orc_join_agg(ctypes.c_int(n_idx), extent, ctypes.c_int(n_in), in_rank, in_idx, data,
                            ctypes.c_int(len(rhs)), out_idx, _ptr(out), ctypes.c_int(FN[fn]), _ptr(p),
                            ctypes.c_int(AGG[agg]), ctypes.c_int(lo), ctypes.c_int(hi))
    if rc != 0:
        raise ValueError(f"orc_join_agg rejected the request (code {rc})")
    return out


def matmul(A, B) -> np.ndarray:
    """Plain-definition matrix multiply (Example 3.4): join on j, SUM over j ascending."""
    A, B = _f64(A), _f64(B)
    M, J = A.shape
    J2, N = B.shape
    assert J == J2
    C = np.empty((M, N), dtype=np.float64)
    lib().orc_matmul(_ptr(A), _ptr(B), _ptr(C), ctypes.c_int64(M), ctypes.c_int64(J), ctypes.c_int64(N))
    return C


def attention(Q, K, V, scale: float, causal: bool = True, qpos=None) -> np.ndarray:
    """Plain-definition dot-product attention on [b, s, h, d] operands, unrounded inside.

    Q may hold a subset of the query rows of each sequence; qpos then gives each row's position."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    B, Sq, H, D = Q.shape
    Sk = K.shape[1]
    assert K.shape == V.shape == (B, Sk, H, D)
    if qpos is None:
        assert Sq == Sk or not causal
        qp = None
    else:
        qpos = np.ascontiguousarray(np.asarray(qpos, dtype=np.int64))
        assert qpos.shape == (Sq,) and (not causal or qpos.max() < Sk)
        qp = _ptr(qpos)
    O = np.empty_like(Q)
    lib().orc_attention(_ptr(Q), _ptr(K), _ptr(V), _ptr(O), ctypes.c_int64(B), ctypes.c_int64(Sq),
                        ctypes.c_int64(Sk), ctypes.c_int64(H), ctypes.c_int64(D), ctypes.c_double(scale),
                        ctypes.c_int(int(causal)), qp)
    return O
