"""ctypes binding of libja's C ABI: the same names, argument marshalling only.

Every step of the join-agg path runs inside libja's CUDA kernels; torch supplies device memory
(`tensor.data_ptr()`) and streams (`torch.cuda.current_stream().cuda_stream`) and nothing else.
There is no CPU fallback: if libja.so is missing and cannot be built, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libja.so")

JA_OK = 0
STATUS = {0: "JA_OK", 1: "JA_ERR_INVALID_ARG", 2: "JA_ERR_PARSE", 3: "JA_ERR_SHAPE", 4: "JA_ERR_TILING",
          5: "JA_ERR_PARTITION_MISMATCH", 6: "JA_ERR_DTYPE", 7: "JA_ERR_UNSUPPORTED", 8: "JA_ERR_ALIGNMENT",
          9: "JA_ERR_OOM", 10: "JA_ERR_CUDA", 11: "JA_ERR_TIMEOUT"}
JA_F32, JA_BF16, JA_F16 = 0, 1, 2
AGG = {"none": 0, "sum": 1, "max": 2, "online_softmax": 3}
FN = {"mul": 0, "ident": 1, "square": 2, "add": 3, "silu_mul": 4, "rms_scale": 5, "exp_sub": 6, "exp_sub_div": 7,
      "rope": 8, "attention": 9, "rmsnorm": 10, "softmax": 11, "matmul_add": 12, "matmul_rope": 13, "swiglu_up": 14}


class JaError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS.get(status, status)}: {message}")
        self.status = status
        self.status_name = STATUS.get(status, str(status))


class ja_plan_node_t(ctypes.Structure):
    _fields_ = [("einsum", ctypes.c_char_p), ("extents", ctypes.POINTER(ctypes.c_int64)),
                ("producers", ctypes.POINTER(ctypes.c_int32)), ("fixed_letters", ctypes.c_uint32)]


class ja_index_part_t(ctypes.Structure):
    _fields_ = [("name", ctypes.c_char), ("extent", ctypes.c_int64), ("nparts", ctypes.c_int32),
                ("splits", ctypes.POINTER(ctypes.c_int64))]


def _load() -> ctypes.CDLL:
    # make-like: compiles what is missing or older than its sources, nothing when libja.so is up to date (a library left over
    # from older sources would otherwise be loaded and lack the newer entry points)
    from .build import build
    build()
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    P = ctypes.POINTER
    sigs = {
        "ja_spec_create": [ctypes.c_char_p, P(ja_index_part_t), i32, ctypes.c_int, P(ctypes.c_double), i32, ctypes.c_int,
                           ctypes.c_int, P(vp)],
        "ja_spec_destroy": [vp],
        "ja_spec_num_tuples": [vp, P(i64), P(i32)],
        "ja_spec_get_tuples": [vp, vp, vp],
        "ja_spec_operand_tiling": [vp, i32, P(i32), vp, vp],
        "ja_spec_cost_terms": [vp, P(i64), P(i64)],
        "ja_relation_bytes": [i32, P(i64), P(i32), P(P(i64)), ctypes.c_int, P(ctypes.c_size_t)],
        "ja_relation_create": [i32, P(i64), P(i32), P(P(i64)), ctypes.c_int, vp, ctypes.c_size_t, P(vp)],
        "ja_relation_destroy": [vp],
        "ja_relation_num_blocks": [vp, P(i64), P(i32)],
        "ja_relation_get_keys": [vp, vp, vp, vp, vp],
        "ja_execute": [vp, P(vp), i32, P(vp), i32, vp],
        "ja_repartition": [vp, vp, vp],
        "ja_execute_join": [vp, P(vp), i32, vp, vp],
        "ja_plan_optimize": [P(ja_plan_node_t), i32, i32, P(i32), P(i64)],
        "ja_plan_cost": [P(ja_plan_node_t), i32, P(i32), P(i64)],
        "ja_attention_combine": [P(vp), P(vp), i32, vp, vp, vp],
        "ja_plan_optimize_graph": [P(ja_plan_node_t), i32, i32, P(i32), P(i64)],
        "ja_plan_select_greedy": [P(ja_plan_node_t), i32, i32, P(i32), P(i64)],
        "ja_repartition_agg": [vp, ctypes.c_int, vp, vp],
        "ja_overlay_atoms": [vp, vp, P(i64), vp, vp, vp, vp],
        "ja_stream_status": [vp, P(ctypes.c_int)],
        "ja_repartition_noalloc": [i32, P(i64), P(i32), P(P(i64)), P(i32), P(P(i64)), ctypes.c_int, vp, vp, vp],
        "ja_debug_set": [ctypes.c_char_p, i64],
        "ja_debug_wait_timeout": [vp, vp],
        "ja_debug_bounded_wait_host": [i64, i64, i64, i64, P(i64), P(i32), P(i32), P(i64)],
    }
    for name, argtypes in sigs.items():
        fn = getattr(lib, name)
        fn.argtypes = argtypes
        fn.restype = ctypes.c_int
    lib.ja_last_error.restype = ctypes.c_char_p
    lib.ja_version.restype = ctypes.c_char_p
    lib.ja_launch_count.restype = ctypes.c_int64
    return lib


LIB = _load()
LIB_PATH = _LIB_PATH


def _check(st: int):
    if st != JA_OK:
        raise JaError(st, LIB.ja_last_error().decode())


def _splits_arrays(splits):
    arrs = [(ctypes.c_int64 * len(s))(*[int(x) for x in s]) for s in splits]
    ptrs = (ctypes.POINTER(ctypes.c_int64) * len(arrs))(*[ctypes.cast(a, ctypes.POINTER(ctypes.c_int64)) for a in arrs])
    return arrs, ptrs


def ja_version() -> str:
    return LIB.ja_version().decode()


def ja_launch_count() -> int:
    return int(LIB.ja_launch_count())


def ja_spec_create(einsum: str, parts: dict, fn: str = "mul", fn_params=(), agg: str = "sum") -> int:
    """parts: {letter: split points}. Returns the opaque spec handle."""
    keep = []
    arr = (ja_index_part_t * len(parts))()
    for i, (name, sp) in enumerate(parts.items()):
        a = (ctypes.c_int64 * len(sp))(*[int(x) for x in sp])
        keep.append(a)
        arr[i].name = name.encode()
        arr[i].extent = int(sp[-1]) if len(sp) else 0
        arr[i].nparts = len(sp) - 1
        arr[i].splits = ctypes.cast(a, ctypes.POINTER(ctypes.c_int64))
    p = (ctypes.c_double * max(1, len(fn_params)))(*[float(x) for x in fn_params])
    out = ctypes.c_void_p()
    _check(LIB.ja_spec_create(einsum.encode(), arr, len(parts), FN[fn] if isinstance(fn, str) else int(fn), p, len(fn_params),
                              AGG[agg] if isinstance(agg, str) else int(agg), JA_F32, ctypes.byref(out)))
    return out.value


def ja_spec_destroy(spec: int):
    _check(LIB.ja_spec_destroy(spec))


def ja_spec_num_tuples(spec: int):
    p, n = ctypes.c_int64(), ctypes.c_int32()
    _check(LIB.ja_spec_num_tuples(spec, ctypes.byref(p), ctypes.byref(n)))
    return p.value, n.value


def ja_spec_get_tuples(spec: int):
    p, n = ja_spec_num_tuples(spec)
    ink = np.zeros((p, n), dtype=np.int32)
    outk = np.zeros(p, dtype=np.int32)
    _check(LIB.ja_spec_get_tuples(spec, ink.ctypes.data, outk.ctypes.data))
    return ink, outk


def ja_spec_operand_tiling(spec: int, operand: int):
    rank = ctypes.c_int32()
    _check(LIB.ja_spec_operand_tiling(spec, operand, ctypes.byref(rank), None, None))
    nb = np.zeros(rank.value, dtype=np.int32)
    _check(LIB.ja_spec_operand_tiling(spec, operand, ctypes.byref(rank), nb.ctypes.data, None))
    flat = np.zeros(int(nb.sum()) + rank.value, dtype=np.int64)
    _check(LIB.ja_spec_operand_tiling(spec, operand, ctypes.byref(rank), nb.ctypes.data, flat.ctypes.data))
    splits, w = [], 0
    for d in range(rank.value):
        splits.append(flat[w: w + nb[d] + 1].tolist())
        w += nb[d] + 1
    return nb.tolist(), splits


def ja_spec_cost_terms(spec: int):
    j, a = ctypes.c_int64(), ctypes.c_int64()
    _check(LIB.ja_spec_cost_terms(spec, ctypes.byref(j), ctypes.byref(a)))
    return j.value, a.value


def ja_relation_bytes(extents, splits, dtype: int) -> int:
    rank = len(extents)
    ext = (ctypes.c_int64 * rank)(*[int(e) for e in extents])
    npar = (ctypes.c_int32 * rank)(*[len(s) - 1 for s in splits])
    keep, ptrs = _splits_arrays(splits)
    out = ctypes.c_size_t()
    _check(LIB.ja_relation_bytes(rank, ext, npar, ptrs, dtype, ctypes.byref(out)))
    return out.value


def ja_relation_create(extents, splits, dtype: int, device_ptr: int, nbytes: int) -> int:
    rank = len(extents)
    ext = (ctypes.c_int64 * rank)(*[int(e) for e in extents])
    npar = (ctypes.c_int32 * rank)(*[len(s) - 1 for s in splits])
    keep, ptrs = _splits_arrays(splits)
    out = ctypes.c_void_p()
    _check(LIB.ja_relation_create(rank, ext, npar, ptrs, dtype, ctypes.c_void_p(device_ptr), nbytes, ctypes.byref(out)))
    return out.value


def ja_relation_destroy(rel: int):
    _check(LIB.ja_relation_destroy(rel))


def ja_relation_get_keys(rel: int):
    nb, rank = ctypes.c_int64(), ctypes.c_int32()
    _check(LIB.ja_relation_num_blocks(rel, ctypes.byref(nb), ctypes.byref(rank)))
    coords = np.zeros((nb.value, rank.value), dtype=np.int32)
    lower = np.zeros((nb.value, rank.value), dtype=np.int64)
    upper = np.zeros((nb.value, rank.value), dtype=np.int64)
    offs = np.zeros(nb.value, dtype=np.int64)
    _check(LIB.ja_relation_get_keys(rel, coords.ctypes.data, lower.ctypes.data, upper.ctypes.data, offs.ctypes.data))
    return coords, lower, upper, offs


def ja_execute(spec: int, inputs, outputs, stream: int = 0):
    ins = (ctypes.c_void_p * len(inputs))(*inputs)
    outs = (ctypes.c_void_p * len(outputs))(*outputs)
    _check(LIB.ja_execute(spec, ins, len(inputs), outs, len(outputs), ctypes.c_void_p(stream)))


def ja_repartition(src: int, dst: int, stream: int = 0):
    _check(LIB.ja_repartition(src, dst, ctypes.c_void_p(stream)))


def ja_execute_join(spec: int, inputs, partials: int, stream: int = 0):
    """Join only: every function spec's output goes, unaggregated, to its copy of the partial relation."""
    ins = (ctypes.c_void_p * len(inputs))(*inputs)
    _check(LIB.ja_execute_join(spec, ins, len(inputs), partials, ctypes.c_void_p(stream)))


def ja_repartition_agg(partials: int, agg, dst: int, stream: int = 0):
    """Aggregating relayout: the m copies of every atom are combined and stored in dst's tiling."""
    _check(LIB.ja_repartition_agg(partials, AGG[agg] if isinstance(agg, str) else int(agg), dst, ctypes.c_void_p(stream)))


JA_PLAN_MAX_LETTERS = 8


def _plan_nodes(ops):
    """ops: [{"einsum": str, "extents": {letter: n}, "inputs": [producer index | None, ...], "fixed": set of letters}]"""
    keep = []
    arr = (ja_plan_node_t * len(ops))()
    for i, op in enumerate(ops):
        lhs = op["einsum"].replace(" ", "").split("->")[0]
        letters = []
        for c in lhs.replace(",", ""):
            if c not in letters:
                letters.append(c)
        ext = (ctypes.c_int64 * len(letters))(*[op["extents"][c] for c in letters])
        prod = (ctypes.c_int32 * len(op["inputs"]))(*[-1 if q is None else q for q in op["inputs"]])
        fixed = sum(1 << letters.index(c) for c in op.get("fixed", ()))
        keep += [ext, prod]
        arr[i] = ja_plan_node_t(op["einsum"].encode(), ext, prod, fixed)
        op["_letters"] = letters
    return arr, keep


def ja_plan_optimize(ops, p: int):
    """Algorithm 1 on a computation tree. Returns (total cost, [{letter: intervals} per operator])."""
    arr, keep = _plan_nodes(ops)
    counts = (ctypes.c_int32 * (len(ops) * JA_PLAN_MAX_LETTERS))()
    total = ctypes.c_int64()
    _check(LIB.ja_plan_optimize(arr, len(ops), p, counts, ctypes.byref(total)))
    plan = [{c: counts[i * JA_PLAN_MAX_LETTERS + l] for l, c in enumerate(op["_letters"])} for i, op in enumerate(ops)]
    return total.value, plan


def ja_plan_optimize_graph(ops, p: int):
    """Section 4.5: a graph with multiply consumed tensors, cut into trees and optimised tree by tree."""
    arr, keep = _plan_nodes(ops)
    counts = (ctypes.c_int32 * (len(ops) * JA_PLAN_MAX_LETTERS))()
    total = ctypes.c_int64()
    _check(LIB.ja_plan_optimize_graph(arr, len(ops), p, counts, ctypes.byref(total)))
    plan = [{c: counts[i * JA_PLAN_MAX_LETTERS + l] for l, c in enumerate(op["_letters"])} for i, op in enumerate(ops)]
    return total.value, plan


def ja_attention_combine(o_parts, lse_parts, o: int, lse: int | None = None, stream: int = 0):
    """Handles of m partial attention results (O_c, lse_c) -> their online-softmax combination in `o` (and `lse`)."""
    m = len(o_parts)
    assert len(lse_parts) == m
    oa = (ctypes.c_void_p * m)(*o_parts)
    la = (ctypes.c_void_p * m)(*lse_parts)
    _check(LIB.ja_attention_combine(oa, la, m, ctypes.c_void_p(o), ctypes.c_void_p(lse) if lse else None, ctypes.c_void_p(stream)))


def ja_plan_select_greedy(ops, p: int):
    """Experiment 3's greedy selector: every operator takes its cheapest spec with the repartition sub-cost ignored."""
    arr, keep = _plan_nodes(ops)
    counts = (ctypes.c_int32 * (len(ops) * JA_PLAN_MAX_LETTERS))()
    total = ctypes.c_int64()
    _check(LIB.ja_plan_select_greedy(arr, len(ops), p, counts, ctypes.byref(total)))
    plan = [{c: counts[i * JA_PLAN_MAX_LETTERS + l] for l, c in enumerate(op["_letters"])} for i, op in enumerate(ops)]
    return total.value, plan


def ja_plan_cost(ops, plan) -> int:
    arr, keep = _plan_nodes(ops)
    counts = (ctypes.c_int32 * (len(ops) * JA_PLAN_MAX_LETTERS))()
    for i, op in enumerate(ops):
        for l, c in enumerate(op["_letters"]):
            counts[i * JA_PLAN_MAX_LETTERS + l] = plan[i][c]
    total = ctypes.c_int64()
    _check(LIB.ja_plan_cost(arr, len(ops), counts, ctypes.byref(total)))
    return total.value


def ja_repartition_noalloc(extents, src_splits, dst_splits, dtype: int, src_ptr: int, dst_ptr: int, stream: int = 0):
    """Relayout between two tilings given as plain split lists and raw device pointers. Unlike ja_repartition this
    never allocates (no cudaMalloc, no cached plan): for callers whose memory is fixed up front. Calls share one
    fixed plan table on the device, so do not let two of them overlap on the GPU."""
    rank = len(extents)
    ext = (ctypes.c_int64 * rank)(*[int(e) for e in extents])
    snp = (ctypes.c_int32 * rank)(*[len(s) - 1 for s in src_splits])
    dnp = (ctypes.c_int32 * rank)(*[len(s) - 1 for s in dst_splits])
    keep_s, sp = _splits_arrays(src_splits)
    keep_d, dp = _splits_arrays(dst_splits)
    _check(LIB.ja_repartition_noalloc(rank, ext, snp, sp, dnp, dp, dtype, ctypes.c_void_p(src_ptr), ctypes.c_void_p(dst_ptr),
                                      ctypes.c_void_p(stream)))


def ja_overlay_atoms(src: int, dst: int):
    n = ctypes.c_int64()
    _check(LIB.ja_overlay_atoms(src, dst, ctypes.byref(n), None, None, None, None))
    nb, rank = ctypes.c_int64(), ctypes.c_int32()
    _check(LIB.ja_relation_num_blocks(src, ctypes.byref(nb), ctypes.byref(rank)))
    lower = np.zeros((n.value, rank.value), dtype=np.int64)
    upper = np.zeros((n.value, rank.value), dtype=np.int64)
    sb = np.zeros(n.value, dtype=np.int32)
    db = np.zeros(n.value, dtype=np.int32)
    _check(LIB.ja_overlay_atoms(src, dst, ctypes.byref(n), lower.ctypes.data, upper.ctypes.data, sb.ctypes.data, db.ctypes.data))
    return lower, upper, sb, db


def ja_stream_status(stream: int = 0) -> int:
    st = ctypes.c_int()
    _check(LIB.ja_stream_status(ctypes.c_void_p(stream), ctypes.byref(st)))
    return st.value


def ja_debug_set(name: str, value: int):
    """Force a kernel form / schedule, or set the limit of the device-side waits ("wait_cap_ns"); -1 = not forced."""
    _check(LIB.ja_debug_set(name.encode(), int(value)))


def ja_debug_wait_timeout(stream: int = 0, waiters_ok_ptr: int = 0):
    """Test hook: a one-CTA kernel whose bounded wait runs out (JA_ERR_TIMEOUT lands in the stream's status word)."""
    _check(LIB.ja_debug_wait_timeout(ctypes.c_void_p(stream), ctypes.c_void_p(waiters_ok_ptr)))


def ja_debug_bounded_wait_host(ready_at_poll: int, ns_per_poll: int, cap_ns: int, abort_at_poll: int = 0):
    """The kernels' wait loop on the host against a scripted barrier and clock: (polls, succeeded, recorded_timeout, ns)."""
    polls, ok, rec, ns = ctypes.c_int64(), ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int64()
    _check(LIB.ja_debug_bounded_wait_host(ready_at_poll, ns_per_poll, cap_ns, abort_at_poll, ctypes.byref(polls), ctypes.byref(ok),
                                          ctypes.byref(rec), ctypes.byref(ns)))
    return polls.value, bool(ok.value), bool(rec.value), ns.value
