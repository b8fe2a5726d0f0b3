"""ctypes binding of the exchange-program part of libja's C ABI (include/ja_exprog.h): the same names, argument
marshalling only.  `ExchangeProgram` owns a handle.  Aggregates are masks over the atoms in declaration order, sets of
sites masks over site numbers, as in the header."""
from __future__ import annotations

import ctypes

from .binding import LIB, _check

JA_FABRIC_NVSWITCH, JA_FABRIC_CUBE_MESH, JA_FABRIC_LINKS = 0, 1, 2
BODY = {"own": 0, "naive": 1, "butterfly": 2, "best": 3}
RULE = {"insert": 0, "delete": 1, "fission": 2, "fusion": 3, "relay_in": 4, "relay_out": 5, "pushdown": 6, "pullup": 7,
        "source": 8}


class ja_machine_t(ctypes.Structure):
    _fields_ = [("fabric", ctypes.c_int32), ("n_sites", ctypes.c_int32), ("hbm_gbs", ctypes.c_double),
                ("link_gbs", ctypes.c_double), ("double_gbs", ctypes.c_double), ("pcie_gbs", ctypes.c_double),
                ("links", ctypes.POINTER(ctypes.c_double))]


def machine_from_links(links, hbm_gbs: float, bridge_gbs: float = 0.0) -> ja_machine_t:
    """A point-to-point topology from a square table links[a][b] = GB/s of the direct link a -> b (0 = none: over the bridge)."""
    n = len(links)
    flat = (ctypes.c_double * (n * n))(*[float(links[a][b]) for a in range(n) for b in range(n)])
    m = ja_machine_t(JA_FABRIC_LINKS, n, hbm_gbs, 1.0, 0.0, bridge_gbs, ctypes.cast(flat, ctypes.POINTER(ctypes.c_double)))
    m._keep = flat           # the table must outlive the machine
    return m


def _declare():
    vp, i32, i64, u64, dbl = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64, ctypes.c_double
    P = ctypes.POINTER
    sigs = {
        "ja_machine_preset": [ctypes.c_char_p, P(ja_machine_t)],
        "ja_exprog_parse": [ctypes.c_char_p, P(vp)],
        "ja_exprog_clone": [vp, P(vp)],
        "ja_exprog_merge": [vp, vp, ctypes.c_char_p, ctypes.c_char_p, P(vp)],
        "ja_exprog_format": [vp, ctypes.c_char_p, i64, P(i64)],
        "ja_exprog_counts": [vp, P(i32), P(i32), P(i32), P(i32), P(i32), P(i32)],
        "ja_exprog_get_actions": [vp, P(u64), P(i32), P(u64)],
        "ja_exprog_get_requirements": [vp, P(i32), P(u64), P(i32)],
        "ja_exprog_get_atoms": [vp, P(i32), P(dbl)],
        "ja_exprog_num_memberships": [vp, P(i64)],
        "ja_exprog_bind": [vp, i64],
        "ja_exprog_membership": [vp, ctypes.c_char_p, P(u64)],
        "ja_exprog_bind_members": [vp, ctypes.c_char_p, P(i32), i32],
        "ja_exprog_closure": [vp, P(i64), P(u64), P(i32)],
        "ja_exprog_check": [vp, P(i32), P(i32)],
        "ja_exprog_valid_any": [vp, P(i32)],
        "ja_exprog_simulate": [vp, P(ja_machine_t), P(dbl), P(dbl), P(dbl), P(dbl)],
        "ja_exprog_body": [vp, i32],
        "ja_exprog_normalise": [vp],
        "ja_exprog_rewrite": [vp, i32, i32, i32, u64, u64, P(i32)],
        "ja_exprog_synthesize": [vp, P(ja_machine_t), i32, i32, P(dbl)],
        "ja_exprog_place": [vp, P(ja_machine_t), i32, P(dbl)],
        "ja_exprog_preamble": [i32, P(i64), P(i32), P(i64), P(i32), i32, P(i32), P(i32), i32, i32, P(vp)],
        "ja_exchange_execute": [vp, vp, P(i32), P(i32), i32, ctypes.c_int, vp, P(i64), vp],
        "ja_exprog_schedule": [vp, P(i32), P(i32), P(i32), P(i32), P(u64)],
        "ja_exchange_plan_create": [vp, vp, P(i32), P(i32), i32, ctypes.c_int, vp, P(i64), P(vp)],
        "ja_exchange_plan_run": [vp, vp],
        "ja_exchange_plan_create_on": [vp, vp, P(i32), P(i32), i32, ctypes.c_int, vp, P(i32), i32, P(i64), P(vp)],
        "ja_exchange_combine": [P(vp), i32, vp, i64, ctypes.c_int, ctypes.c_int, vp],
    }
    for name, argtypes in sigs.items():
        fn = getattr(LIB, name)
        fn.argtypes = argtypes
        fn.restype = ctypes.c_int
    LIB.ja_exchange_plan_destroy.argtypes = [vp]
    LIB.ja_exchange_plan_destroy.restype = None
    LIB.ja_exchange_trim.argtypes = []
    LIB.ja_exchange_trim.restype = ctypes.c_int
    LIB.ja_exprog_destroy.argtypes = [vp]
    LIB.ja_exprog_destroy.restype = None


_declare()


def _program_arg(fn):
    """Lets a call take an ExchangeProgram object where it takes a handle; the object stays referenced for the call's duration
    (a handle taken from a temporary object would die before the call runs)."""
    import functools

    @functools.wraps(fn)
    def inner(prog, *args, **kw):
        return fn(getattr(prog, "handle", prog), *args, **kw)
    return inner


def ja_machine_preset(name: str) -> ja_machine_t:
    m = ja_machine_t()
    _check(LIB.ja_machine_preset(name.encode(), ctypes.byref(m)))
    return m


def ja_exprog_parse(text: str) -> int:
    h = ctypes.c_void_p()
    _check(LIB.ja_exprog_parse(text.encode(), ctypes.byref(h)))
    return h.value


@_program_arg
def ja_exprog_clone(prog: int) -> int:
    h = ctypes.c_void_p()
    _check(LIB.ja_exprog_clone(prog, ctypes.byref(h)))
    return h.value


def ja_exprog_merge(a, b, prefix_a: str, prefix_b: str) -> int:
    h = ctypes.c_void_p()
    _check(LIB.ja_exprog_merge(getattr(a, "handle", a), getattr(b, "handle", b), prefix_a.encode(), prefix_b.encode(), ctypes.byref(h)))
    return h.value


def ja_exprog_destroy(prog: int):
    LIB.ja_exprog_destroy(prog)


@_program_arg
def ja_exprog_format(prog: int) -> str:
    need = ctypes.c_int64()
    _check(LIB.ja_exprog_format(prog, None, 0, ctypes.byref(need)))
    buf = ctypes.create_string_buffer(need.value)
    _check(LIB.ja_exprog_format(prog, buf, need.value, ctypes.byref(need)))
    return buf.value.decode()


@_program_arg
def ja_exprog_counts(prog: int) -> dict:
    v = [ctypes.c_int32() for _ in range(6)]
    _check(LIB.ja_exprog_counts(prog, *[ctypes.byref(x) for x in v]))
    return dict(zip(("gpus", "partitions", "atoms", "out", "actions", "expanded"), (x.value for x in v)))


@_program_arg
def ja_exprog_get_actions(prog: int):
    """[(aggregate mask, source site, destination mask)] of the expanded actions."""
    n = ja_exprog_counts(prog)["expanded"]
    agg, src, dst = (ctypes.c_uint64 * max(n, 1))(), (ctypes.c_int32 * max(n, 1))(), (ctypes.c_uint64 * max(n, 1))()
    _check(LIB.ja_exprog_get_actions(prog, agg, src, dst))
    return [(agg[i], src[i], dst[i]) for i in range(max(n, 0))]


@_program_arg
def ja_exprog_get_requirements(prog: int):
    n = ctypes.c_int32()
    _check(LIB.ja_exprog_get_requirements(prog, ctypes.byref(n), None, None))
    agg, site = (ctypes.c_uint64 * max(n.value, 1))(), (ctypes.c_int32 * max(n.value, 1))()
    _check(LIB.ja_exprog_get_requirements(prog, ctypes.byref(n), agg, site))
    return [(agg[i], site[i]) for i in range(n.value)]


@_program_arg
def ja_exprog_get_atoms(prog: int):
    n = ja_exprog_counts(prog)["atoms"]
    site, gb = (ctypes.c_int32 * max(n, 1))(), (ctypes.c_double * max(n, 1))()
    _check(LIB.ja_exprog_get_atoms(prog, site, gb))
    return [(site[i], gb[i]) for i in range(n)]


@_program_arg
def ja_exprog_num_memberships(prog: int) -> int:
    n = ctypes.c_int64()
    _check(LIB.ja_exprog_num_memberships(prog, ctypes.byref(n)))
    return n.value


@_program_arg
def ja_exprog_bind(prog: int, index: int):
    _check(LIB.ja_exprog_bind(prog, index))


@_program_arg
def ja_exprog_membership(prog: int, partition: str) -> int:
    m = ctypes.c_uint64()
    _check(LIB.ja_exprog_membership(prog, partition.encode(), ctypes.byref(m)))
    return m.value


@_program_arg
def ja_exprog_bind_members(prog: int, partition: str, sites):
    _check(LIB.ja_exprog_bind_members(prog, partition.encode(), (ctypes.c_int32 * len(sites))(*[int(x) for x in sites]), len(sites)))


@_program_arg
def ja_exprog_closure(prog: int):
    n = ctypes.c_int64()
    _check(LIB.ja_exprog_closure(prog, ctypes.byref(n), None, None))
    agg, site = (ctypes.c_uint64 * max(n.value, 1))(), (ctypes.c_int32 * max(n.value, 1))()
    _check(LIB.ja_exprog_closure(prog, ctypes.byref(n), agg, site))
    return [(agg[i], site[i]) for i in range(n.value)]


@_program_arg
def ja_exprog_check(prog: int):
    wf, v = ctypes.c_int32(), ctypes.c_int32()
    _check(LIB.ja_exprog_check(prog, ctypes.byref(wf), ctypes.byref(v)))
    return bool(wf.value), bool(v.value)


@_program_arg
def ja_exprog_valid_any(prog: int) -> bool:
    v = ctypes.c_int32()
    _check(LIB.ja_exprog_valid_any(prog, ctypes.byref(v)))
    return bool(v.value)


@_program_arg
def ja_exprog_simulate(prog: int, machine: ja_machine_t, trace: bool = False):
    ms = ctypes.c_double()
    if not trace:
        _check(LIB.ja_exprog_simulate(prog, ctypes.byref(machine), ctypes.byref(ms), None, None, None))
        return ms.value
    n = max(ja_exprog_counts(prog)["expanded"], 1)
    a, b, c = (ctypes.c_double * n)(), (ctypes.c_double * n)(), (ctypes.c_double * n)()
    _check(LIB.ja_exprog_simulate(prog, ctypes.byref(machine), ctypes.byref(ms), a, b, c))
    return ms.value, [(a[i], b[i], c[i]) for i in range(n)]


@_program_arg
def ja_exprog_body(prog: int, body: str):
    _check(LIB.ja_exprog_body(prog, BODY[body]))


@_program_arg
def ja_exprog_normalise(prog: int):
    _check(LIB.ja_exprog_normalise(prog))


@_program_arg
def ja_exprog_rewrite(prog: int, rule: str, i: int = 0, j: int = 0, a: int = 0, b: int = 0) -> bool:
    applied = ctypes.c_int32()
    _check(LIB.ja_exprog_rewrite(prog, RULE[rule], i, j, a, b, ctypes.byref(applied)))
    return bool(applied.value)


@_program_arg
def ja_exprog_synthesize(prog: int, machine: ja_machine_t, depth: int = 4, beam: int = 16) -> float:
    ms = ctypes.c_double()
    _check(LIB.ja_exprog_synthesize(prog, ctypes.byref(machine), depth, beam, ctypes.byref(ms)))
    return ms.value


@_program_arg
def ja_exprog_place(prog: int, machine: ja_machine_t, body: str = "best") -> float:
    ms = ctypes.c_double()
    _check(LIB.ja_exprog_place(prog, ctypes.byref(machine), BODY[body], ctypes.byref(ms)))
    return ms.value


def ja_exprog_preamble(producer_splits, consumer_splits, m: int, copy_site, consumer_specs, width_bytes: int) -> int:
    rank = len(producer_splits)
    flat_p = [int(x) for s in producer_splits for x in s]
    flat_c = [int(x) for s in consumer_splits for x in s]
    h = ctypes.c_void_p()
    _check(LIB.ja_exprog_preamble(
        rank, (ctypes.c_int64 * len(flat_p))(*flat_p), (ctypes.c_int32 * rank)(*[len(s) for s in producer_splits]),
        (ctypes.c_int64 * len(flat_c))(*flat_c), (ctypes.c_int32 * rank)(*[len(s) for s in consumer_splits]), m,
        (ctypes.c_int32 * len(copy_site))(*[int(x) for x in copy_site]),
        (ctypes.c_int32 * len(consumer_specs))(*[int(x) for x in consumer_specs]), len(consumer_specs), width_bytes,
        ctypes.byref(h)))
    return h.value


@_program_arg
def ja_exchange_execute(prog: int, partials: int, copy_site, consumer_specs, agg, dst: int, stream: int = 0) -> dict:
    """Relation handles as in binding.ja_repartition_agg; returns the call's statistics."""
    from .binding import AGG
    stats = (ctypes.c_int64 * 5)()
    _check(LIB.ja_exchange_execute(prog, partials, (ctypes.c_int32 * len(copy_site))(*[int(x) for x in copy_site]),
                                   (ctypes.c_int32 * len(consumer_specs))(*[int(x) for x in consumer_specs]), len(consumer_specs),
                                   AGG[agg] if isinstance(agg, str) else int(agg), dst, stats, stream))
    return {"aggregations": stats[0], "transfers": stats[1], "transfer_bytes": stats[2], "scratch_bytes": stats[3],
            "aggregation_bytes": stats[4]}


@_program_arg
def ja_exprog_schedule(prog: int):
    """[(expanded action index, [part masks in combination order])] in firing order."""
    n, total = ctypes.c_int32(), ctypes.c_int32()
    _check(LIB.ja_exprog_schedule(prog, ctypes.byref(n), ctypes.byref(total), None, None, None))
    act, begin, parts = (ctypes.c_int32 * max(n.value, 1))(), (ctypes.c_int32 * (n.value + 1))(), (ctypes.c_uint64 * max(total.value, 1))()
    _check(LIB.ja_exprog_schedule(prog, ctypes.byref(n), ctypes.byref(total), act, begin, parts))
    return [(act[k], [parts[i] for i in range(begin[k], begin[k + 1])]) for k in range(n.value)]


def ja_exchange_combine(part_ptrs, out_ptr: int, nbytes: int, dtype: int, agg, stream: int = 0):
    from .binding import AGG
    arr = (ctypes.c_void_p * len(part_ptrs))(*[int(p) for p in part_ptrs])
    _check(LIB.ja_exchange_combine(arr, len(part_ptrs), out_ptr, nbytes, dtype, AGG[agg] if isinstance(agg, str) else int(agg), stream))


def _stats(stats):
    return {"aggregations": stats[0], "transfers": stats[1], "transfer_bytes": stats[2], "scratch_bytes": stats[3],
            "aggregation_bytes": stats[4]}


@_program_arg
def ja_exchange_plan_create(prog: int, partials: int, copy_site, consumer_specs, agg, dst: int, site_device=None):
    """Returns (plan handle, statistics).  site_device[s] = device label of site s (None: every site on the current device)."""
    from .binding import AGG
    stats = (ctypes.c_int64 * 5)()
    h = ctypes.c_void_p()
    sd = None if site_device is None else (ctypes.c_int32 * len(site_device))(*[int(x) for x in site_device])
    _check(LIB.ja_exchange_plan_create_on(prog, partials, (ctypes.c_int32 * len(copy_site))(*[int(x) for x in copy_site]),
                                          (ctypes.c_int32 * len(consumer_specs))(*[int(x) for x in consumer_specs]), len(consumer_specs),
                                          AGG[agg] if isinstance(agg, str) else int(agg), dst, sd,
                                          0 if site_device is None else len(site_device), stats, ctypes.byref(h)))
    return h.value, _stats(stats)


def ja_exchange_plan_run(plan: int, stream: int = 0):
    _check(LIB.ja_exchange_plan_run(plan, stream))


def ja_exchange_plan_destroy(plan: int):
    LIB.ja_exchange_plan_destroy(plan)


def ja_exchange_trim():
    _check(LIB.ja_exchange_trim())


class ExchangePlan:
    """An exchange plan with its lifetime; keeps the two relations alive, as the plan holds their payload addresses."""

    def __init__(self, prog: "ExchangeProgram", partials, copy_site, consumer_specs, agg, dst, site_device=None):
        self.partials, self.dst = partials, dst
        self.handle, self.stats = ja_exchange_plan_create(prog.handle, partials.handle, copy_site, consumer_specs, agg, dst.handle,
                                                          site_device)

    def run(self, stream=None):
        import torch
        ja_exchange_plan_run(self.handle, torch.cuda.current_stream().cuda_stream if stream is None else stream)

    def close(self, _destroy=LIB.ja_exchange_plan_destroy):   # bound at definition: module globals may be gone at interpreter exit
        if getattr(self, "handle", None):
            _destroy(self.handle)
            self.handle = None

    def __del__(self):
        self.close()


class ExchangeProgram:
    """A handle with its lifetime; methods are the calls above.  The handle is destroyed with the object: keep the object
    for as long as its `.handle` is in use (do not pass `ExchangeProgram(text).handle` of a temporary)."""

    def __init__(self, text: str | None = None, handle: int | None = None):
        self.handle = ja_exprog_parse(text) if handle is None else handle

    def __del__(self, _destroy=LIB.ja_exprog_destroy):       # bound at definition: module globals may be gone at interpreter exit
        if getattr(self, "handle", None):
            _destroy(self.handle)
            self.handle = None

    def clone(self):
        return ExchangeProgram(handle=ja_exprog_clone(self.handle))

    def merge(self, other: "ExchangeProgram", prefix_self: str, prefix_other: str):
        return ExchangeProgram(handle=ja_exprog_merge(self.handle, other.handle, prefix_self, prefix_other))

    def __str__(self):
        return ja_exprog_format(self.handle)

    def execute(self, partials, copy_site, consumer_specs, agg, dst, stream=None):
        """partials, dst: relations.Relation objects (payloads on the GPU); enqueues on torch's current stream by default."""
        import torch
        st = torch.cuda.current_stream().cuda_stream if stream is None else stream
        return ja_exchange_execute(self.handle, partials.handle, copy_site, consumer_specs, agg, dst.handle, st)


def best_valid_body(preamble: str, bodies, machine: ja_machine_t):
    """Candidate bodies for one (bound) preamble from any source -- the paper has a language model propose them -- filtered by
    Definition "Closure; validity" and ranked by the simulator.  Returns (index of the winner, its milliseconds, verdicts) where
    verdicts[i] is None for a candidate that does not parse, is not valid, or is not for this preamble's sites, else its time;
    (None, None, verdicts) if no candidate is valid."""
    from .binding import JaError
    verdicts, best = [], None
    head = preamble.strip("\n").split("\n\n")[0]
    for i, body in enumerate(bodies):
        try:
            h = ExchangeProgram(head + "\n\n" + body.strip("\n") + "\n")
            ok = ja_exprog_check(h.handle)[1]
            ms = ja_exprog_simulate(h.handle, machine) if ok else None
        except JaError:
            ms = None
        verdicts.append(ms)
        if ms is not None and (best is None or ms < verdicts[best]):
            best = i
    return best, (verdicts[best] if best is not None else None), verdicts
