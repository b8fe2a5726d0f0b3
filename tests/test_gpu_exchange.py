"""An exchange program executed on one GPU (ja_exchange_execute) against the oracle's executor (oracle/exprog.py) on the
same seeded partial relations: decompose, the program's aggregations and transfers, recompose.  MAX and programs whose
aggregations have two parts of f32 cells are bit-exact; sums are compared with the same firing order restated in f32
(bit-exact) and with the oracle (tolerance)."""
import json
import os

import numpy as np
import pytest
import torch

from oracle import blocked, core
from oracle import exprog as E
from paper_2609_03905_b200 import exprog as X
from paper_2609_03905_b200.binding import JaError
import synth_inputs as si
from gpu_util import TOL, check_status, download, download_bits, empty_like_tiling, relfro, upload

pytestmark = pytest.mark.gpu
BF, F16, F32 = torch.bfloat16, torch.float16, torch.float32
ORC_DT = {BF: "bf16", F16: "f16", F32: "f32"}
ES = blocked.equal_splits
G = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "exprog_examples.json")))

CASES = {
    # the preamble example of Section 5.3: 2 copies, four GPUs
    "preamble": dict(ext=[256, 256], ps=[[0, 128, 256], [0, 256]], cs=[[0, 64, 128, 192, 256], [0, 256]], m=2,
                     copy_site=[0, 1, 2, 3], specs=[0, 1, 2, 3]),
    # an all-to-all: every GPU holds a copy of every producer block's share, consumer cut the other way
    "crossed": dict(ext=[192, 160], ps=[ES(192, 2), ES(160, 1)], cs=[ES(192, 1), ES(160, 4)], m=4,
                    copy_site=[0, 1, 2, 3, 3, 2, 1, 0], specs=[0, 1, 2, 3]),
    # replication: two function specs consume the same block; odd sizes (scalar accesses); rank 3
    "replicated": dict(ext=[6, 33, 10], ps=[ES(6, 2), [0, 10, 33], [0, 10]], cs=[ES(6, 1), [0, 33], [0, 3, 10]], m=3,
                       copy_site=[0, 1, 2, 2, 0, 1, 1, 2, 0, 0, 2, 1], specs=[0, 1, 1]),
    # an all-reduce shape: every GPU holds one copy of the one block and every GPU consumes it
    "allreduce": dict(ext=[128, 64], ps=[[0, 128], [0, 64]], cs=[[0, 128], [0, 64]], m=4, copy_site=[0, 1, 2, 3],
                      specs=[0, 0, 0, 0]),
}


def build(case, body, machine="hgx_b200"):
    c = CASES[case]
    pre_o = E.preamble(c["ext"], c["ps"], {(b, k): c["copy_site"][b * c["m"] + k] for b in range(len(c["copy_site"]) // c["m"]) for k in range(c["m"])},
                       c["cs"], c["specs"], 2)
    h = X.ExchangeProgram(handle=X.ja_exprog_preamble(c["ps"], c["cs"], c["m"], c["copy_site"], c["specs"], 2))
    m = X.ja_machine_preset(machine)
    if body == "synth":
        X.ja_exprog_place(h.handle, m, "best")
        X.ja_exprog_synthesize(h.handle, m, 2, 6)
    else:
        X.ja_exprog_place(h.handle, m, body)
    return h, E.parse(str(h))        # the oracle executes the library's program, read from its text


@pytest.mark.parametrize("dtype", [BF, F16, F32])
@pytest.mark.parametrize("agg", ["sum", "max"])
@pytest.mark.parametrize("body", ["naive", "butterfly", "synth"])
@pytest.mark.parametrize("case", list(CASES))
def test_exchange_program_on_one_gpu(case, body, agg, dtype):
    c = CASES[case]
    m = c["m"]
    es = 4 if dtype == F32 else 2
    # the preamble's sizes depend on the cell width: rebuild for this dtype
    h = X.ExchangeProgram(handle=X.ja_exprog_preamble(c["ps"], c["cs"], m, c["copy_site"], c["specs"], es))
    mach = X.ja_machine_preset("hgx_b200")
    X.ja_exprog_place(h.handle, mach, "best" if body == "synth" else body)
    if body == "synth":
        X.ja_exprog_synthesize(h.handle, mach, 2, 6)
    assert X.ja_exprog_check(h.handle) == (True, True)
    q = E.parse(str(h))
    assert E.valid_bound(q)
    P = si.normal([m] + c["ext"], 0.0, 1.0, dtype, 5, 17)
    rP = upload(P, blocked.partial_splits(m, c["ps"]))
    rD = empty_like_tiling(c["ext"], c["cs"], dtype, fill=float("nan"))
    before = download_bits(rP).copy()
    stats = h.execute(rP, c["copy_site"], c["specs"], agg, rD)
    got = download(rD)
    check_status()
    assert np.array_equal(download_bits(rP), before)                      # partials are borrowed, unchanged
    P64 = si.to_f64(P)
    sched = E.schedule(q)
    assert stats["aggregations"] == sum(len(cover) >= 2 for _, _, _, cover in sched)
    held, fresh = set(), 0
    for x, s, d, _ in sched:                                               # a delivery to a site that already holds the aggregate moves nothing
        held.add((x, s))
        for t in d:
            fresh += (x, t) not in held
            held.add((x, t))
    assert stats["transfers"] == fresh
    want = E.exchange(q, P64, c["ps"], c["cs"], c["specs"], agg, ORC_DT[dtype])
    consumed = ~np.isnan(want)
    assert consumed.all()                                                  # every block of these cases is consumed
    if agg == "max":
        assert np.array_equal(got, want)                                   # bit-exact
        assert np.array_equal(got, blocked.aggregate_repartition(P64, c["ps"], c["cs"], "max", ORC_DT[dtype]))
        return

    def f32_sum(parts):                                                    # the kernel's arithmetic: f32, the order given, one rounding
        acc = np.asarray(parts[0], dtype=np.float64).astype(np.float32)
        for p in parts[1:]:
            acc = acc + np.asarray(p, dtype=np.float64).astype(np.float32)
        return core.round_to(acc.astype(np.float64), ORC_DT[dtype])

    same_order = E.exchange(q, P64, c["ps"], c["cs"], c["specs"], "sum", ORC_DT[dtype], combine=f32_sum)
    assert np.array_equal(got, same_order)
    assert relfro(got, want) <= (1e-6 if dtype == F32 else 1e-3)
    # whatever the program, the result is the aggregate of all m copies (intermediate aggregates are rounded to the cell type)
    assert relfro(got, blocked.aggregate_repartition(P64, c["ps"], c["cs"], "sum", ORC_DT[dtype])) <= TOL[dtype]


def test_the_doubling_body_is_what_runs_for_the_allreduce_shape():
    h, q = build("allreduce", "best", "dgx_h100")
    acts = X.ja_exprog_get_actions(h.handle)
    assert sum(1 for a, s, d in acts if d) == 8 and max(bin(a).count("1") for a, s, d in acts if d) == 2   # two rounds of four sends
    hn, _ = build("allreduce", "naive", "dgx_h100")
    assert X.ja_exprog_simulate(h.handle, X.ja_machine_preset("dgx_h100")) < X.ja_exprog_simulate(hn.handle, X.ja_machine_preset("dgx_h100"))


def test_exchange_refusals():
    c = CASES["preamble"]
    h, q = build("preamble", "naive")
    P = si.normal([2] + c["ext"], 0.0, 1.0, BF, 1, 2)
    rP = upload(P, blocked.partial_splits(2, c["ps"]))
    rD = empty_like_tiling(c["ext"], c["cs"], BF)
    with pytest.raises(JaError) as e:                      # other copy sites than the program's preamble
        h.execute(rP, [1, 0, 2, 3], c["specs"], "sum", rD)
    assert e.value.status_name == "JA_ERR_INVALID_ARG"
    with pytest.raises(JaError) as e:                      # another consumer tiling
        h.execute(rP, c["copy_site"], c["specs"], "sum", empty_like_tiling(c["ext"], [ES(256, 2), [0, 256]], BF))
    assert e.value.status_name == "JA_ERR_INVALID_ARG"
    with pytest.raises(JaError) as e:
        h.execute(rP, c["copy_site"], c["specs"], "sum", empty_like_tiling(c["ext"], c["cs"], F32))
    assert e.value.status_name == "JA_ERR_DTYPE"
    with pytest.raises(JaError) as e:                      # two copies need an aggregation
        h.execute(rP, c["copy_site"], c["specs"], "none", rD)
    assert e.value.status_name == "JA_ERR_INVALID_ARG"
    # a body that does not satisfy OUT
    bad = X.ExchangeProgram(str(h).split("\n\n")[0] + "\n\n")
    with pytest.raises(JaError) as e:
        bad.execute(rP, c["copy_site"], c["specs"], "sum", rD)
    assert e.value.status_name == "JA_ERR_INVALID_ARG"
    unbound = X.ExchangeProgram(handle=X.ja_exprog_preamble(c["ps"], c["cs"], 2, c["copy_site"], c["specs"], 2))
    with pytest.raises(JaError):
        unbound.execute(rP, c["copy_site"], c["specs"], "sum", rD)
    check_status()


@pytest.mark.parametrize("dtype", [BF, F16, F32])
@pytest.mark.parametrize("agg", ["sum", "max"])
@pytest.mark.parametrize("n_parts", [2, 5, 16])
def test_the_local_aggregation_primitive(n_parts, agg, dtype):
    from paper_2609_03905_b200 import exchange_dist
    n = 4096 + 8 * 37                                                   # whole 16-byte accesses, several blocks and a ragged last one
    parts = [si.normal([n], 0.0, 1.0, dtype, 9, k).cuda() for k in range(n_parts)]
    out = exchange_dist.library_combine(parts, agg)
    torch.cuda.synchronize()
    check_status()
    P64 = [si.to_f64(p.cpu()) for p in parts]
    if agg == "max":
        assert np.array_equal(si.to_f64(out.cpu()), np.max(np.stack(P64), axis=0))
    else:
        acc = P64[0].astype(np.float32)
        for p in P64[1:]:
            acc = acc + p.astype(np.float32)
        assert np.array_equal(si.to_f64(out.cpu()), core.round_to(acc.astype(np.float64), ORC_DT[dtype]))
        assert relfro(si.to_f64(out.cpu()), core.round_to(np.sum(np.stack(P64), axis=0), ORC_DT[dtype])) <= (1e-6 if dtype == F32 else 1e-3)
    with pytest.raises(JaError) as e:
        X.ja_exchange_combine([parts[0].data_ptr(), parts[1].data_ptr() + 2], out.data_ptr(), 64, 1, "sum")
    assert e.value.status_name == "JA_ERR_ALIGNMENT"
    with pytest.raises(JaError) as e:
        X.ja_exchange_combine([parts[0].data_ptr(), parts[1].data_ptr()], out.data_ptr(), 40, 1, "sum")
    assert e.value.status_name == "JA_ERR_ALIGNMENT"


def test_exchange_refuses_a_stream_that_is_being_captured():
    c = CASES["preamble"]
    h, q = build("preamble", "naive")
    rP = upload(si.normal([2] + c["ext"], 0.0, 1.0, BF, 1, 3), blocked.partial_splits(2, c["ps"]))
    rD = empty_like_tiling(c["ext"], c["cs"], BF)
    h.execute(rP, c["copy_site"], c["specs"], "sum", rD)                      # outside any capture: fine
    torch.cuda.synchronize()
    want = download_bits(rD).copy()
    g = torch.cuda.CUDAGraph()
    marker = torch.zeros(1, device="cuda")
    with torch.cuda.graph(g):
        marker.add_(1.0)                                                        # so that the capture is not empty
        with pytest.raises(JaError, match="captured") as e:
            h.execute(rP, c["copy_site"], c["specs"], "sum", rD)
        assert e.value.status_name == "JA_ERR_UNSUPPORTED"
    g.replay()
    torch.cuda.synchronize()
    assert marker.item() == 1.0 and np.array_equal(download_bits(rD), want)    # the refused call recorded nothing
    X.ja_exchange_trim()
    check_status()


@pytest.mark.parametrize("case,body", [("preamble", "naive"), ("crossed", "synth"), ("replicated", "naive"), ("allreduce", "butterfly")])
def test_exchange_plan_runs_as_dataflow_and_inside_a_graph(case, body):
    c = CASES[case]
    m = c["m"]
    h, q = build(case, body)
    P = si.normal([m] + c["ext"], 0.0, 1.0, BF, 6, 19)
    rP = upload(P, blocked.partial_splits(m, c["ps"]))
    rA = empty_like_tiling(c["ext"], c["cs"], BF, fill=float("nan"))
    rB = empty_like_tiling(c["ext"], c["cs"], BF, fill=float("nan"))
    stats = h.execute(rP, c["copy_site"], c["specs"], "sum", rA)
    plan = X.ExchangePlan(h, rP, c["copy_site"], c["specs"], "sum", rB)
    assert plan.stats == stats
    plan.run()
    torch.cuda.synchronize()
    check_status()
    assert np.array_equal(download_bits(rB), download_bits(rA))            # the same program, the same bits
    # captured: the graph holds the program's steps; new contents of the partial relation, no host work at replay
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        plan.run()
    P2 = si.normal([m] + c["ext"], 0.0, 1.0, BF, 6, 23)
    packed = download_packed(P2, blocked.partial_splits(m, c["ps"]))
    rP.payload[: packed.numel()].copy_(packed)
    rB.payload.zero_()
    for _ in range(2):
        g.replay()
    torch.cuda.synchronize()
    check_status()
    h.execute(rP, c["copy_site"], c["specs"], "sum", rA)
    torch.cuda.synchronize()
    assert np.array_equal(download(rB), download(rA))                      # cell for cell (the payloads' padding was cleared in one only)
    want = E.exchange(q, si.to_f64(P2), c["ps"], c["cs"], c["specs"], "sum", "bf16")
    assert relfro(download(rB), want) <= 1e-3
    # and eagerly again after the capture, on another stream
    rB.payload.zero_()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        plan.run()
    side.synchronize()
    check_status()
    assert np.array_equal(download(rB), download(rA))
    plan.close()


def download_packed(dense, splits):
    """The oracle's packing of a dense tensor into a payload, as a CUDA tensor of the relation's cell type."""
    from gpu_util import from_bits, np_bits
    packed = blocked.pack(np_bits(dense), splits)
    return from_bits(packed, dense.dtype).cuda()


@pytest.mark.parametrize("seed", range(10))
def test_randomly_rewritten_programs_on_random_preambles(seed):
    """Random tilings, copy sites and function specs; the body is the trivial program after a random walk through the
    rewriting rules (relays, fissions, eager and lazy aggregation, redirected sources), so the aggregation trees, the
    duplicates and the order of arrival differ from anything a constructor emits."""
    import random
    rng = random.Random(100 + seed)
    rank = rng.choice([1, 2, 2, 3])
    ext = [rng.choice([24, 40, 64, 96]) for _ in range(rank)]

    def cut(e, n):
        pts = sorted(rng.sample(range(1, e), n - 1)) if n > 1 else []
        return [0] + pts + [e]

    n_sites = rng.choice([2, 3, 4])
    while True:
        ps = [cut(e, rng.choice([1, 2])) for e in ext]
        cs = [cut(e, rng.choice([1, 2, 3])) for e in ext]
        n_pb = int(np.prod([len(s) - 1 for s in ps]))
        n_cb = int(np.prod([len(s) - 1 for s in cs]))
        m = rng.choice([1, 2, 3])
        cells = int(np.prod([len(set(a) | set(b)) - 1 for a, b in zip(ps, cs)]))
        if cells * m <= 24:
            break
    copy_site = [rng.randrange(n_sites) for _ in range(n_pb * m)]
    specs = [rng.randrange(n_cb) for _ in range(n_sites)]
    dtype = rng.choice([BF, F16, F32])
    agg = rng.choice(["sum", "max"]) if m > 1 else "none"
    es = 4 if dtype == F32 else 2
    h0 = X.ExchangeProgram(handle=X.ja_exprog_preamble(ps, cs, m, copy_site, specs, es))
    X.ja_exprog_bind(h0.handle, rng.randrange(X.ja_exprog_num_memberships(h0.handle)))
    X.ja_exprog_body(h0.handle, "naive")
    q = E.normalised(E.parse(str(h0)))
    for _ in range(rng.randint(0, 8)):
        nb = E.neighbours(q)
        if nb:
            q = rng.choice(nb)
    assert E.valid_bound(q)
    h = X.ExchangeProgram(E.format_program(q))
    assert X.ja_exprog_check(h.handle) == (True, True)
    P = si.normal([m] + ext, 0.0, 1.0, dtype, 7, seed)
    rP = upload(P, blocked.partial_splits(m, ps))
    rD = empty_like_tiling(ext, cs, dtype, fill=float("nan"))
    h.execute(rP, copy_site, specs, agg, rD)
    plan = X.ExchangePlan(h, rP, copy_site, specs, agg, empty_like_tiling(ext, cs, dtype, fill=float("nan")))
    plan.run()
    got, got_plan = download(rD), download(plan.dst)
    check_status()
    P64 = si.to_f64(P)
    want = E.exchange(q, P64, ps, cs, specs, "sum" if agg == "none" else agg, ORC_DT[dtype])
    consumed = ~np.isnan(want)                                              # blocks no function spec consumes stay untouched
    assert consumed.any() and np.isnan(got[~consumed]).all()
    assert np.array_equal(got_plan[consumed], got[consumed]) and np.isnan(got_plan[~consumed]).all()
    if agg != "sum":
        assert np.array_equal(got[consumed], want[consumed])
    else:
        def f32_sum(parts):
            acc = np.asarray(parts[0], dtype=np.float64).astype(np.float32)
            for p in parts[1:]:
                acc = acc + np.asarray(p, dtype=np.float64).astype(np.float32)
            return core.round_to(acc.astype(np.float64), ORC_DT[dtype])
        same = E.exchange(q, P64, ps, cs, specs, "sum", ORC_DT[dtype], combine=f32_sum)
        assert np.array_equal(got[consumed], same[consumed])
        assert relfro(got[consumed], want[consumed]) <= (1e-6 if dtype == F32 else 2e-3)
    plan.close()


@pytest.mark.parametrize("case,body", [("preamble", "naive"), ("crossed", "synth"), ("replicated", "naive"), ("allreduce", "butterfly")])
def test_exchange_plan_with_sites_on_device_labels(case, body):
    """Every site on a device label of its own.  With fewer devices than labels the labels wrap around, so on one GPU this
    runs every path a plan over several devices takes -- per-device pools, staging at home, copies for the atoms that leave
    home, for every transfer and for the aggregates that come home -- and must give the one-stream execution's bits."""
    c = CASES[case]
    m = c["m"]
    h, q = build(case, body)
    P = si.normal([m] + c["ext"], 0.0, 1.0, BF, 6, 29)
    rP = upload(P, blocked.partial_splits(m, c["ps"]))
    rA = empty_like_tiling(c["ext"], c["cs"], BF, fill=float("nan"))
    rB = empty_like_tiling(c["ext"], c["cs"], BF, fill=float("nan"))
    stats = h.execute(rP, c["copy_site"], c["specs"], "sum", rA)
    n_sites = X.ja_exprog_counts(h)["gpus"]
    for labels in ([s + 1 for s in range(n_sites)],            # nobody at home: everything is staged
                   [0] + [5] * (n_sites - 1),                  # site 0 at home, the others together elsewhere
                   [torch.cuda.current_device()] * n_sites):   # everybody at home: the plan of the test above
        plan = X.ExchangePlan(h, rP, c["copy_site"], c["specs"], "sum", rB, site_device=labels)
        assert {k: v for k, v in plan.stats.items() if k != "scratch_bytes"} == {k: v for k, v in stats.items() if k != "scratch_bytes"}
        rB.payload.zero_()
        plan.run()
        torch.cuda.synchronize()
        check_status()
        assert np.array_equal(download(rB), download(rA))
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            plan.run()
        rB.payload.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert np.array_equal(download(rB), download(rA))
        plan.close()
    with pytest.raises(JaError):
        X.ExchangePlan(h, rP, c["copy_site"], c["specs"], "sum", rB, site_device=[-1] * n_sites)
