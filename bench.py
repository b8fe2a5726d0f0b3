"""Benchmark of the join-agg hot path on B200: one step = one forward pass of a LLaMA-7B-shaped transformer
block (batch 8, seq 2048, hidden 4096, 32 heads x 128, FFN 11008, bf16, causal) executed as a chain of
join-aggs over tensor relations, with the ja_repartition relayouts of the chosen decomposition inside.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--plan mixed|seq|head] [--shape 7b|65b] [--impl reference]

Prints ONE JSON line. `value` is dense-contraction TFLOP/s of the whole job (inputs resident in HBM);
`e2e` is the same metric with host->device and device->host copies of the step's input and output inside
the timed region; `roofline` describes the dominant kernel (the tensor-core matmul join-agg), timed live
with CUDA events around each of its launches; `cpu_baseline` is the CPU oracle timed on a bounded sample.
With --gpus N > 1 (under torchrun) every rank runs an independent replica (the path does not shard).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

SHAPES = {"7b": dict(batch=8, seq=2048, hidden=4096, heads=32, ffn=11008),
          "65b": dict(batch=1, seq=4096, hidden=8192, heads=64, ffn=22016),
          # the paper's own block (Section 6): grouped-query attention, 32 query heads on 8 key/value heads, FFN 14336
          "paper_b8_1k": dict(batch=8, seq=1024, hidden=4096, heads=32, kv_heads=8, ffn=14336),
          "paper_1x8k": dict(batch=1, seq=8192, hidden=4096, heads=32, kv_heads=8, ffn=14336),
          "paper_b128_1k": dict(batch=128, seq=1024, hidden=4096, heads=32, kv_heads=8, ffn=14336),
          "paper_1x1k": dict(batch=1, seq=1024, hidden=4096, heads=32, kv_heads=8, ffn=14336),
          "paper_1x128k": dict(batch=1, seq=131072, hidden=4096, heads=32, kv_heads=8, ffn=14336)}
METRIC = "join-agg TFLOP/s, LLaMA-block forward on 1 B200"


def block_flops(batch, seq, hidden, ffn, heads=None, kv_heads=None):
    T = batch * seq
    kv_hidden = hidden if not kv_heads else hidden // heads * kv_heads
    return 2.0 * T * hidden * (2 * hidden + 2 * kv_hidden) + 2.0 * T * hidden * ffn * 3 + 4.0 * T * seq * hidden / 2


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "bf16": d["bf16_tflops"], "bf16_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


# ---- CPU oracle leg ------------------------------------------------------------------------------------------
def oracle_sample(shape, rows_n=16, prefix=None):
    """The oracle on a bounded sample of the workload: the first `prefix` tokens of sequence 0 of the batch (causal, so
    a prefix is a self-contained sub-problem), K and V for that whole prefix, block output for `rows_n` token rows spread
    over it. Returns (flops of the sample, seconds, threads)."""
    import numpy as np
    import synth_inputs as si
    from oracle import core, operators
    import torch
    S, hidden, heads, ffn = prefix or shape["seq"], shape["hidden"], shape["heads"], shape["ffn"]
    kvh = shape.get("kv_heads") or heads
    kv_hidden = hidden // heads * kvh
    w = {k: si.to_f64(v) for k, v in si.llama_weights(hidden, ffn, kv_hidden=kv_hidden).items()}
    x = si.to_f64(si.normal((S, hidden), 0.0, 1.0, torch.bfloat16, 5, 0))
    rows = np.linspace(0, S - 1, rows_n).astype(np.int64)
    t0 = time.perf_counter()
    operators.llama_block(x, w, heads, 1e4, 1e-5, rows=rows, n_kv_heads=kvh)
    dt = time.perf_counter() - t0
    fl = 2.0 * S * hidden * kv_hidden * 2 + 2.0 * rows_n * hidden * hidden * 2 + 2.0 * rows_n * hidden * ffn * 3 \
        + 4.0 * float(np.sum(rows + 1)) * hidden
    return fl, dt, core.num_threads()


def run_reference(args, shape):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    prefix = min(512, shape["seq"])
    for _ in range(args.warmup_ref):
        oracle_sample(shape, args.ref_rows, prefix)
    times, fl, cores = [], 0.0, 1
    for _ in range(args.steps_ref):
        fl, dt, cores = oracle_sample(shape, args.ref_rows, prefix)
        times.append(dt)
    t = sum(times) / len(times)
    val = fl / t / 1e12
    sample = (f"first {prefix} tokens of sequence 0 of {shape['batch']}: RMSNorm + K,V projections for the prefix, block "
              f"output for {args.ref_rows} token rows ({fl / 1e9:.1f} GFLOP per step)")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus, "steps": args.steps_ref,
        "warmup": args.warmup_ref, "ms_per_step": t * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"LLaMA-{args.shape} block forward, oracle on a bounded sample", **shape},
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


# ---- replicas: the path does not shard, so N GPUs run N independent replicas ------------------------------------------
def replica_aggregate(ms_values, flops_per_replica_step, steps, world, device="cpu"):
    """Whole-job throughput of `world` independent replicas: every rank contributes its device-timed milliseconds for
    `steps` steps; the job time is the MAX over ranks; the job did world x steps x flops. Returns (ms maxima, TFLOP/s)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(ms_values), dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms = t.tolist()
    return ms, [world * flops_per_replica_step / (m / steps * 1e-3) / 1e12 for m in ms]


# ---- GPU leg ---------------------------------------------------------------------------------------------------
class ClockSampler:
    """nvidia-smi polled every 20 ms in a child process that is started well before the timed region (its start-up takes longer
    than a short region lasts); every sample carries nvidia-smi's own timestamp, and only those that fall inside the region
    marked by mark_start() / mark_end() are reported."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.proc = None
        self.t0 = self.t1 = None
        self.lines = []
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            import threading
            self.reader = threading.Thread(target=lambda: self.lines.extend(self.proc.stdout), daemon=True)   # keeps the pipe drained
            self.reader.start()
        except Exception:
            self.proc = None

    def mark_start(self):
        self.t0 = time.time()

    def mark_end(self):
        self.t1 = time.time()

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        import datetime
        time.sleep(0.05)
        self.proc.terminate()
        self.reader.join(timeout=10)
        rows = []
        for line in list(self.lines):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(f[1]), float(f[2]), f[4:8]))
            except ValueError:
                continue
        t0 = self.t0 if self.t0 is not None else 0.0
        t1 = self.t1 if self.t1 is not None else float("inf")
        inside = [r for r in rows if t0 <= r[0] <= t1]
        note = None
        if not inside and rows:   # a region shorter than the polling period: the samples nearest to it
            mid = 0.5 * (t0 + min(t1, t0 + 3600.0))
            inside = sorted(rows, key=lambda r: abs(r[0] - mid))[:3]
            note = "no sample fell inside the timed region; the three nearest are reported"
        sm = [r[1] for r in inside]
        mx = [r[2] for r in inside]
        reasons = set()
        for r in inside:
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        res = {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
               "reasons": sorted(reasons), "samples": len(sm)}
        if note:
            res["note"] = note
        return res


TRAFFIC_PROFILE = os.path.join("profiles", "gemm_tc_kernel_dram_traffic_llama7b_block.md")


def recorded_traffic(args):
    """DRAM bytes per launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum, mean over the launches
    of one step) as recorded in the ncu summary under profiles/. The summary names the workload it was captured on and the
    SHA-256 of the kernel source it was captured with; the figure is reported only for that workload and that source,
    otherwise traffic is null with the reason."""
    import hashlib
    import re
    path = os.path.join(ROOT, TRAFFIC_PROFILE)
    if not os.path.exists(path):
        return {"traffic": None, "traffic_note": f"{TRAFFIC_PROFILE} is missing"}
    text = open(path).read()
    m_t = re.search(r"traffic_bytes_per_launch:\s*([0-9.eE+]+)", text)
    m_a = re.search(r"algorithmic_bytes_per_launch:\s*([0-9.eE+]+)", text)
    m_h = re.search(r"sha256\(k_gemm_tc\.cu\):\s*([0-9a-f]{64})", text)
    m_c = re.search(r"captured_at_commit:\s*([0-9a-f]{7,40})", text)
    if not (m_t and m_h):
        return {"traffic": None, "traffic_note": f"{TRAFFIC_PROFILE} carries no machine-readable traffic record"}
    src = os.path.join(ROOT, "paper_2609_03905_b200", "csrc", "k_gemm_tc.cu")
    digest = hashlib.sha256(open(src, "rb").read()).hexdigest()
    if digest != m_h.group(1):
        return {"traffic": None, "traffic_note": f"k_gemm_tc.cu has changed since {TRAFFIC_PROFILE} was captured; no current figure"}
    if not (args.shape == "7b" and args.plan == "mixed" and not args.unfused):
        return {"traffic": None, "traffic_note": "the recorded capture is of the 7b / mixed / fused step only"}
    return {"traffic": float(m_t.group(1)), "traffic_unit": "bytes per launch (ncu, one pass, full workload)",
            "traffic_algorithmic": float(m_a.group(1)) if m_a else None, "traffic_source": TRAFFIC_PROFILE,
            "traffic_commit": m_c.group(1) if m_c else None}


def run_gpu(args, shape):
    import torch
    import torch.distributed as dist
    import paper_2609_03905_b200 as ja
    from paper_2609_03905_b200.llama_block import LlamaBlock
    import synth_inputs as si

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    sampler = ClockSampler(local) if rank == 0 else None   # started during set-up so that it is polling long before the timed region
    bf = torch.float16 if args.dtype == "f16" else torch.bfloat16     # cell type of every relation of the block
    Bt, S, hidden, heads, ffn = shape["batch"], shape["seq"], shape["hidden"], shape["heads"], shape["ffn"]
    T = Bt * S
    kvh = shape.get("kv_heads") or heads
    weights = si.llama_weights(hidden, ffn, dtype=bf, kv_hidden=hidden // heads * kvh)
    blk = LlamaBlock(Bt, S, hidden, heads, ffn, weights, plan=args.plan, fused=not args.unfused, n_kv_heads=kvh, dtype=bf)
    x_host = si.normal((T, hidden), 0.0, 1.0, bf, 5, 0).pin_memory()
    out_host = torch.empty((T, hidden), dtype=bf).pin_memory()
    x_dev = torch.empty((T, hidden), dtype=bf, device="cuda")
    x_dense = ja.Relation([T, hidden], [[0, T], [0, hidden]], bf, x_dev.reshape(-1))
    out_dense = ja.Relation([T, hidden], [[0, T], [0, hidden]], bf)
    x_dev.copy_(x_host)
    ja.repartition(x_dense, blk.x)
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()

    # ---- op-level timing hooks: CUDA events around every libja call of a step ------------------------------
    events = []  # (name, start, end)

    def timed_forward(record: bool):
        if not record:
            blk.forward()
            return
        import paper_2609_03905_b200.relations as R
        orig_exec, orig_rep = R.B.ja_execute, R.B.ja_repartition
        names = iter(blk.op_names())

        def wrap(fn):
            def inner(*a, **k):
                s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                s.record(stream)
                fn(*a, **k)
                e.record(stream)
                events.append((next(names), s, e))
            return inner
        R.B.ja_execute, R.B.ja_repartition = wrap(orig_exec), wrap(orig_rep)
        try:
            blk.forward()
        finally:
            R.B.ja_execute, R.B.ja_repartition = orig_exec, orig_rep

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        timed_forward(False)
    sync_all()
    assert ja.ja_stream_status(stream.cuda_stream) == 0, "device status word set during warm-up"

    # ---- timed region: K steps, inputs resident in HBM ---------------------------------------------------------
    launches0 = ja.ja_launch_count()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    if sampler:
        sampler.mark_start()
    t_start.record(stream)
    for _ in range(args.steps):
        timed_forward(True)
    t_end.record(stream)
    sync_all()
    if sampler:
        sampler.mark_end()
    launches = ja.ja_launch_count() - launches0
    clocks = sampler.stop() if sampler else None
    ms_total = t_start.elapsed_time(t_end)
    assert ja.ja_stream_status(stream.cuda_stream) == 0, "device status word set during the timed region"

    # ---- the same K steps replayed from one CUDA graph of the chain (no per-op events inside a graph, so the per-op
    # breakdown and the roofline above come from the eager region) ------------------------------------------------
    graph = blk.capture()
    sync_all()
    for _ in range(3):
        graph.replay()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    g0.record(stream)
    for _ in range(args.steps):
        graph.replay()
    g1.record(stream)
    sync_all()
    ms_graph = g0.elapsed_time(g1)
    assert ja.ja_stream_status(stream.cuda_stream) == 0, "device status word set during graph replay"
    del graph

    # ---- end to end: every step copies its input from pinned host memory, packs it into the block's input relation
    # (ja_repartition), runs the block, recomposes the output (ja_repartition) and copies it back to the host. Steps are
    # independent, so the copies of neighbouring steps overlap the compute of this one: H2D on one stream, kernels on the
    # caller's stream, D2H on a third, two staging buffers each, ordered by events.
    x_devs = [x_dev, torch.empty_like(x_dev)]
    x_denses = [x_dense, ja.Relation([T, hidden], [[0, T], [0, hidden]], bf, x_devs[1].reshape(-1))]
    out_denses = [out_dense, ja.Relation([T, hidden], [[0, T], [0, hidden]], bf)]
    out_hosts = [out_host, torch.empty((T, hidden), dtype=bf).pin_memory()]
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]         # H2D of buffer b finished
    ev_packed = [torch.cuda.Event() for _ in range(2)]     # buffer b consumed by the pack relayout
    ev_out = [torch.cuda.Event() for _ in range(2)]        # output buffer b written
    ev_d2h = [torch.cuda.Event() for _ in range(2)]        # output buffer b copied to the host
    step_no = [0]

    def e2e_step():
        i = step_no[0]
        b = i & 1
        step_no[0] += 1
        with torch.cuda.stream(s_in):
            if i >= 2:
                s_in.wait_event(ev_packed[b])
            x_devs[b].copy_(x_host, non_blocking=True)
            ev_in[b].record(s_in)
        stream.wait_event(ev_in[b])
        ja.repartition(x_denses[b], blk.x)
        ev_packed[b].record(stream)
        blk.forward()
        if i >= 2:
            stream.wait_event(ev_d2h[b])
        ja.repartition(blk.out, out_denses[b])
        ev_out[b].record(stream)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_out[b])
            out_hosts[b].copy_(out_denses[b].payload[: T * hidden].view(T, hidden), non_blocking=True)
            ev_d2h[b].record(s_out)

    def e2e_drain():
        stream.wait_stream(s_in)
        stream.wait_stream(s_out)

    for _ in range(min(args.warmup, 3)):
        e2e_step()
    e2e_drain()
    sync_all()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        e2e_step()
    e2e_drain()
    e1.record(stream)
    sync_all()
    ms_e2e = e0.elapsed_time(e1)
    assert torch.equal(out_hosts[0], out_hosts[1]), "end-to-end outputs of consecutive steps differ"

    fl = block_flops(Bt, S, hidden, ffn, heads, shape.get("kv_heads"))
    (ms_total, ms_e2e, ms_graph), (value, e2e_val, graph_val) = replica_aggregate([ms_total, ms_e2e, ms_graph], fl, args.steps, world, device="cuda")
    ms_step = ms_total / args.steps

    # ---- per-op breakdown and the roofline of the dominant kernel -----------------------------------------------------
    per_op = {}
    for name, s, e in events:
        per_op.setdefault(name, []).append(s.elapsed_time(e))
    ops = {k: sum(v) / len(v) for k, v in per_op.items()}
    kv_hidden = hidden // heads * kvh
    fl_h, fl_f, fl_kv = 2.0 * T * hidden * hidden, 2.0 * T * hidden * ffn, 2.0 * T * hidden * kv_hidden
    gemm_flops_all = {"q_proj": fl_h, "k_proj": fl_kv, "v_proj": fl_kv, "o_proj": fl_h, "w1_proj": fl_f, "w3_proj": fl_f, "w2_proj": fl_f,
                      "q_proj_rope": fl_h, "k_proj_rope": fl_kv, "o_proj_add": fl_h, "w13_swiglu": 2 * fl_f, "w2_proj_add": fl_f}
    gemm_flops = {k: v for k, v in gemm_flops_all.items() if k in ops}
    gemm_ms = sum(ops[k] for k in gemm_flops)
    peaks = measured_peaks()
    achieved = sum(gemm_flops.values()) / (gemm_ms * 1e-3) / 1e12
    # Denominator: the burst cuBLAS figure when the timed region is short (under a second the part has not settled at its
    # power-capped clock: the condition the burst peak was measured in), the sustained one for long regions.
    short_region = ms_total < 1000.0
    peak_used = peaks["bf16"] if short_region else peaks["bf16_sustained"]
    roof = {"bound": "tensor", "kernel": f"gemm_tc_kernel ({len(gemm_flops)} launches per step)", "achieved": achieved,
            "peak": peak_used, "unit": "TFLOP/s", "frac": achieved / peak_used,
            "peak_source": peaks["source"] + (" (burst cuBLAS bf16: timed region %.0f ms)" % ms_total if short_region
                                              else " (sustained cuBLAS bf16: timed region %.0f ms)" % ms_total),
            "frac_of_burst_peak": achieved / peaks["bf16"], "frac_of_sustained_peak": achieved / peaks["bf16_sustained"],
            "traffic": None, "share_of_step": gemm_ms / ms_step,
            "algorithmic_flops_per_launch": sum(gemm_flops.values()) / len(gemm_flops)}
    roof.update(recorded_traffic(args))
    mem_bytes = {"rmsnorm_1": 4.0 * T * hidden, "rmsnorm_2": 4.0 * T * hidden, "rope_q": 4.0 * T * hidden, "rope_k": 4.0 * T * kv_hidden,
                 "residual_1": 6.0 * T * hidden, "residual_2": 6.0 * T * hidden, "silu_mul": 6.0 * T * ffn}
    for k in ops:
        if k.startswith("repartition"):
            mem_bytes[k] = 4.0 * T * (kv_hidden if k in ("repartition_k", "repartition_v") else hidden)
    hbm = {k: {"ms": ops[k], "GBps": mem_bytes[k] / (ops[k] * 1e-3) / 1e9, "frac_of_measured_hbm": mem_bytes[k] / (ops[k] * 1e-3) / 1e9 / peaks["hbm_gbs"]}
           for k in mem_bytes if k in ops}
    attn_fl = 4.0 * T * S * hidden / 2
    detail = {"ops_ms": ops, "memory_bound_ops": hbm,
              "attention": {"ms": ops["attention"], "TFLOPs": attn_fl / (ops["attention"] * 1e-3) / 1e12},
              "gemm_TFLOPs": {k: gemm_flops[k] / (ops[k] * 1e-3) / 1e12 for k in gemm_flops},
              "fused_chains": {"rope": blk.fuse_rope, "residual_add": blk.fuse_add, "swiglu": blk.fuse_swiglu}}

    # ---- configurations 1-4 of the benchmark definition: their kernels in isolation, after the headline region (the block's
    # relations stay allocated; every timed launch is preceded by an L2 flush), with the clocks of this sub-run
    configs = None
    if rank == 0 and args.shape == "7b" and not args.no_configs:
        cs = ClockSampler(local)
        time.sleep(0.3)
        cs.mark_start()
        configs = {c: case_results(c, args.config_reps) for c in ("cfg1", "cfg2", "cfg3", "cfg4")}
        torch.cuda.synchronize()
        cs.mark_end()
        configs = {"l2": L2_NOTE, "reps_per_kernel": args.config_reps, "clocks": cs.stop(), "kernels": configs,
                   "peaks": {"hbm_GBps": peaks["hbm_gbs"], "bf16_TFLOPs_burst": peaks["bf16"], "source": peaks["source"]}}

    if rank != 0:
        return
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cfl, cdt, cores = oracle_sample(shape, args.ref_rows)
        cpu = {"value": cfl / cdt / 1e12, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "seconds": cdt,
               "sample": f"sequence 0 of {Bt}: RMSNorm + K,V projections for all {S} tokens, block output for {args.ref_rows} "
                         f"token rows ({cfl / 1e9:.1f} GFLOP)"}
    print(json.dumps({
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": args.dtype,
        "data": "synthetic",
        "config": {"workload": f"LLaMA-{args.shape} block forward as chained join-aggs, plan '{args.plan}' "
                               f"({blk.n_relayouts} ja_repartition relayouts per step; fused chains: {'on' if not args.unfused else 'off'})", **shape,
                   "l2": "working set per step (weights 405 MB + activations) exceeds the 126 MB L2; no flush needed",
                   "replicas": "independent replica per GPU (path does not shard)" if world > 1 else "single GPU"},
        "clocks": clocks, "gpu_launches": launches,
        "e2e": {"value": e2e_val, "unit": "TFLOP/s", "ms_per_step": ms_e2e / args.steps,
                "h2d_bytes_per_step": x_host.numel() * 2, "d2h_bytes_per_step": out_host.numel() * 2},
        "cuda_graph_replay": {"value": graph_val, "unit": "TFLOP/s", "ms_per_step": ms_graph / args.steps,
                              "note": "the same steps replayed from one CUDA graph of the chain, timed after the eager region"},
        "roofline": roof, "cpu_baseline": cpu, "configs": configs, "detail": detail}))
    if world > 1:
        dist.destroy_process_group()


# ---- single-config kernel benchmarks (configs 2, 3, 4 of the benchmark definition) ----------------------------------
L2_NOTE = "512 MiB flush buffer written, then a 256 MiB buffer read (clean lines), before every timed launch"


def physical_results():
    """Section 6, Experiment 4 in miniature, on the library's simulator (host only, no GPU): the exchange programs that link the
    operators of a plan the logical optimizer chose for eight GPUs -- the 7B block and matrix chains A and B -- compiled
    naively (function spec i on GPU i, every aggregated block gathered and aggregated where it is consumed) and with
    placement and synthesis, on the NVSwitch model of the DGX-A100 and on the cube mesh of the DGX-V100."""
    import paper_2609_03905_b200 as ja
    from paper_2609_03905_b200 import exprog as X, physical
    from paper_2609_03905_b200.planned_block import block_graph
    workloads = {}
    ops = block_graph(8, 2048, 4096, 32, 11008)
    workloads["llama7b_block"] = (ops, ja.ja_plan_optimize_graph(ops, 8)[1])
    chains = {"chain_A": ([10240] + [16384, 6144] * 4 + [10240], ((0, 1), (((2, 3), ((4, 5), (6, 7))), 8))),
              "chain_B": ([9216, 20480, 5120, 20480, 5120, 9216], ((0, 1), ((2, 3), 4)))}
    for name, (dims, tree) in chains.items():
        ops = []

        def build(t):   # returns (producer index or None, rows, cols)
            if isinstance(t, int):
                return None, dims[t], dims[t + 1]
            (a, m, j), (b, _, n) = build(t[0]), build(t[1])
            ops.append({"einsum": "ij,jk->ik", "extents": {"i": m, "j": j, "k": n}, "inputs": [a, b]})
            return len(ops) - 1, m, n
        build(tree)
        workloads[name] = (ops, ja.ja_plan_optimize(ops, 8)[1])
    res = {}
    # Experiments 3 and 5 in miniature on the simulator: the three plan selectors for the block at p = 8 -- the dynamic program,
    # greedy (no repartition sub-cost), twenty uniform draws -- by the simulated time of their optimised exchange programs, and
    # the Pearson correlation between a plan's proxy cost and that time over all 22 plans
    import random
    ops = workloads["llama7b_block"][0]

    def valid_specs(op, p_):
        letters = []
        for term in op["einsum"].replace("->", ",").split(","):
            letters += [c for c in term if c not in letters]
        out = []

        def rec(i, rest, acc):
            if i == len(letters):
                if rest == 1:
                    out.append(dict(zip(letters, acc)))
                return
            if letters[i] in op.get("fixed", ()):
                rec(i + 1, rest, acc + [1])
                return
            for c_ in range(1, rest + 1):
                if rest % c_ == 0 and c_ <= op["extents"][letters[i]]:
                    rec(i + 1, rest // c_, acc + [c_])
        rec(0, p_, [])
        return out

    def pearson(xs, ys):
        n = len(xs)
        mx, my = sum(xs) / n, sum(ys) / n
        sxy = sum((x - mx) * (y - my) for x, y in zip(xs, ys))
        sxx, syy = sum((x - mx) ** 2 for x in xs), sum((y - my) ** 2 for y in ys)
        return sxy / (sxx * syy) ** 0.5 if sxx > 0 and syy > 0 else float("nan")

    rng = random.Random(3905)
    cand = [valid_specs(op, 8) for op in ops]
    plans = {"optimizer": workloads["llama7b_block"][1], "greedy": ja.ja_plan_select_greedy(ops, 8)[1]}
    for i in range(20):
        plans["random_%02d" % i] = [rng.choice(c_) for c_ in cand]
    for mname in ("dgx_a100", "dgx_v100"):
        mach = X.ja_machine_preset(mname)
        ms = {k: physical.compile_exchanges(ops, pl, mach, True, depth=1, beam=4)[0] for k, pl in plans.items()}
        cost = {k: ja.ja_plan_cost(ops, pl) for k, pl in plans.items()}
        draws = sorted(v for k, v in ms.items() if k.startswith("random"))
        res["plan_selection_p8_%s" % mname] = {
            "optimizer_exchange_ms": ms["optimizer"], "greedy_exchange_ms": ms["greedy"], "random_best_ms": draws[0],
            "random_median_ms": (draws[9] + draws[10]) / 2, "random_worst_ms": draws[-1],
            "plans_beating_the_optimizer": sum(1 for k, v in ms.items() if v < ms["optimizer"] * (1 - 1e-9)),
            "pearson_r_proxy_cost_vs_exchange_ms": pearson([cost[k] for k in plans], [ms[k] for k in plans]), "n_plans": len(plans)}
    for name, (ops, plan) in workloads.items():
        for mname in ("dgx_a100", "dgx_v100"):
            mach = X.ja_machine_preset(mname)
            naive, en = physical.compile_exchanges(ops, plan, mach, False)
            opt, eo = physical.compile_exchanges(ops, plan, mach, True, depth=2, beam=6)
            res["%s_%s" % (name, mname)] = {"naive_ms": naive, "optimised_ms": opt, "naive_over_optimised": naive / opt if opt > 0 else 1.0,
                                            "operators_with_produced_operands": len(en), "of_them_with_traffic": sum(1 for e in en if e["ms"] > 0),
                                            "proxy_cost_cells": ja.ja_plan_cost(ops, plan)}
    return res


def run_case(args):
    """Times the kernels of one benchmark configuration in isolation and prints one JSON line."""
    if args.case == "physical":
        print(json.dumps({"case": "physical", "simulated": True, "results": physical_results()}))
        return
    import torch
    torch.cuda.set_device(0)
    res = case_results(args.case, args.steps)
    print(json.dumps({"case": args.case, "reps": args.steps, "l2": L2_NOTE, "peaks": measured_peaks(), "kernels": res}))


def case_results(case, reps):
    """The kernels of one benchmark configuration in isolation: CUDA events around each launch on the current stream, L2
    flushed before every timed launch. Returns {kernel: {ms_mean, ms_min, ms_median, TFLOPs | GBps, fraction of measured peak}}."""
    import torch
    import paper_2609_03905_b200 as ja
    import synth_inputs as si
    ES = ja.equal_splits
    bf, f32 = torch.bfloat16, torch.float32
    stream = torch.cuda.current_stream()
    peaks = measured_peaks()

    class _A:
        pass
    args = _A()
    args.case, args.steps = case, reps
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    # Writing the flush buffer evicts the inputs but leaves L2 full of DIRTY lines, whose write-back (up to the L2 size,
    # about as many bytes as a small kernel moves) would then be charged to the kernel under test; a read sweep over a
    # second buffer larger than L2 leaves clean lines instead, as a kernel meets in a running program.
    clean = torch.zeros(256 << 20, dtype=torch.uint8, device="cuda").view(torch.int32)

    def timeit(fn, reps, flush_l2):
        for _ in range(3):
            fn(0)
        torch.cuda.synchronize()
        ts = []
        for r in range(reps):
            if flush_l2:
                flush.fill_(r & 0xFF)
                clean.sum()
            s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s.record(stream)
            fn(r)
            e.record(stream)
            torch.cuda.synchronize()
            ts.append(s.elapsed_time(e))
        ts.sort()
        return {"ms_mean": sum(ts) / len(ts), "ms_min": ts[0], "ms_median": ts[len(ts) // 2]}

    def timeit_graph(fn, reps, flush_l2):
        """As timeit, for launches shorter than the host's own marshalling of the call (~15 us per relation through
        Python): the call is recorded into a CUDA graph once and each timed region is one replay."""
        for _ in range(3):
            fn(0)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn(0)
        return timeit(lambda r: g.replay(), reps, flush_l2)

    def rel(shape, splits, dtype=bf, std=1.0):
        r = ja.Relation(list(shape), splits, dtype)
        r.payload.normal_(0.0, std)
        return r

    res = {}
    reps = args.steps
    if args.case == "cfg1":
        # 33.5 MFLOP: not a throughput case. Two figures per decomposition: one launch on an idle GPU between two events (what a
        # caller that waits for every result sees: launch latency + event resolution dominate), and the time per launch in a
        # train of 20 launches between the two events (what the kernel costs inside a running program).
        def train(fn, n=20):
            """n launches recorded into one CUDA graph (the host's enqueue cost per call, ~15 us through Python, would
            otherwise be what is measured) and the replay timed between two events."""
            for _ in range(3):
                fn(0)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for _ in range(n):
                    fn(0)
            g.replay()
            torch.cuda.synchronize()
            ts = []
            for r in range(max(5, reps // 4)):
                s_, e_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                s_.record(stream)
                g.replay()
                e_.record(stream)
                torch.cuda.synchronize()
                ts.append(s_.elapsed_time(e_) / n)
            ts.sort()
            return {"ms_mean": sum(ts) / len(ts), "ms_min": ts[0], "ms_median": ts[len(ts) // 2]}

        for grid in ((4, 4, 4), (2, 8, 4)):
            ti, tj, tk = (ES(256, g) for g in grid)
            A, Bm, C = rel((256, 256), [ti, tj], f32), rel((256, 256), [tj, tk], f32), rel((256, 256), [ti, tk], f32)
            sp = ja.Spec("ij,jk->ik", {"i": ti, "j": tj, "k": tk})
            t1 = timeit(lambda r: sp.execute([A, Bm], C), reps, False)
            t = train(lambda r: sp.execute([A, Bm], C))
            res["matmul_f32_256_grid_%dx%dx%d" % grid] = {**t, "GFLOPs": 2.0 * 256 ** 3 / (t["ms_mean"] * 1e-3) / 1e9,
                                                          "single_launch_on_idle_gpu_ms": t1["ms_mean"],
                                                          "note": "plain fp32 ALUs; ms = per launch in a CUDA graph of 20 launches; launch-latency bound at this size"}
        # supplementary, not one of the benchmark configurations: the same kernel where it has work to do. fp32 FMA peak from
        # the device: SMs x 128 lanes x 2 flop x clock
        n = 4096
        tb = ES(n, 8)
        A, Bm, C = rel((n, n), [tb, tb], f32), rel((n, n), [tb, tb], f32), rel((n, n), [tb, tb], f32)
        sp = ja.Spec("ij,jk->ik", {"i": tb, "j": tb, "k": tb})
        t = timeit(lambda r: sp.execute([A, Bm], C), max(3, reps // 10), True)
        props = torch.cuda.get_device_properties(0)
        clock_khz = getattr(props, "clock_rate", None) or 1965000
        peak = props.multi_processor_count * 128 * 2 * clock_khz * 1e3 / 1e12
        tf = 2.0 * n ** 3 / (t["ms_mean"] * 1e-3) / 1e12
        res["supplementary_matmul_f32_4096_grid_8x8x8"] = {**t, "TFLOPs": tf, "fp32_fma_peak_TFLOPs": peak, "frac_of_fp32_fma_peak": tf / peak,
                                                           "note": "not a benchmark configuration; peak = SMs x 128 FMA lanes x 2 x max clock"}
    elif args.case == "cfg2":
        T, d, f = 2048, 4096, 11008
        ti, td, tf = ES(T, 8), ES(d, 8), ES(f, 8)
        x, W1, W3, W2 = rel((T, d), [ti, td]), rel((d, f), [td, tf], std=0.02), rel((d, f), [td, tf], std=0.02), rel((f, d), [tf, td], std=0.02)
        a, b, h, y = rel((T, f), [ti, tf]), rel((T, f), [ti, tf]), rel((T, f), [ti, tf]), rel((T, d), [ti, td])
        up = ja.Spec("ij,jk->ik", {"i": ti, "j": td, "k": tf})
        down = ja.Spec("ij,jk->ik", {"i": ti, "j": tf, "k": td})
        silu = ja.Spec("ij,ij->ij", {"i": ti, "j": tf}, "silu_mul", (), "none")
        fl = 2.0 * T * d * f
        for name, fn in (("gemm_x_W1", lambda r: up.execute([x, W1], a)), ("gemm_x_W3", lambda r: up.execute([x, W3], b)),
                         ("gemm_h_W2", lambda r: down.execute([h, W2], y))):
            t = timeit(fn, reps, True)
            res[name] = {**t, "TFLOPs": fl / (t["ms_mean"] * 1e-3) / 1e12, "frac_of_burst_bf16_peak": fl / (t["ms_mean"] * 1e-3) / 1e12 / peaks["bf16"]}
        t = timeit(lambda r: silu.execute([a, b], h), reps, True)
        res["silu_mul"] = {**t, "GBps": 6.0 * T * f / (t["ms_mean"] * 1e-3) / 1e9, "frac_of_measured_hbm": 6.0 * T * f / (t["ms_mean"] * 1e-3) / 1e9 / peaks["hbm_gbs"]}

        def chain(r):
            up.execute([x, W1], a); up.execute([x, W3], b); silu.execute([a, b], h); down.execute([h, W2], y)
        t = timeit(chain, reps, True)
        res["mlp_chain"] = {**t, "TFLOPs": 3 * fl / (t["ms_mean"] * 1e-3) / 1e12}
    elif args.case == "cfg3":
        ti, tj = ES(8192, 8), ES(4096, 8)
        parts = {"i": ti, "j": tj}
        X, G, Y = rel((8192, 4096), [ti, tj], std=2.0), rel((4096,), [tj]), rel((8192, 4096), [ti, tj])
        SS = ja.Relation([8192], [ti], f32)
        hb = lambda nbytes, t: {**t, "GBps": nbytes / (t["ms_mean"] * 1e-3) / 1e9, "frac_of_measured_hbm": nbytes / (t["ms_mean"] * 1e-3) / 1e9 / peaks["hbm_gbs"]}
        nb = 8192 * 4096 * 2.0
        s_fused = ja.Spec("ij,j->ij", parts, "rmsnorm", (1e-5,), "none")
        s_ss = ja.Spec("ij->i", parts, "square", (), "sum")
        s_sc = ja.Spec("ij,i,j->ij", parts, "rms_scale", (1e-5,), "none")
        res["rmsnorm_fused"] = hb(2 * nb, timeit(lambda r: s_fused.execute([X, G], Y), reps, True))
        res["rmsnorm_sumsq"] = hb(nb, timeit(lambda r: s_ss.execute([X], SS), reps, True))
        res["rmsnorm_scale"] = hb(2 * nb, timeit(lambda r: s_sc.execute([X, SS, G], Y), reps, True))
        th, si_, sj = ES(32, 32), ES(2048, 8), ES(2048, 8)
        p3 = {"h": th, "i": si_, "j": sj}
        S, P = rel((32, 2048, 2048), [th, si_, sj], std=2.0), rel((32, 2048, 2048), [th, si_, sj])
        M, L = ja.Relation([32, 2048], [th, si_], f32), ja.Relation([32, 2048], [th, si_], f32)
        nb = 32 * 2048 * 2048 * 2.0
        s_sm = ja.Spec("hij->hij", p3, "softmax", (), "none")
        s_mx = ja.Spec("hij->hi", p3, "ident", (), "max")
        s_es = ja.Spec("hij,hi->hi", p3, "exp_sub", (), "sum")
        s_dv = ja.Spec("hij,hi,hi->hij", p3, "exp_sub_div", (), "none")
        res["softmax_fused"] = hb(2 * nb, timeit(lambda r: s_sm.execute([S], P), reps, True))
        res["softmax_max"] = hb(nb, timeit(lambda r: s_mx.execute([S], M), reps, True))
        res["softmax_expsum"] = hb(nb, timeit(lambda r: s_es.execute([S, M], L), reps, True))
        res["softmax_divide"] = hb(2 * nb, timeit(lambda r: s_dv.execute([S, M, L], P), reps, True))
        src = rel((16384, 4096), [ES(16384, 128), ES(4096, 8)])
        dst = ja.Relation([16384, 4096], [ES(16384, 128), ES(4096, 32)], bf)
        res["repartition_128x512_to_128x128"] = hb(2 * 16384 * 4096 * 2.0, timeit(lambda r: ja.repartition(src, dst), reps, True))
    elif args.case == "cfg4":
        Bn, S, H, D = 4, 2048, 32, 128
        sp = [ES(Bn, Bn), ES(S, S // 128), ES(H, H), [0, D]]
        Q, K, V, O = (rel((Bn, S, H, D), sp) for _ in range(4))
        parts = {"b": sp[0], "q": sp[1], "h": sp[2], "d": sp[3], "k": sp[1]}
        spec = ja.Spec("bqhd,bkhd,bkhd->bqhd", parts, "attention", (1.0 / D ** 0.5, 1.0), "online_softmax")
        t = timeit(lambda r: spec.execute([Q, K, V], O), reps, True)
        fl = 4.0 * Bn * H * S * S * D / 2
        res["attention_causal"] = {**t, "TFLOPs": fl / (t["ms_mean"] * 1e-3) / 1e12, "TFLOPs_executed_blocks": fl * 136 / 128 / (t["ms_mean"] * 1e-3) / 1e12,
                                   "frac_of_burst_bf16_peak": fl / (t["ms_mean"] * 1e-3) / 1e12 / peaks["bf16"]}
    elif args.case == "gqa":
        # Example 3.10: 32 query heads on 8 key/value heads, sequence index 4096 holding sequences that end at 1024, 2560, 4096
        Bn, S, Hq, Hkv, D, grp = 8, 4096, 32, 8, 128, 4
        ends = [1024, 2560, 4096]
        gs = list(range(Hkv + 1))
        hs = [grp * v for v in gs]
        fl_packed = 4.0 * Bn * Hq * D * sum((b - a) ** 2 for a, b in zip([0] + ends[:-1], ends)) / 2
        for name, s_split, prm_ends, fl in (("gqa_packed_cut_at_ends", [0] + ends, ends, fl_packed),
                                            ("gqa_packed_128_row_blocks", ES(S, S // 128), ends, fl_packed),
                                            ("gqa_one_sequence", ES(S, S // 128), [], 4.0 * Bn * Hq * S * S * D / 2)):
            q_sp, k_sp = [ES(Bn, Bn), s_split, hs, [0, D]], [ES(Bn, Bn), s_split, gs, [0, D]]
            Q, O = rel((Bn, S, Hq, D), q_sp), rel((Bn, S, Hq, D), q_sp)
            K, V = rel((Bn, S, Hkv, D), k_sp), rel((Bn, S, Hkv, D), k_sp)
            parts = {"b": q_sp[0], "q": s_split, "h": hs, "d": [0, D], "k": s_split, "g": gs}
            spec = ja.Spec("bqhd,bkgd,bkgd->bqhd", parts, "attention", (1.0 / D ** 0.5, 1.0) + tuple(map(float, prm_ends)), "online_softmax")
            t = timeit(lambda r: spec.execute([Q, K, V], O), reps, True)
            res[name] = {**t, "TFLOPs": fl / (t["ms_mean"] * 1e-3) / 1e12, "frac_of_burst_bf16_peak": fl / (t["ms_mean"] * 1e-3) / 1e12 / peaks["bf16"],
                         "tuples": ja.ja_spec_num_tuples(spec.handle)[0]}
    elif args.case == "agg":
        # a producer executed through its join (m unaggregated copies per output block) and the aggregating relayout
        # that delivers aggregated blocks in the consumer's tiling: the down projection of the 7B block, contracted index
        # cut into m blocks; the consumer wants 128-row x 512-column blocks
        T, f, d = 16384, 11008, 4096
        hb = lambda nbytes, t: {**t, "GBps": nbytes / (t["ms_mean"] * 1e-3) / 1e9, "frac_of_measured_hbm": nbytes / (t["ms_mean"] * 1e-3) / 1e9 / peaks["hbm_gbs"]}
        for m, pdt in ((2, bf), (4, bf), (8, bf), (4, f32)):
            ti, tf, td = ES(T, 16), ES(f, m), ES(d, 8)
            h, W2 = rel((T, f), [ti, tf]), rel((f, d), [tf, td], std=0.02)
            P = ja.partial_relation(m, [T, d], [ti, td], pdt)
            y = ja.Relation([T, d], [ES(T, 128), ES(d, 8)], bf)
            spec = ja.Spec("ij,jk->ik", {"i": ti, "j": tf, "k": td})
            tag = "m%d_%s" % (m, "f32" if pdt == f32 else "bf16")
            t = timeit(lambda r: spec.execute_join([h, W2], P), reps, True)
            fl = 2.0 * T * f * d
            res["join_only_matmul_" + tag] = {**t, "TFLOPs": fl / (t["ms_mean"] * 1e-3) / 1e12, "frac_of_burst_bf16_peak": fl / (t["ms_mean"] * 1e-3) / 1e12 / peaks["bf16"]}
            es = 4 if pdt == f32 else 2
            res["aggregating_relayout_" + tag] = hb((m * es + 2.0) * T * d, timeit(lambda r: ja.repartition_agg(P, "sum", y), reps, True))
            del h, W2, P, y, spec
        # the same for attention: the key index of B4 x 8192 keys cut into m ranges of 2048, one ja_execute (O_c, lse_c) per
        # range against the 2048 queries, then the online-softmax aggregation as its own step (ja_attention_combine)
        Bn, S, H, D = 4, 2048, 32, 128
        sp = [ES(Bn, Bn), ES(S, S // 128), ES(H, H), [0, D]]
        parts = {"b": sp[0], "q": sp[1], "h": sp[2], "d": sp[3], "k": sp[1]}
        aspec = ja.Spec("bqhd,bkhd,bkhd->bqhd", parts, "attention", (1.0 / D ** 0.5, 0.0), "online_softmax")
        Q = rel((Bn, S, H, D), sp)
        for m in (2, 4):
            KV = [(rel((Bn, S, H, D), sp), rel((Bn, S, H, D), sp)) for _ in range(m)]
            Oc = [ja.Relation([Bn, S, H, D], sp, bf) for _ in range(m)]
            Lc = [ja.Relation([Bn, S, H], sp[:3], f32) for _ in range(m)]
            O, L = ja.Relation([Bn, S, H, D], sp, bf), ja.Relation([Bn, S, H], sp[:3], f32)

            def partials(r):
                for c in range(m):
                    aspec.execute([Q, KV[c][0], KV[c][1]], [Oc[c], Lc[c]])
            t = timeit(partials, reps, True)
            fl = 4.0 * Bn * H * S * (m * S) * D
            res["attention_partials_m%d" % m] = {**t, "TFLOPs": fl / (t["ms_mean"] * 1e-3) / 1e12, "frac_of_burst_bf16_peak": fl / (t["ms_mean"] * 1e-3) / 1e12 / peaks["bf16"]}
            nbytes = (m + 1.0) * Bn * S * H * (D * 2 + 4)
            res["attention_combine_m%d" % m] = hb(nbytes, timeit_graph(lambda r: ja.attention_combine(Oc, Lc, O, L), reps, True))
            del KV, Oc, Lc, O, L
    elif args.case == "opt":
        # logical optimization (Algorithm 1) of the SwiGLU MLP tree of config 2, then the chosen plan and three hand
        # plans executed as join-aggs (a relayout wherever a producer's tiling differs from what its consumer's spec needs)
        import time
        T, d, f = 2048, 4096, 11008
        ops = [{"einsum": "ij,jk->ik", "extents": {"i": T, "j": d, "k": f}, "inputs": [None, None]},
               {"einsum": "ij,jk->ik", "extents": {"i": T, "j": d, "k": f}, "inputs": [None, None]},
               {"einsum": "ik,ik->ik", "extents": {"i": T, "k": f}, "inputs": [0, 1]},
               {"einsum": "ik,kl->il", "extents": {"i": T, "k": f, "l": d}, "inputs": [2, None]}]

        def run_plan(plan):
            t_up = [ES(T, plan[0]["i"]), ES(d, plan[0]["j"]), ES(f, plan[0]["k"])]
            t_up3 = [ES(T, plan[1]["i"]), ES(d, plan[1]["j"]), ES(f, plan[1]["k"])]
            t_act = [ES(T, plan[2]["i"]), ES(f, plan[2]["k"])]
            t_dn = [ES(T, plan[3]["i"]), ES(f, plan[3]["k"]), ES(d, plan[3]["l"])]
            x1, W1 = rel((T, d), t_up[:2]), rel((d, f), t_up[1:], std=0.02)
            x3, W3 = rel((T, d), t_up3[:2]), rel((d, f), t_up3[1:], std=0.02)
            a, b = rel((T, f), [t_up[0], t_up[2]]), rel((T, f), [t_up3[0], t_up3[2]])
            a2 = a if [t_up[0], t_up[2]] == t_act else rel((T, f), t_act)
            b2 = b if [t_up3[0], t_up3[2]] == t_act else rel((T, f), t_act)
            h = rel((T, f), t_act)
            h2 = h if t_act == t_dn[:2] else rel((T, f), t_dn[:2])
            W2, y = rel((f, d), t_dn[1:], std=0.02), rel((T, d), [t_dn[0], t_dn[2]])
            s1 = ja.Spec("ij,jk->ik", dict(zip("ijk", t_up)))
            s3 = ja.Spec("ij,jk->ik", dict(zip("ijk", t_up3)))
            sa = ja.Spec("ik,ik->ik", dict(zip("ik", t_act)), "silu_mul", (), "none")
            s2 = ja.Spec("ik,kl->il", dict(zip("ikl", t_dn)))

            def chain(r):
                s1.execute([x1, W1], a); s3.execute([x3, W3], b)
                if a2 is not a: ja.repartition(a, a2)
                if b2 is not b: ja.repartition(b, b2)
                sa.execute([a2, b2], h)
                if h2 is not h: ja.repartition(h, h2)
                s2.execute([h2, W2], y)
            return timeit(chain, reps, True), (a2 is not a) + (b2 is not b) + (h2 is not h)

        for p_ in (8, 64):
            t0 = time.perf_counter()
            best_cost, best = ja.ja_plan_optimize(ops, p_)
            opt_ms = (time.perf_counter() - t0) * 1e3
            q = round(p_ ** (1 / 3))
            hand = {"optimizer": best,
                    "rows_only": [{"i": p_, "j": 1, "k": 1}, {"i": p_, "j": 1, "k": 1}, {"i": p_, "k": 1}, {"i": p_, "k": 1, "l": 1}],
                    "contracted_only": [{"i": 1, "j": p_, "k": 1}, {"i": 1, "j": p_, "k": 1}, {"i": 1, "k": p_}, {"i": 1, "k": p_, "l": 1}],
                    "cube": [{"i": q, "j": q, "k": q}, {"i": q, "j": q, "k": q}, {"i": q, "k": p_ // q}, {"i": q, "k": q, "l": q}]}
            for name, plan in hand.items():
                t, n_rep = run_plan(plan)
                res["p%d_%s" % (p_, name)] = {**t, "proxy_cost_cells": ja.ja_plan_cost(ops, plan), "relayouts": n_rep,
                                              "TFLOPs": 6.0 * T * d * f / (t["ms_mean"] * 1e-3) / 1e12, "plan": plan}
            res["p%d_optimizer_host_ms" % p_] = {"ms_mean": opt_ms, "ms_min": opt_ms, "ms_median": opt_ms, "cost": best_cost}
        # Section 6 ablation in miniature: 20 plans drawn at random (one spec per operator, uniformly from specs(Op) for p = 8,
        # seeded), their proxy cost and measured chain time against the optimizer's plan
        import random

        def all_specs(op, p_):
            letters = []
            for term in op["einsum"].replace("->", ",").split(","):
                letters += [c for c in term if c not in letters]
            out = []

            def rec(i, rest, acc):
                if i == len(letters):
                    if rest == 1: out.append(dict(zip(letters, acc)))
                    return
                for c_ in range(1, rest + 1):
                    if rest % c_ == 0: rec(i + 1, rest // c_, acc + [c_])
            rec(0, p_, [])
            return out

        rng = random.Random(3905)
        cand = [all_specs(op, 8) for op in ops]
        draws = []
        for n_ in range(20):
            plan = [rng.choice(c_) for c_ in cand]
            t, n_rep = run_plan(plan)
            draws.append({"ms": t["ms_median"], "proxy_cost_cells": ja.ja_plan_cost(ops, plan), "relayouts": n_rep, "plan": plan})
        ms_sorted = sorted(d_["ms"] for d_ in draws)
        res["p8_random_20"] = {"ms_mean": sum(ms_sorted) / 20, "ms_min": ms_sorted[0], "ms_median": 0.5 * (ms_sorted[9] + ms_sorted[10]),
                               "ms_max": ms_sorted[-1], "proxy_cost_cells_median": sorted(d_["proxy_cost_cells"] for d_ in draws)[10],
                               "proxy_cost_cells_min": min(d_["proxy_cost_cells"] for d_ in draws), "draws": draws}
    elif args.case == "optblock":
        # Section 4 on the whole block: the optimizer's plans for p = 8 and p = 64 function specs per operator
        # (ja_plan_optimize_graph on the eleven-operator graph, three multiply consumed tensors) executed by PlannedBlock -- a
        # ja_repartition per repartition charge of the plan -- beside the three hand decompositions of LlamaBlock written as
        # interval counts of the same graph, so that the proxy cost (cells) and the measured time stand side by side.
        import time
        from paper_2609_03905_b200.llama_block import LlamaBlock
        from paper_2609_03905_b200.planned_block import PlannedBlock, block_graph, plan_repartition_charges
        shape = SHAPES["7b"]
        Bt, S, hidden, heads, ffn = shape["batch"], shape["seq"], shape["hidden"], shape["heads"], shape["ffn"]
        ops = block_graph(Bt, S, hidden, heads, ffn)
        weights = si.llama_weights(hidden, ffn)
        fl = block_flops(Bt, S, hidden, ffn)
        sb, fb = S // 128, ffn // 256      # the hand plans cut tokens into 128-row blocks and the FFN index into 256-wide ones

        def hand_counts(e_c, h_proj, h_att, wo_h):
            tok = {"b": Bt, "s": sb}
            return [{**tok, "e": e_c}] + [{**tok, "e": e_c, "h": h_proj, "d": 1}] * 3 + \
                   [{"b": Bt, "q": sb, "h": h_att, "d": 1, "k": sb}, {**tok, "h": wo_h, "d": 1, "e": e_c}, {**tok, "e": e_c},
                    {**tok, "e": e_c, "f": fb}, {**tok, "e": e_c, "f": fb}, {**tok, "f": fb}, {**tok, "f": fb, "e": e_c}]
        hands = {"seq": hand_counts(8, 8, heads, 8), "head": hand_counts(heads, heads, heads, heads), "mixed": hand_counts(8, 8, 8, 8)}
        for name, counts in hands.items():
            blk = LlamaBlock(Bt, S, hidden, heads, ffn, weights, plan=name)
            t = timeit(lambda r: blk.forward(), reps, True)
            res["hand_" + name] = {**t, "TFLOPs": fl / (t["ms_mean"] * 1e-3) / 1e12, "proxy_cost_cells": ja.ja_plan_cost(ops, counts),
                                   "repartition_charges": plan_repartition_charges(ops, counts)[0], "relayouts_executed": blk.n_relayouts,
                                   "function_specs_per_matmul": "tokens x %d column blocks" % (len(blk.act_c) - 1)}
            del blk
            torch.cuda.empty_cache()
        for p_ in (8, 64):
            t0 = time.perf_counter()
            cost, plan = ja.ja_plan_optimize_graph(ops, p_)
            opt_ms = (time.perf_counter() - t0) * 1e3
            blk = PlannedBlock(Bt, S, hidden, heads, ffn, weights, plan)
            t = timeit(lambda r: blk.forward(), reps, True)
            res["optimizer_p%d" % p_] = {**t, "TFLOPs": fl / (t["ms_mean"] * 1e-3) / 1e12, "proxy_cost_cells": cost,
                                         "repartition_charges": plan_repartition_charges(ops, plan)[0], "relayouts_executed": blk.n_relayouts,
                                         "optimizer_host_ms": opt_ms, "launches": len(blk.steps), "plan": plan}
            del blk
            torch.cuda.empty_cache()
        # the two other selectors of the paper's plan-selection experiment (Section 6, Experiment 3) at p = 8: greedy (the
        # same program without the repartition sub-cost) and twenty uniform draws among the valid specs of every operator
        cost, plan = ja.ja_plan_select_greedy(ops, 8)
        blk = PlannedBlock(Bt, S, hidden, heads, ffn, weights, plan)
        t = timeit(lambda r: blk.forward(), reps, True)
        res["greedy_p8"] = {**t, "TFLOPs": fl / (t["ms_mean"] * 1e-3) / 1e12, "proxy_cost_cells": cost,
                            "repartition_charges": plan_repartition_charges(ops, plan)[0], "relayouts_executed": blk.n_relayouts,
                            "launches": len(blk.steps), "plan": plan}
        del blk
        torch.cuda.empty_cache()
        import random

        def valid_specs(op, p_):   # specs(Op): interval counts with product p over the shardable letters
            letters = []
            for term in op["einsum"].replace("->", ",").split(","):
                letters += [c for c in term if c not in letters]
            out = []

            def rec(i, rest, acc):
                if i == len(letters):
                    if rest == 1:
                        out.append(dict(zip(letters, acc)))
                    return
                if letters[i] in op.get("fixed", ()):
                    rec(i + 1, rest, acc + [1])
                    return
                for c_ in range(1, rest + 1):
                    if rest % c_ == 0 and c_ <= op["extents"][letters[i]]:
                        rec(i + 1, rest // c_, acc + [c_])
            rec(0, p_, [])
            return out

        rng = random.Random(3905)
        cand = [valid_specs(op, 8) for op in ops]
        draws = []
        for _ in range(20):
            plan = [rng.choice(c_) for c_ in cand]
            blk = PlannedBlock(Bt, S, hidden, heads, ffn, weights, plan)
            t = timeit(lambda r: blk.forward(), max(3, reps // 4), True)
            draws.append({"ms_mean": t["ms_mean"], "proxy_cost_cells": ja.ja_plan_cost(ops, plan), "relayouts_executed": blk.n_relayouts})
            del blk
            torch.cuda.empty_cache()
        ms = sorted(d["ms_mean"] for d in draws)
        res["random_p8_20_draws"] = {"ms_mean": sum(ms) / len(ms), "ms_best": ms[0], "ms_median": (ms[9] + ms[10]) / 2, "ms_worst": ms[-1],
                                     "proxy_cost_cells_median": sorted(d["proxy_cost_cells"] for d in draws)[10],
                                     "relayouts_executed_median": sorted(d["relayouts_executed"] for d in draws)[10]}
        # Section 6, Experiment 5 in miniature: Pearson correlation between the proxy cost of a plan and its measured time, over
        # the twenty draws and over all p = 8 plans timed here (draws, greedy, optimizer, hand plans)

        def pearson(xs, ys):
            n = len(xs)
            mx, my = sum(xs) / n, sum(ys) / n
            sxy = sum((x - mx) * (y - my) for x, y in zip(xs, ys))
            sxx, syy = sum((x - mx) ** 2 for x in xs), sum((y - my) ** 2 for y in ys)
            return sxy / (sxx * syy) ** 0.5 if sxx > 0 and syy > 0 else float("nan")

        pts = [(d["proxy_cost_cells"], d["ms_mean"]) for d in draws]
        more = [(v["proxy_cost_cells"], v["ms_mean"]) for k, v in res.items() if k.endswith("p8") and "proxy_cost_cells" in v]
        res["proxy_cost_against_time_p8"] = {"pearson_r_random_draws": pearson(*zip(*pts)), "n_random_draws": len(pts),
                                             "pearson_r_all_p8_plans": pearson(*zip(*(pts + more))), "n_all": len(pts) + len(more)}
    elif args.case == "exchange":
        # Section 5: the exchange that links the down projection of the 7B block, compiled through its join with the contracted
        # index cut four ways (copy c of the one output block on GPU c), to a consumer cut into four row intervals (one function
        # spec per GPU: a reduce-scatter) or to four function specs that all consume the whole tensor (an all-reduce, rows cut
        # into four atoms by giving the producer four row blocks). Per case: the simulator's completion time of the naive and
        # of the synthesised program on the nominal NVSwitch model of this part, and the SAME program executed on this one GPU
        # (sites = regions of its memory) beside the fused aggregating relayout.
        from paper_2609_03905_b200 import exprog as X
        hb = lambda nbytes, t: {**t, "GBps": nbytes / (t["ms_mean"] * 1e-3) / 1e9, "frac_of_measured_hbm": nbytes / (t["ms_mean"] * 1e-3) / 1e9 / peaks["hbm_gbs"]}
        T, d, m = 16384, 4096, 4
        mach = X.ja_machine_preset("hgx_b200")
        for tag, ps, cs, specs in (("reduce_scatter", [[0, T], [0, d]], [ES(T, 4), [0, d]], [0, 1, 2, 3]),
                                   ("all_reduce", [ES(T, 4), [0, d]], [[0, T], [0, d]], [0, 0, 0, 0])):
            npb = (len(ps[0]) - 1) * (len(ps[1]) - 1)
            copy_site = [c for _ in range(npb) for c in range(m)]
            P = ja.partial_relation(m, [T, d], ps, bf)
            P.payload.normal_(0.0, 1.0)
            y = ja.Relation([T, d], cs, bf)
            for body in ("naive", "best"):
                h = X.ExchangeProgram(handle=X.ja_exprog_preamble(ps, cs, m, copy_site, specs, 2))
                sim = X.ja_exprog_place(h.handle, mach, body)
                if body == "best":
                    sim = X.ja_exprog_synthesize(h.handle, mach, 2, 8)
                stats = h.execute(P, copy_site, specs, "sum", y)
                t = timeit(lambda r: h.execute(P, copy_site, specs, "sum", y), reps, True)
                acts = X.ja_exprog_get_actions(h.handle)
                # HBM traffic on this GPU: decompose reads and writes every copy once, recompose the tensor once, a transfer reads
                # and writes its atom, an aggregation reads its parts and writes one atom
                nbytes = 2.0 * m * T * d * 2 + 2.0 * T * d * 2 + 2.0 * stats["transfer_bytes"] + stats["aggregation_bytes"]
                # the same program as an exchange plan: buffers and tables resident, one stream per site (dataflow), and the
                # plan's run captured into a CUDA graph and replayed
                plan = X.ExchangePlan(h, P, copy_site, specs, "sum", y)
                tp = timeit(lambda r: plan.run(), reps, True)
                tg = timeit_graph(lambda r: plan.run(), reps, True)
                plan.close()
                # every site on a device label of its own (the labels wrap around on one GPU): the paths a plan over several devices
                # takes -- atoms leave the relations' device through a staging area, aggregates come back before recompose
                staged = X.ExchangePlan(h, P, copy_site, specs, "sum", y, site_device=[s + 1 for s in range(4)])
                ts = timeit_graph(lambda r: staged.run(), reps, True)
                staged.close()
                res["%s_%s" % (tag, "synthesised" if body == "best" else body)] = {
                    **hb(nbytes, t), "plan_dataflow_ms": tp["ms_mean"], "plan_graph_replay_ms": tg["ms_mean"],
                    "plan_graph_replay_frac_of_measured_hbm": nbytes / (tg["ms_mean"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
                    "plan_all_sites_staged_graph_replay_ms": ts["ms_mean"],
                    "simulated_ms_hgx_b200_nominal": sim, "actions": len(acts), "aggregations": stats["aggregations"],
                    "transfers": stats["transfers"], "transfer_MB": stats["transfer_bytes"] / 1e6, "scratch_MB": stats["scratch_bytes"] / 1e6}
            res["%s_fused_aggregating_relayout" % tag] = hb((m + 1.0) * T * d * 2, timeit(lambda r: ja.repartition_agg(P, "sum", y), reps, True))
            del P, y
        # cpu_baseline leg of this case: the oracle's executor beside it, on the host cores, on one sixteenth of the rows (the programs and their traffic per
        # byte of tensor are the same at that size): the naive reduce-scatter program, fp64 sums, one rounding to bf16 per aggregate
        import time
        import numpy as np
        from oracle import exprog as OE
        Ts = T // 16
        ps, cs, specs = [[0, Ts], [0, d]], [ES(Ts, 4), [0, d]], [0, 1, 2, 3]
        pre = OE.preamble([Ts, d], ps, {(0, c): c for c in range(m)}, cs, specs, 2)
        q = OE.naive_body(OE.bind(pre, {"S%d" % (i + 1): (i,) for i in range(4)}))
        Ph = np.random.default_rng(0).standard_normal((m, Ts, d))
        t0 = time.perf_counter()
        OE.exchange(q, Ph, ps, cs, specs, "sum", "bf16")
        dt = time.perf_counter() - t0
        res["cpu_baseline_oracle_reduce_scatter_naive"] = {"kind": "oracle", "seconds": dt, "rows": Ts, "GBps_of_bf16_tensor_traffic": (2.82e9 / 16) / dt / 1e9,
                                                      "note": "oracle/exprog.py executor, numpy fp64, 1/16 of the rows"}
    elif args.case == "chains":
        # Section 6, second workload: five fixed matrix chains, each parenthesization executed as a sequence of matmul
        # join-aggs (every intermediate stored once, in bf16); operands N(0, 1/rows) so that magnitudes stay O(1)
        def right(lo, hi):   # M_lo (M_lo+1 (... M_hi))
            return lo if lo == hi else (lo, right(lo + 1, hi))

        chains = {
            "A": ([10240] + [16384, 6144] * 4 + [10240], ((0, 1), (((2, 3), ((4, 5), (6, 7))), 8))),
            "B": ([9216, 20480, 5120, 20480, 5120, 9216], ((0, 1), ((2, 3), 4))),
            "C": ([10240, 12288, 32768, 2048], (0, (1, 2))),
            "D": ([24576, 1536] + [20480] * 6 + [1536, 24576], (0, (right(1, 7), 8))),
            "E": ([49152, 1024] + [20480] * 10 + [1024, 49152], (0, (right(1, 11), 12))),
        }
        blk = lambda n: ES(n, n // 512)

        for name, (dims, tree) in chains.items():
            mats = [rel((dims[i], dims[i + 1]), [blk(dims[i]), blk(dims[i + 1])], std=dims[i] ** -0.5) for i in range(len(dims) - 1)]
            steps, flops = [], [0.0]

            def build(t):   # allocates the intermediates and the specs once; returns (relation, rows, cols)
                if isinstance(t, int):
                    return mats[t], dims[t], dims[t + 1]
                (A, m, j), (Bm, j2, n) = build(t[0]), build(t[1])
                out = ja.Relation([m, n], [blk(m), blk(n)], bf)
                steps.append((ja.Spec("ij,jk->ik", {"i": blk(m), "j": blk(j), "k": blk(n)}), A, Bm, out))
                flops[0] += 2.0 * m * j * n
                return out, m, n

            build(tree)

            def run(r):
                for sp, A, Bm, out in steps:
                    sp.execute([A, Bm], out)
            t = timeit(run, reps, True)
            res["chain_" + name] = {**t, "multiplies": len(steps), "TFLOPs": flops[0] / (t["ms_mean"] * 1e-3) / 1e12,
                                    "frac_of_burst_bf16_peak": flops[0] / (t["ms_mean"] * 1e-3) / 1e12 / peaks["bf16"],
                                    "mean_multiply_vs_8192_cubed": flops[0] / 2 / len(steps) / 8192.0 ** 3}
            del mats, steps
            torch.cuda.empty_cache()
    assert ja.ja_stream_status(stream.cuda_stream) == 0
    del flush, clean
    torch.cuda.empty_cache()
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--plan", choices=["seq", "head", "mixed"], default="mixed",
                    help="hand decomposition of the block: mixed (default) = tokens x 8 column blocks everywhere, attention over 8 blocks of 4 heads, no "
                         "relayout inside the block; seq = the same with attention over 32 single heads (4 relayouts); head = 32 column blocks")
    ap.add_argument("--shape", choices=list(SHAPES), default="7b")
    ap.add_argument("--impl", choices=["ja", "reference"], default="ja")
    ap.add_argument("--ref-rows", type=int, default=16)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the kernels of configurations 1-4 after the headline region")
    ap.add_argument("--config-reps", type=int, default=20, help="timed launches per kernel of configurations 1-4")
    ap.add_argument("--dtype", choices=["bf16", "f16"], default="bf16",
                    help="cell type of the block's relations (--case block): bf16 as the benchmark configurations state, or f16, the paper's precision")
    ap.add_argument("--unfused", action="store_true", help="run every join-agg of the block as its own launch (no fused chains)")
    ap.add_argument("--case", choices=["block", "cfg1", "cfg2", "cfg3", "cfg4", "gqa", "agg", "opt", "optblock", "chains", "exchange", "physical"], default="block",
                    help="block = the headline step; cfgN = the kernels of benchmark configuration N in isolation; "
                         "gqa = grouped-query attention over packed sequences; agg = join-only matmul + aggregating relayout; "
                         "opt = logical optimizer's plan for the MLP tree against hand plans; optblock = the optimizer's plans for the whole "
                         "7B block against the hand decompositions; chains = the five matrix chains; exchange = exchange programs for a "
                         "reduce-scatter and an all-reduce of the down projection's partial copies, simulated and executed on this GPU; "
                         "physical = naive against optimised exchange programs for the block and chains A, B on the simulator (host only)")
    args = ap.parse_args()
    shape = SHAPES[args.shape]
    if args.case != "block":
        run_case(args)
    elif args.impl == "reference":
        args.steps_ref, args.warmup_ref = args.steps, args.warmup
        run_reference(args, shape)
    else:
        run_gpu(args, shape)


if __name__ == "__main__":
    main()
