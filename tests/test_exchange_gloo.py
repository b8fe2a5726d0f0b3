"""The multi-process driver of exchange programs (paper_2609_03905_b200/exchange_dist.py) under `gloo`, one process per
site on CPU: every rank walks the library's firing order, posts its sends and receives, and combines locally with a torch
stand-in for the library's kernel (which needs a GPU); the aggregates each site ends with are compared with the oracle's
executor.  What is checked is the schedule and the pairing of the transfers, not arithmetic."""
import json
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import paper_2609_03905_b200  # noqa: F401  (loads, and if need be builds, the library once here, before the ranks start)
from oracle import exprog as E

G = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "exprog_examples.json")))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _torch_combine(parts, agg):
    acc = parts[0].clone()
    for p in parts[1:]:
        acc = acc + p if agg == "sum" else torch.maximum(acc, p)
    return acc


def _worker(rank, world, port, text, agg, q):
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from paper_2609_03905_b200 import exchange_dist, exprog as X
        prog = X.ExchangeProgram(text)
        sites = X.ja_exprog_get_atoms(prog.handle)
        gen = torch.Generator().manual_seed(1234)
        values = [torch.randn(8, 6, generator=gen, dtype=torch.float64) for _ in sites]      # the same on every rank
        mine = {a: values[a].clone() for a, (s, _) in enumerate(sites) if s == rank}
        with pytest.raises(RuntimeError):                                                     # the product's combine refuses CPU tensors
            exchange_dist.library_combine([values[0], values[1]], "sum")
        store = exchange_dist.run_site(prog, rank, mine, agg, combine=_torch_combine)
        q.put((rank, {int(k): v.numpy() for k, v in store.items()}))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("name,world,agg", [("swap", 2, "sum"), ("doubling", 4, "sum"), ("doubling", 4, "max")])
def test_sites_as_processes(name, world, agg):
    text = G[name]["program"]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, text, agg, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = dict(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    prog = E.parse(text)
    gen = torch.Generator().manual_seed(1234)
    values = {a: torch.randn(8, 6, generator=gen, dtype=torch.float64).numpy() for a in prog.atoms}
    want = E.execute(prog, values, agg)
    order = {a: i for i, a in enumerate(prog.atoms)}
    for (x, s), v in want.items():
        mask = sum(1 << order[a] for a in x)
        assert mask in got[s], (sorted(x), s)
        assert np.array_equal(got[s][mask], v)                    # same parts, same order, fp64 on both sides
    for x, s in E.requirements(prog):
        assert sum(1 << order[a] for a in x) in got[s]
