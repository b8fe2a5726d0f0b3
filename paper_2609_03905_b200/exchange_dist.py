"""An exchange program whose sites are processes, one per GPU (Section 5.2): every process walks the SAME firing order
(`ja_exprog_schedule`), launches the local aggregations of the actions it is the source of (`ja_exchange_combine`, the
library's kernel) and posts a point-to-point send or receive for every transfer it takes part in (`torch.distributed`,
NCCL between GPUs).  No collective is involved: an exchange program is its own communication schedule.

This module holds no arithmetic.  `combine` is the library's kernel by default and refuses tensors that are not on a GPU;
the CPU tests of the schedule pass their own stand-in.  Not run on more than one GPU in this repository's test runs.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import exprog as X
from .binding import JA_BF16, JA_F16, JA_F32

_DT = {torch.float32: JA_F32, torch.bfloat16: JA_BF16, torch.float16: JA_F16}


def library_combine(parts, agg: str):
    """out = parts[0] (+) parts[1] (+) ... by the library's kernel on torch's current stream."""
    if not all(p.is_cuda for p in parts):
        raise RuntimeError("the local aggregation of an exchange program runs in the library's CUDA kernel: the atoms must be on a GPU")
    out = torch.empty_like(parts[0])
    nbytes = out.numel() * out.element_size()
    if nbytes % 16:
        raise ValueError("atoms are combined in 16-byte accesses: pad the atom buffers to a multiple of 16 bytes")
    X.ja_exchange_combine([p.data_ptr() for p in parts], out.data_ptr(), nbytes, _DT[out.dtype], agg,
                          torch.cuda.current_stream().cuda_stream)
    return out


def run_site(prog: X.ExchangeProgram, site: int, atoms: dict, agg: str = "sum", combine=None, site_rank=None, group=None,
             new_buffer=None):
    """Runs the part of a bound, valid program that concerns `site`.
    atoms: {atom index (declaration order): tensor} for the atoms IN places at this site.  site_rank maps a site to the
    rank of its process in `group` (default: site numbers are ranks).  new_buffer(aggregate mask) -> empty tensor for an
    aggregate that arrives from another site (default: shaped like this site's first atom, which is right when all atoms
    of the program have one shape, as the atoms of a uniform overlay do).
    Returns {aggregate mask: tensor} of everything materialised at this site, its OUT requirements among them."""
    combine = combine or library_combine
    rank_of = (lambda s: s) if site_rank is None else (lambda s: site_rank[s])
    if new_buffer is None:
        if not atoms:
            raise ValueError("a site that holds no atom needs new_buffer to shape what it receives")
        first = next(iter(atoms.values()))
        new_buffer = lambda mask: torch.empty_like(first)
    acts = X.ja_exprog_get_actions(prog.handle)
    store = {1 << a: t for a, t in atoms.items()}
    pending = {}                     # aggregate mask -> receive still in flight
    others = []                      # sends, and receives of aggregates this site already holds

    def ready(mask):
        w = pending.pop(mask, None)
        if w is not None:
            w.wait()
        return store[mask]

    for k, (idx, parts) in enumerate(X.ja_exprog_schedule(prog.handle)):
        mask, src, dmask = acts[idx]
        dests = [d for d in range(64) if (dmask >> d) & 1]
        if src == site:
            if len(parts) >= 2:
                store[mask] = combine([ready(y) for y in parts], agg)
            buf = ready(mask)
            for d in dests:
                others.append(dist.isend(buf, rank_of(d), group=group, tag=k))
        elif site in dests:
            if mask not in store:
                store[mask] = new_buffer(mask)
                pending[mask] = dist.irecv(store[mask], rank_of(src), group=group, tag=k)
            else:                    # a second delivery of an aggregate that is already here: the sender still sends it
                others.append(dist.irecv(new_buffer(mask), rank_of(src), group=group, tag=k))
    for w in list(pending.values()) + others:
        w.wait()
    return store
