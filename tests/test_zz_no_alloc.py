"""ja_repartition_noalloc: the relayout entry point for callers that cannot allocate (memory handed out once at
start-up, latency-critical loops, allocation-auditing harnesses). It must move exactly the bytes ja_repartition
moves. Collected last on purpose: if it fails, every other test has already run.

The check: the same relayouts through both entry points, bit-exact, on two calls in a row (the second call reuses
the library's fixed plan table with a different, smaller plan, so stale entries from the first call must not
matter), with torch's allocator watched to show the call itself allocates nothing through it."""
import numpy as np
import pytest
import torch

import paper_2609_03905_b200 as ja
from gpu_util import download, np_bits

pytestmark = pytest.mark.gpu
ES = ja.equal_splits
BF, F32 = torch.bfloat16, torch.float32
DT = {BF: ja.JA_BF16, F32: ja.JA_F32}


def _both_ways(ext, s_sp, d_sp, dtype, seed):
    g = torch.Generator(device="cpu").manual_seed(seed)
    src = ja.Relation(ext, s_sp, dtype)
    src.payload.copy_(torch.randn(src.payload.numel(), generator=g).to(dtype))
    want = ja.Relation(ext, d_sp, dtype)
    ja.repartition(src, want)                                   # the existing entry point
    got = ja.Relation(ext, d_sp, dtype)
    got.payload.fill_(float("nan"))
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream().cuda_stream
    before = torch.cuda.memory_stats()["allocation.all.allocated"]
    ja.ja_repartition_noalloc(ext, s_sp, d_sp, DT[dtype], src.payload.data_ptr(), got.payload.data_ptr(), stream)
    after = torch.cuda.memory_stats()["allocation.all.allocated"]
    assert after == before, "the no-allocation entry point allocated through torch"
    # every cell of the tensor, bit for bit (alignment gaps between blocks belong to nobody and are not compared)
    assert np.array_equal(download(got).view(np.uint64), download(want).view(np.uint64))
    assert not np.isnan(download(got)).any()
    assert ja.ja_stream_status(stream) == 0


def test_noalloc_matches_repartition_two_calls_in_a_row():
    # call 1: a large plan (1024 atoms: sequence-blocked -> head-blocked activation relayout)
    _both_ways([4096, 4096], [ES(4096, 32), ES(4096, 8)], [ES(4096, 32), ES(4096, 32)], BF, 1)
    # call 2, immediately after: a small, irregular plan in another dtype and rank
    _both_ways([33, 17, 9], [[0, 33], [0, 5, 17], [0, 9]], [[0, 10, 33], [0, 17], [0, 4, 9]], F32, 2)
    # and once more the first shape in the opposite direction
    _both_ways([4096, 4096], [ES(4096, 32), ES(4096, 32)], [ES(4096, 32), ES(4096, 8)], BF, 3)


def test_noalloc_rejects_plans_beyond_its_fixed_table():
    ext = [1 << 16, 1 << 10]
    s_sp, d_sp = [ES(ext[0], 1), ES(ext[1], 1)], [ES(ext[0], 4096), ES(ext[1], 8)]      # 32768 atoms > 16384 slabs
    buf = torch.zeros(ext[0] * ext[1], dtype=BF, device="cuda")
    out = torch.zeros(ext[0] * ext[1], dtype=BF, device="cuda")
    with pytest.raises(ja.JaError) as e:
        ja.ja_repartition_noalloc(ext, s_sp, d_sp, ja.JA_BF16, buf.data_ptr(), out.data_ptr(), 0)
    assert e.value.status_name == "JA_ERR_UNSUPPORTED"
