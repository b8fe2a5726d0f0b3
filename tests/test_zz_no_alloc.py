"""ja_repartition_noalloc: the relayout entry point for callers that cannot allocate (memory handed out once at
start-up, loops that must never take cudaMalloc's device synchronisation, allocation-auditing harnesses). It must move
exactly the bytes ja_repartition moves. Collected last on purpose: if it fails, every other test has already run.

The checks: the same relayouts through both entry points AND through the CPU oracle's relayout, bit for bit, on calls
in a row (a later call reuses the library's fixed plan table with a different, smaller plan, so stale entries of an
earlier call must not matter); the device's free memory, as the driver reports it, is the same before and after a call
-- that sees an allocation made inside the library, which torch's own counters would not; the limits of the fixed
tables are refused with a clear error; a call on a stream that is being captured is refused."""
import numpy as np
import pytest
import torch

import paper_2609_03905_b200 as ja
from gpu_util import download_bits, from_bits, np_bits
from oracle import blocked

pytestmark = pytest.mark.gpu
ES = ja.equal_splits
BF, F32 = torch.bfloat16, torch.float32
DT = {BF: ja.JA_BF16, F32: ja.JA_F32}


def _filled(ext, sp, dtype, seed):
    g = torch.Generator(device="cpu").manual_seed(seed)
    r = ja.Relation(ext, sp, dtype)
    r.payload.copy_(torch.randn(r.payload.numel(), generator=g).to(dtype))
    return r


def _both_ways(ext, s_sp, d_sp, dtype, seed, check_free_memory=True):
    src = _filled(ext, s_sp, dtype, seed)
    want = ja.Relation(ext, d_sp, dtype)
    ja.repartition(src, want)                                   # the existing entry point
    got = ja.Relation(ext, d_sp, dtype)
    got.payload.fill_(float("nan"))
    stream = torch.cuda.current_stream().cuda_stream
    if check_free_memory:
        # the same call once unmeasured: the first launch of a kernel variant in a process makes the driver load its module,
        # which may take device memory of the driver's own (with many kernels loaded before this test, a fresh 2 MiB granule)
        ja.ja_repartition_noalloc(ext, s_sp, d_sp, DT[dtype], src.payload.data_ptr(), got.payload.data_ptr(), stream)
        got.payload.fill_(float("nan"))
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    ja.ja_repartition_noalloc(ext, s_sp, d_sp, DT[dtype], src.payload.data_ptr(), got.payload.data_ptr(), stream)
    torch.cuda.synchronize()
    free_after = torch.cuda.mem_get_info()[0]
    if check_free_memory:
        assert free_after == free_before, "the no-allocation entry point changed the device's free memory"
    # every cell of the tensor, bit for bit, against the other entry point and against the oracle's relayout of the
    # same payload (alignment gaps between blocks belong to nobody and are not compared)
    got_cells = blocked.unpack(download_bits(got), ext, d_sp)
    assert np.array_equal(got_cells, blocked.unpack(download_bits(want), ext, d_sp))
    ref_payload = blocked.repartition(np_bits(src.payload.cpu()), ext, s_sp, d_sp)
    assert np.array_equal(got_cells, blocked.unpack(ref_payload, ext, d_sp))
    assert not torch.isnan(from_bits(got_cells, dtype).float()).any()
    assert ja.ja_stream_status(stream) == 0


def test_noalloc_matches_repartition_and_oracle_on_calls_in_a_row():
    # warm-up call: the first call on a device resolves the plan table's address (and loads the kernel's module), which
    # may itself change what the driver reports as free
    _both_ways([64, 64], [ES(64, 2), ES(64, 2)], [ES(64, 4), ES(64, 1)], BF, 9, check_free_memory=False)
    # call 1: a large plan (1024 atoms: sequence-blocked -> head-blocked activation relayout)
    _both_ways([4096, 4096], [ES(4096, 32), ES(4096, 8)], [ES(4096, 32), ES(4096, 32)], BF, 1)
    # call 2, immediately after: a small, irregular plan in another dtype and rank
    _both_ways([33, 17, 9], [[0, 33], [0, 5, 17], [0, 9]], [[0, 10, 33], [0, 17], [0, 4, 9]], F32, 2)
    # and once more the first shape in the opposite direction
    _both_ways([4096, 4096], [ES(4096, 32), ES(4096, 32)], [ES(4096, 32), ES(4096, 8)], BF, 3)


def test_the_free_memory_probe_does_see_an_allocation_inside_the_library():
    """Sanity arm of the check above: the first ja_repartition between two fresh relations builds its copy plan in a
    cudaMalloc'ed table (here 131072 slabs, 5 MB), and the same probe moves."""
    ext = [1 << 17, 4, 8]
    s_sp, d_sp = [[0, ext[0]], [0, 4], [0, 8]], [[0, ext[0]], [0, 2, 4], [0, 8]]
    src, dst = _filled(ext, s_sp, BF, 5), ja.Relation(ext, d_sp, BF)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    ja.repartition(src, dst)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] < free_before


def _refused(ext, s_sp, d_sp, match):
    n = int(np.prod(ext))
    buf = torch.zeros(n + 4096 * 64, dtype=BF, device="cuda")
    out = torch.zeros(n + 4096 * 64, dtype=BF, device="cuda")
    with pytest.raises(ja.JaError, match=match) as e:
        ja.ja_repartition_noalloc(ext, s_sp, d_sp, ja.JA_BF16, buf.data_ptr(), out.data_ptr(), 0)
    assert e.value.status_name == "JA_ERR_UNSUPPORTED"


def test_noalloc_refuses_what_its_fixed_tables_cannot_hold():
    one = lambda ext: [[0, e] for e in ext]
    # more than 16384 copy slabs: one block on both sides, but 20000 outer coordinates = 20000 slabs
    _refused([20000, 4, 8], one([20000, 4, 8]), one([20000, 4, 8]), "copy slabs")
    # more than 4096 blocks in a tiling (split lists and slab count within their limits)
    _refused([100, 100], [ES(100, 100), ES(100, 100)], one([100, 100]), "4096 blocks")
    # more than 1024 overlay split points along one dimension
    _refused([1 << 16, 8], [ES(1 << 16, 4096), [0, 8]], one([1 << 16, 8]), "split points")


def test_noalloc_takes_a_plan_that_fills_its_table_exactly():
    ext = [16384, 4, 8]                     # 16384 outer coordinates = 16384 slabs, the table's size
    _both_ways(ext, [[0, e] for e in ext], [[0, e] for e in ext], BF, 7)


def test_noalloc_refuses_a_stream_that_is_being_captured():
    ext, s_sp, d_sp = [256, 256], [ES(256, 2), ES(256, 2)], [ES(256, 4), ES(256, 1)]
    src, dst = _filled(ext, s_sp, BF, 11), ja.Relation(ext, d_sp, BF)
    ja.ja_repartition_noalloc(ext, s_sp, d_sp, ja.JA_BF16, src.payload.data_ptr(), dst.payload.data_ptr(),
                              torch.cuda.current_stream().cuda_stream)          # first call outside any capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    marker = torch.zeros(1, device="cuda")
    with torch.cuda.graph(g):
        marker.add_(1.0)                                                        # so that the capture is not empty
        with pytest.raises(ja.JaError, match="captured") as e:
            ja.ja_repartition_noalloc(ext, s_sp, d_sp, ja.JA_BF16, src.payload.data_ptr(), dst.payload.data_ptr(),
                                      torch.cuda.current_stream().cuda_stream)
        assert e.value.status_name == "JA_ERR_UNSUPPORTED"
    g.replay()
    torch.cuda.synchronize()
    assert marker.item() == 1.0                                                 # the refused call recorded nothing
