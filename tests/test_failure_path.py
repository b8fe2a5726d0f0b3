"""The failure path of libja's device-side waits, exercised without faulting, trapping or hanging anything.

Every kernel waits on its mbarriers through ONE loop (csrc/ja_wait.h): poll; every 64th poll look at the CTA's abort
flag and at the clock; past the limit record JA_ERR_TIMEOUT, raise the flag, give up. The CPU tests run that same loop,
compiled for the host, against a scripted barrier and clock. The GPU test launches a one-CTA test kernel whose barrier
nobody arrives at, with a 1 ms limit: the kernel must return normally, the stream's status word must read JA_ERR_TIMEOUT
once and be clear afterwards, and ordinary launches (the persistent attention kernel, whose work counters the status
call resets) must then pass parity as if nothing had happened. No product kernel is made to stall."""
import numpy as np
import pytest
import torch

import paper_2609_03905_b200 as ja

JA_ERR_TIMEOUT = 11


# ---- the wait loop on the host -------------------------------------------------------------------------------------
def test_wait_succeeds_at_once_without_reading_the_clock():
    polls, ok, recorded, ns = ja.ja_debug_bounded_wait_host(ready_at_poll=1, ns_per_poll=10**9, cap_ns=1)
    assert (polls, ok, recorded) == (1, True, False)


@pytest.mark.parametrize("ready_at", [2, 3, 64, 65, 66, 1000, 4097])
def test_wait_succeeds_when_the_barrier_completes_before_the_limit(ready_at):
    polls, ok, recorded, ns = ja.ja_debug_bounded_wait_host(ready_at, ns_per_poll=100, cap_ns=10**9)
    assert ok and not recorded and polls == ready_at


def test_wait_gives_up_past_the_limit_and_records_it_once():
    # 100 ns per poll, limit 1 ms -> 10 000 polls; the clock is read on every 64th poll of the loop only
    polls, ok, recorded, ns = ja.ja_debug_bounded_wait_host(ready_at_poll=0, ns_per_poll=100, cap_ns=1_000_000)
    assert not ok and recorded
    assert 1_000_000 < ns <= 1_000_000 + 2 * 64 * 100       # past the limit by less than two check periods
    assert (polls - 1) % 64 == 0                            # gave up at a check, not between two


def test_wait_is_never_abandoned_before_the_limit():
    for cap in (6_400, 64_000, 1_000_000):
        polls, ok, recorded, ns = ja.ja_debug_bounded_wait_host(0, 100, cap)
        assert not ok and recorded and ns > cap


def test_a_barrier_that_completes_just_before_the_limit_wins():
    # completes at poll 9 000 = 0.9 ms of a 1 ms limit
    polls, ok, recorded, ns = ja.ja_debug_bounded_wait_host(9_000, 100, 1_000_000)
    assert ok and not recorded and polls == 9_000


def test_wait_follows_the_abort_flag_without_recording_a_second_error():
    # another role of the CTA gives up at poll 500: this waiter leaves at its next check, long before its own limit
    polls, ok, recorded, ns = ja.ja_debug_bounded_wait_host(0, 100, 10**12, abort_at_poll=500)
    assert not ok and not recorded
    assert 500 <= polls <= 500 + 64


def test_switches_reject_unknown_names_and_bad_limits():
    with pytest.raises(ja.JaError):
        ja.ja_debug_set("no_such_switch", 1)
    with pytest.raises(ja.JaError):
        ja.ja_debug_set("wait_cap_ns", 5)
    ja.ja_debug_set("attn_persistent", 0)
    ja.ja_debug_set("attn_persistent", -1)


# ---- on the GPU -----------------------------------------------------------------------------------------------------
@pytest.mark.gpu
def test_expired_wait_is_reported_once_and_the_library_carries_on():
    import synth_inputs as si
    from gpu_util import TOL, download, empty_like_tiling, relfro, upload
    from oracle import blocked, operators
    ES = blocked.equal_splits
    stream = torch.cuda.current_stream().cuda_stream
    assert ja.ja_stream_status(stream) == 0
    ja.ja_debug_set("wait_cap_ns", 1_000_000)                      # 1 ms
    flags = torch.full((2,), 7, dtype=torch.int32, device="cuda")
    ja.ja_debug_wait_timeout(stream, flags.data_ptr())
    other = torch.cuda.Stream()
    assert ja.ja_stream_status(other.cuda_stream) == 0             # another stream's word is untouched
    assert ja.ja_stream_status(stream) == JA_ERR_TIMEOUT           # reported ...
    assert flags.tolist() == [0, 0]                                # ... by the waiter that ran out; the second one saw the flag
    assert ja.ja_stream_status(stream) == 0                        # ... once
    ja.ja_debug_set("wait_cap_ns", 2_000_000_000)
    # an ordinary join-agg afterwards: causal attention in the persistent form (its work counters were reset by the status call)
    ja.ja_debug_set("attn_persistent", 1)
    B, S, H, D = 1, 512, 2, 128
    Q, K, V = (si.normal((B, S, H, D), 0.0, 1.0, torch.bfloat16, 4, o) for o in (41, 42, 43))
    sp = [ES(B, B), ES(S, S // 128), ES(H, H), [0, D]]
    rQ, rK, rV = upload(Q, sp), upload(K, sp), upload(V, sp)
    rO = empty_like_tiling([B, S, H, D], sp, torch.bfloat16, fill=float("nan"))
    spec = ja.Spec("bqhd,bkhd,bkhd->bqhd", {"b": sp[0], "q": sp[1], "h": sp[2], "d": sp[3], "k": sp[1]}, "attention",
                   (1.0 / np.sqrt(D), 1.0), "online_softmax")
    for _ in range(2):
        spec.execute([rQ, rK, rV], rO)
    got = download(rO)
    assert ja.ja_stream_status(stream) == 0
    ref = operators.attention(si.to_f64(Q), si.to_f64(K), si.to_f64(V), True, "bf16")
    assert relfro(got, ref) <= TOL[torch.bfloat16]
