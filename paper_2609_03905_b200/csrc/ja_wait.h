// The bounded wait every kernel of libja uses for its mbarrier phases, written once for device and host.
//
//   try_wait()  true when the awaited phase has completed
//   now_ns()    a monotonic clock in nanoseconds
//   aborted()   true when another role of the same CTA has already given up
//   fail()      called exactly once by the waiter whose limit ran out (records the error, raises the abort flag)
//
// Returns true when the phase completed, false when the wait was abandoned. The clock and the abort flag are read on
// every 64th poll only, so a satisfied wait costs one or two polls and nothing else.
#pragma once

#include <stdint.h>

#if defined(__CUDACC__)
#define JA_HD __host__ __device__ __forceinline__
#else
#define JA_HD inline
#endif

template <class TryWait, class Clock, class Aborted, class Fail>
JA_HD bool ja_bounded_wait(TryWait try_wait, Clock now_ns, Aborted aborted, Fail fail, uint64_t cap_ns) {
    if (try_wait()) return true;
    const uint64_t t0 = now_ns();
    for (uint32_t it = 0;; ++it) {
        if (try_wait()) return true;
        if ((it & 63) == 63) {
            if (aborted()) return false;
            if (now_ns() - t0 > cap_ns) {
                fail();
                return false;
            }
        }
    }
}
