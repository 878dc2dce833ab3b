// The one polling loop behind every wait in the device code (mbarrier phases, arrival counters of other thread
// blocks).  A wait never spins for ever: it ends when the condition holds, when another party of the same block
// has already given up (the abort word is set), or when `limit` ticks of the caller's clock have passed, in which
// case it sets the abort word itself.  The caller then stops issuing work, lets its own copies land, frees what
// it holds and returns, and the host later reads the sticky error word as AED_ERR_TIMEOUT.
//
// The loop is plain C++ with the condition and the clock passed in, so the same source compiles for the host
// (steady clock, threads instead of warps), which is how its give-up path is tested without a GPU.
#pragma once

#if defined(__CUDACC__)
#define AED_WAIT_FN __device__ __forceinline__
#else
#define AED_WAIT_FN inline
#endif

namespace aed {

template <class Ready, class Now>
AED_WAIT_FN bool bounded_poll(Ready ready, Now now, long long limit, volatile int *abort_flag)
{
    if (ready()) return true;
    const long long start = now();
    while (true) {
        if (ready()) return true;
        if (*abort_flag) return false;
        if (now() - start > limit) { *abort_flag = 1; return false; }
    }
}

}  // namespace aed
