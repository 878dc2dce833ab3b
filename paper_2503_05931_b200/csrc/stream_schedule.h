// Continuous batching: which utterance enters which slot, how many steps to issue before looking again, and when a
// finished utterance's result is collected.  Host-only and free of CUDA: the library instantiates it with operations
// that launch kernels and copies, the CPU tests with a simulated device.
//
// Ops must provide (each returning 0 on success or a negative status that ends the schedule):
//   int admit(const StreamAdmission *adm, int n)   new utterances enter their slots (n <= max_admit)
//   int steps(int want, int *done)                 issue up to `want` greedy steps over the occupied slots
//   int read_lens(int32_t *lens)                   lengths of the slots as of all steps issued so far (0: still
//                                                  decoding); only called when lengths are not known in advance
//   int harvest(int slot, int utterance)           collect the slot's result; ordered after the steps issued so far
//                                                  and before anything a later admit does to the slot
#pragma once
#include <stdint.h>

#include <algorithm>
#include <vector>

namespace aed {

struct StreamAdmission { int slot; int utterance; };

struct StreamTotals { long long steps = 0, row_steps = 0; };

// n utterances with forced lengths max_lens[u] (upper bounds if early_stop) arrive in the order order[0..n) (or
// 0, 1, 2, ... if order is null) and pass through `slots` slots.  Without early stopping the host knows the step in
// which every utterance ends: it issues exactly the steps up to the next departure and never asks the device.  With it,
// it issues poll_steps steps at a time and reads the slots' lengths back.
template <class Ops>
int run_stream_schedule(int n, int slots, const int32_t *order, const int32_t *max_lens, bool early_stop, int poll_steps,
                        int max_admit, Ops &ops, StreamTotals *totals)
{
    std::vector<int> occupant(slots, -1), remaining(slots, 0);
    std::vector<int32_t> lens(slots, 0);
    std::vector<StreamAdmission> batch;
    int next = 0, rc = 0;
    StreamTotals tot;
    auto fill = [&]() -> int {
        batch.clear();
        for (int s = 0; s < slots && next < n; ++s) {
            if (occupant[s] >= 0) continue;
            const int u = order ? order[next] : next;
            ++next;
            batch.push_back(StreamAdmission{s, u});
            occupant[s] = u;
            remaining[s] = max_lens[u];
            if (static_cast<int>(batch.size()) == max_admit) {
                if ((rc = ops.admit(batch.data(), max_admit)) < 0) return rc;
                batch.clear();
            }
        }
        if (!batch.empty() && (rc = ops.admit(batch.data(), static_cast<int>(batch.size()))) < 0) return rc;
        return 0;
    };
    if ((rc = fill()) < 0) return rc;
    for (;;) {
        int busy = 0, lo = 1 << 30, hi = 0;
        for (int s = 0; s < slots; ++s)
            if (occupant[s] >= 0) { ++busy; lo = std::min(lo, remaining[s]); hi = std::max(hi, remaining[s]); }
        if (!busy) break;
        const int want = early_stop ? std::min(poll_steps, hi) : lo;
        int done = 0;
        if ((rc = ops.steps(want, &done)) < 0) return rc;
        tot.steps += done;
        for (int s = 0; s < slots; ++s)
            if (occupant[s] >= 0) { tot.row_steps += std::min(done, remaining[s]); remaining[s] = std::max(remaining[s] - done, 0); }
        if (early_stop && (rc = ops.read_lens(lens.data())) < 0) return rc;
        for (int s = 0; s < slots; ++s)
            if (occupant[s] >= 0 && (remaining[s] == 0 || (early_stop && lens[s] > 0))) {
                if ((rc = ops.harvest(s, occupant[s])) < 0) return rc;
                occupant[s] = -1;
            }
        if ((rc = fill()) < 0) return rc;
        if (done == 0 && next >= n) break;
    }
    if (totals) *totals = tot;
    return 0;
}

}  // namespace aed
