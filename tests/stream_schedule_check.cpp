// Host check of the continuous-batching schedule (csrc/stream_schedule.h) against a simulated device: every
// utterance decodes for its true length (shorter than its forced length when it "emits end-of-sequence"), a slot's
// length becomes visible in the step that finishes it, and the simulated library issues a step only while the host's
// own bounds say that some slot still decodes.  Usage: stream_schedule_check n slots early_stop poll_steps seed
// Prints "ok steps row_steps sum_true_len max_forced sum_forced"; exits non-zero with a message on a violated rule.
#include <cstdio>
#include <cstdlib>
#include <numeric>
#include <random>
#include <vector>

#include "../paper_2503_05931_b200/csrc/stream_schedule.h"

#define REQUIRE(cond, ...) do { if (!(cond)) { std::fprintf(stderr, __VA_ARGS__); std::fprintf(stderr, "\n"); std::exit(1); } } while (0)

struct FakeDevice {
    int n, slots;
    bool early_stop;
    std::vector<int32_t> forced, true_len, order;
    std::vector<int> occupant, t, host_t;          // per slot: utterance, tokens produced, steps the host counted
    std::vector<int32_t> lens;                     // per slot, as the device shows it
    std::vector<int> admitted_at, harvested;       // per utterance
    int next_arrival = 0;
    long long steps_issued = 0;

    int admit(const aed::StreamAdmission *a, int k)
    {
        REQUIRE(k >= 1 && k <= 16, "admit of %d utterances", k);
        for (int i = 0; i < k; ++i) {
            const int s = a[i].slot, u = a[i].utterance;
            REQUIRE(s >= 0 && s < slots && u >= 0 && u < n, "admission out of range");
            REQUIRE(u == order[next_arrival], "utterance %d admitted out of arrival order", u);
            ++next_arrival;
            REQUIRE(admitted_at[u] < 0, "utterance %d admitted twice", u);
            if (occupant[s] >= 0) {
                REQUIRE(t[s] == true_len[occupant[s]], "slot %d reused while utterance %d still decodes", s, occupant[s]);
                REQUIRE(harvested[occupant[s]] == 1, "slot %d reused before utterance %d was collected", s, occupant[s]);
            }
            for (int j = 0; j < i; ++j) REQUIRE(a[j].slot != s, "slot %d twice in one admission", s);
            occupant[s] = u; t[s] = 0; host_t[s] = 0; lens[s] = 0;
            admitted_at[u] = static_cast<int>(steps_issued);
        }
        return 0;
    }
    int steps(int want, int *done)
    {
        REQUIRE(want >= 1, "asked for %d steps", want);
        *done = 0;
        for (int k = 0; k < want; ++k) {
            bool host_alive = false;
            for (int s = 0; s < slots; ++s) host_alive |= occupant[s] >= 0 && host_t[s] < forced[occupant[s]];
            if (!host_alive) break;
            for (int s = 0; s < slots; ++s) {
                if (occupant[s] < 0) continue;
                if (host_t[s] < forced[occupant[s]]) ++host_t[s];
                if (t[s] < true_len[occupant[s]]) {
                    if (++t[s] == true_len[occupant[s]]) lens[s] = t[s];
                }
            }
            ++steps_issued;
            ++*done;
        }
        return 0;
    }
    int read_lens(int32_t *out)
    {
        REQUIRE(early_stop, "lengths read back although they are known in advance");
        for (int s = 0; s < slots; ++s) out[s] = lens[s];
        return 0;
    }
    int harvest(int s, int u)
    {
        REQUIRE(occupant[s] == u, "slot %d collected as utterance %d but holds %d", s, u, occupant[s]);
        REQUIRE(t[s] == true_len[u], "utterance %d collected after %d of %d tokens", u, t[s], true_len[u]);
        REQUIRE(harvested[u] == 0, "utterance %d collected twice", u);
        harvested[u] = 1;
        return 0;
    }
};

int main(int argc, char **argv)
{
    REQUIRE(argc == 6, "usage: n slots early_stop poll_steps seed");
    const int n = std::atoi(argv[1]), slots = std::atoi(argv[2]), poll = std::atoi(argv[4]);
    const bool early = std::atoi(argv[3]) != 0;
    std::mt19937 rng(static_cast<unsigned>(std::atoi(argv[5])));
    FakeDevice dev;
    dev.n = n; dev.slots = slots; dev.early_stop = early;
    dev.forced.resize(n); dev.true_len.resize(n); dev.order.resize(n);
    for (int u = 0; u < n; ++u) {
        dev.forced[u] = 1 + static_cast<int>(rng() % 40);
        dev.true_len[u] = early && rng() % 2 ? 1 + static_cast<int>(rng() % dev.forced[u]) : dev.forced[u];
    }
    std::iota(dev.order.begin(), dev.order.end(), 0);
    for (int i = n - 1; i > 0; --i) std::swap(dev.order[i], dev.order[rng() % (i + 1)]);
    dev.occupant.assign(slots, -1); dev.t.assign(slots, 0); dev.host_t.assign(slots, 0); dev.lens.assign(slots, 0);
    dev.admitted_at.assign(n, -1); dev.harvested.assign(n, 0);
    aed::StreamTotals tot;
    const int rc = aed::run_stream_schedule(n, slots, dev.order.data(), dev.forced.data(), early, poll, 16, dev, &tot);
    REQUIRE(rc == 0, "schedule returned %d", rc);
    for (int u = 0; u < n; ++u) REQUIRE(dev.admitted_at[u] >= 0 && dev.harvested[u] == 1, "utterance %d was lost", u);
    REQUIRE(tot.steps == dev.steps_issued, "the schedule counted %lld steps, the device ran %lld", tot.steps, dev.steps_issued);
    long long sum_true = 0, sum_forced = 0;
    int max_forced = 0;
    for (int u = 0; u < n; ++u) { sum_true += dev.true_len[u]; sum_forced += dev.forced[u]; max_forced = std::max(max_forced, dev.forced[u]); }
    std::printf("ok %lld %lld %lld %d %lld\n", tot.steps, tot.row_steps, sum_true, max_forced, sum_forced);
    return 0;
}
