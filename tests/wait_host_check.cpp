// Host build of the device code's bounded wait: two threads stand in for two warps of a block.
//   case "complete": both parties arrive at a counter that expects two arrivals -> both waits return true.
//   case "withheld": one arrival never comes -> the first waiter runs out of time, returns false and raises the
//                    abort word; the second waiter sees the abort word and returns false without waiting out its
//                    own limit.
// Prints one line per case: <case> <result of waiter 0> <result of waiter 1> <abort word> <elapsed ms of waiter 1>.
#include <atomic>
#include <chrono>
#include <cstdio>
#include <thread>

#include "../paper_2503_05931_b200/csrc/bounded_wait.h"

static long long now_us()
{
    return std::chrono::duration_cast<std::chrono::microseconds>(std::chrono::steady_clock::now().time_since_epoch()).count();
}

static void run_case(const char *name, bool second_arrives)
{
    std::atomic<int> arrivals{0};
    volatile int abort_word = 0;
    bool r0 = true, r1 = true;
    long long t1 = 0;
    auto ready = [&] { return arrivals.load(std::memory_order_acquire) >= 2; };
    std::thread a([&] {
        arrivals.fetch_add(1, std::memory_order_release);
        r0 = aed::bounded_poll(ready, now_us, 50 * 1000, &abort_word);          // 50 ms
    });
    std::thread b([&] {
        if (second_arrives) arrivals.fetch_add(1, std::memory_order_release);
        const long long s = now_us();
        r1 = aed::bounded_poll(ready, now_us, 5 * 1000 * 1000, &abort_word);    // 5 s: must end through the abort word
        t1 = now_us() - s;
    });
    a.join();
    b.join();
    std::printf("%s %d %d %d %lld\n", name, (int)r0, (int)r1, (int)abort_word, t1 / 1000);
}

int main()
{
    run_case("complete", true);
    run_case("withheld", false);
    return 0;
}
