// Host test of the launchers' per-device memory (csrc/launch_cache.hpp): entries are looked up by
// (kernel, device, shared-memory size); a value computed for one device is never handed to another,
// a failing query is not remembered, and concurrent callers see one query per key.
#include <atomic>
#include <cstdio>
#include <thread>
#include <vector>

#include "launch_cache.hpp"

static int fail(const char *what)
{
    std::printf("FAIL: %s\n", what);
    return 1;
}

int main()
{
    daf::LaunchCache cache;
    int kernel_a = 0, kernel_b = 0;                               // stand-ins for two kernels' addresses
    std::atomic<int> queries{0};
    auto query_for = [&](int device) {
        return [&, device](int *value) {
            queries++;
            *value = 100 * (device + 1);                          // "CTAs that fit device `device`"
            return 0;
        };
    };
    int v = 0;
    // two made-up devices: each gets its own entry and its own query
    if (cache.get(&kernel_a, 0, 0, &v, query_for(0)) != 0 || v != 100) return fail("device 0, first request");
    if (cache.get(&kernel_a, 1, 0, &v, query_for(1)) != 0 || v != 200) return fail("device 1 must not see device 0's entry");
    if (queries != 2) return fail("one query per device");
    if (cache.get(&kernel_a, 0, 0, &v, query_for(0)) != 0 || v != 100 || queries != 2) return fail("device 0 again: remembered");
    if (cache.get(&kernel_a, 1, 0, &v, query_for(1)) != 0 || v != 200 || queries != 2) return fail("device 1 again: remembered");
    // another kernel, another shared-memory size: separate entries
    if (cache.get(&kernel_b, 0, 0, &v, query_for(0)) != 0 || queries != 3) return fail("second kernel has its own entry");
    if (cache.get(&kernel_a, 0, 90000, &v, query_for(0)) != 0 || queries != 4) return fail("second size has its own entry");
    if (cache.size() != 4) return fail("four entries");
    // a failing query is passed through and not remembered
    if (cache.get(&kernel_b, 5, 0, &v, [](int *) { return 7; }) != 7 || cache.size() != 4) return fail("failed query");
    if (cache.get(&kernel_b, 5, 0, &v, query_for(5)) != 0 || v != 600) return fail("retry after a failed query");
    // concurrent callers: one query per key, everybody gets the value
    const int before = queries;
    std::vector<std::thread> threads;
    std::atomic<int> wrong{0};
    for (int t = 0; t < 8; t++)
        threads.emplace_back([&] {
            for (int device = 10; device < 14; device++) {
                int got = 0;
                if (cache.get(&kernel_a, device, 0, &got, query_for(device)) != 0 || got != 100 * (device + 1)) wrong++;
            }
        });
    for (auto &t : threads) t.join();
    if (wrong != 0 || queries != before + 4) return fail("concurrent callers");
    std::printf("ok\n");
    return 0;
}
