// Host-side page pool for packed activation buffers: bookkeeping only.
//
// The paper keeps compressed activations in one preallocated contiguous block that is handed
// out in pages with a first-fit search (Sec. 3.4.2), and tags every stored activation with an
// importance so that the least valuable one is dropped first when room is needed (Sec. 3.4.3).
// This stand-in keeps that behaviour -- arena, fixed-size pages, first-fit runs, eviction by
// importance per byte -- with an ordered map instead of the paper's dual red-black trees and
// without the time budget.  It never touches the arena's memory and stays off the GPU path.
#include <map>
#include <new>
#include <vector>

#include "../../include/daf.h"

struct daf_pool {
    uint64_t arena_bytes = 0, page_bytes = 0, pages_total = 0, pages_used = 0, bytes_requested = 0, evictions = 0;
    uint64_t next_handle = 1;
    std::vector<uint8_t> used;                       // one flag per page
    struct Alloc {
        uint64_t first_page, n_pages, bytes;
        double importance;
    };
    std::map<uint64_t, Alloc> live;                  // handle -> allocation
    std::multimap<double, uint64_t> by_value;        // importance per byte -> handle (ascending)
};

extern "C" daf_pool *daf_pool_create(uint64_t arena_bytes, uint64_t page_bytes)
{
    if (page_bytes == 0) page_bytes = 65536;
    if (arena_bytes < page_bytes) return nullptr;
    daf_pool *p = new (std::nothrow) daf_pool();
    if (!p) return nullptr;
    p->arena_bytes = arena_bytes;
    p->page_bytes = page_bytes;
    p->pages_total = arena_bytes / page_bytes;
    p->used.assign(p->pages_total, 0);
    return p;
}

extern "C" void daf_pool_destroy(daf_pool *pool) { delete pool; }

extern "C" uint64_t daf_pool_alloc(daf_pool *pool, uint64_t bytes, double importance, uint64_t *offset)
{
    if (!pool || bytes == 0) return 0;
    const uint64_t need = (bytes + pool->page_bytes - 1) / pool->page_bytes;
    uint64_t run = 0;
    for (uint64_t i = 0; i < pool->pages_total; i++) {          // first fit: lowest run of `need` free pages
        run = pool->used[i] ? 0 : run + 1;
        if (run == need) {
            const uint64_t first = i + 1 - need;
            for (uint64_t j = first; j <= i; j++) pool->used[j] = 1;
            const uint64_t h = pool->next_handle++;
            pool->live[h] = daf_pool::Alloc{first, need, bytes, importance};
            pool->by_value.emplace(importance / (double)bytes, h);
            pool->pages_used += need;
            pool->bytes_requested += bytes;
            if (offset) *offset = first * pool->page_bytes;
            return h;
        }
    }
    return 0;
}

static void release(daf_pool *pool, uint64_t handle, const daf_pool::Alloc &a)
{
    for (uint64_t j = a.first_page; j < a.first_page + a.n_pages; j++) pool->used[j] = 0;
    pool->pages_used -= a.n_pages;
    pool->bytes_requested -= a.bytes;
    auto range = pool->by_value.equal_range(a.importance / (double)a.bytes);
    for (auto it = range.first; it != range.second; ++it)
        if (it->second == handle) {
            pool->by_value.erase(it);
            break;
        }
    pool->live.erase(handle);
}

extern "C" daf_status daf_pool_free(daf_pool *pool, uint64_t handle)
{
    if (!pool) return DAF_ERR_INVALID_ARG;
    auto it = pool->live.find(handle);
    if (it == pool->live.end()) return DAF_ERR_INVALID_ARG;
    const daf_pool::Alloc a = it->second;
    release(pool, handle, a);
    return DAF_OK;
}

extern "C" uint64_t daf_pool_evict_lowest(daf_pool *pool)
{
    if (!pool || pool->by_value.empty()) return 0;
    const uint64_t h = pool->by_value.begin()->second;
    const daf_pool::Alloc a = pool->live[h];
    release(pool, h, a);
    pool->evictions++;
    return h;
}

extern "C" daf_status daf_pool_get_stats(const daf_pool *pool, daf_pool_stats *stats)
{
    if (!pool || !stats) return DAF_ERR_INVALID_ARG;
    uint64_t best = 0, run = 0;
    for (uint64_t i = 0; i < pool->pages_total; i++) {
        run = pool->used[i] ? 0 : run + 1;
        if (run > best) best = run;
    }
    stats->arena_bytes = pool->arena_bytes;
    stats->page_bytes = pool->page_bytes;
    stats->pages_total = pool->pages_total;
    stats->pages_used = pool->pages_used;
    stats->live_allocations = pool->live.size();
    stats->bytes_requested = pool->bytes_requested;
    stats->largest_free_run_pages = best;
    stats->evictions = pool->evictions;
    return DAF_OK;
}
