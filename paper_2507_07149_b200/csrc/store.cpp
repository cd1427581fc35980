// Importance-aware activation store (host side, bookkeeping only): which saved activations are kept, at
// which bit width, and where in a preallocated arena (Sec. 3.4 of the paper).
//
//   Sec. 3.4.1  storage control as a greedy bi-objective knapsack: keep the total importance of what
//               is stored as high as the memory budget and the time budget allow; width 0 = not stored.
//               While a budget is exceeded, the constraint with the smaller remaining proportion is the
//               tighter one; the activation that is worth least per unit of that resource gives way
//               (ties: worth least per unit of the other resource).
//   Sec. 3.4.2  one contiguous arena handed out in pages, first fit.
//   Sec. 3.4.3  the page table is two ordered indices (red-black trees: std::set) over the same
//   + Alg. 3    activations, keyed importance / size and importance / time; whenever one is updated the
//               other is too.  SelectMax / UpdateSize / Evict / UpdateKey / InsertPage of Alg. 3 are
//               select_victim / update_size / evict / update_key / insert_page below.
//   Sec. 3.4.4  the arena follows a changing memory budget in fixed steps (100 MB unless told
//               otherwise): it grows by a step when an allocation does not fit and shrinks by steps
//               when the budget falls, moving or evicting what lies beyond the new end.
//
// Reading of Alg. 3 where the paper leaves the orientation open: the activation that gives way is the
// one at the LOW end of the tighter index (least importance per byte, or per unit of time); under
// memory pressure an activation that has not been stored yet this iteration gives way by going down one
// width (UpdateSize; below the smallest width it is dropped), one that already sits in pages is evicted;
// under time pressure the victim is always evicted.
//
// The store never touches the arena's memory: the caller owns it, compresses into the offsets the
// store hands out, and carries out the moves a shrinking budget asks for.
#include <algorithm>
#include <cmath>
#include <map>
#include <new>
#include <set>
#include <utility>
#include <vector>

#include "../../include/daf.h"

namespace {

struct Entry {
    uint64_t id = 0, numel = 0;
    uint32_t group_size = 256;
    double importance = 0.0, time = 0.0;       // time: what keeping it costs per iteration (compress + decompress)
    uint32_t level = 0;                        // index into the allowed widths, or kDropped
    bool stored = false;                       // sits in pages (InsertPage done)
    uint64_t first_page = 0, n_pages = 0;
    double mem_key = 0.0, time_key = 0.0;      // the keys it is filed under
};
constexpr uint32_t kDropped = 0xFFFFFFFFu;

}  // namespace

struct daf_store {
    daf_store_config cfg;
    std::vector<uint32_t> widths;              // allowed widths, ascending
    std::map<uint64_t, Entry> entries;
    std::set<std::pair<double, uint64_t>> mem_tree, time_tree;   // (key, id): the two ordered indices
    std::vector<uint8_t> page_used;            // arena pages (the arena's current size = page_used.size() pages)
    uint64_t used_pages = 0;
    double used_time = 0.0;
    uint64_t evictions = 0, resizes = 0, grows = 0, shrinks = 0, moves = 0;

    uint64_t bytes_of(const Entry &e, uint32_t level) const
    {
        return level == kDropped ? 0 : daf_store_bytes(e.numel, e.group_size, widths[level]);
    }
    uint64_t pages_of(const Entry &e, uint32_t level) const
    {
        return (bytes_of(e, level) + cfg.page_bytes - 1) / cfg.page_bytes;
    }
    // memory the kept entries count for: the pages each has, or will need once it is placed (kept up to date by
    // file / unfile, so that the loop of Alg. 3 costs one tree operation per step)
    uint64_t planned = 0;
    uint64_t planned_pages() const { return planned; }
    void unfile(Entry &e)
    {
        if (mem_tree.erase({e.mem_key, e.id})) planned -= pages_of(e, e.level);
        time_tree.erase({e.time_key, e.id});
    }
    void file(Entry &e)                        // UpdateKey: both indices together
    {
        const double size = (double)std::max<uint64_t>(1, pages_of(e, e.level == kDropped ? 0 : e.level) * cfg.page_bytes);
        e.mem_key = e.importance / size;
        e.time_key = e.importance / std::max(e.time, 1e-30);
        if (e.level != kDropped) {
            mem_tree.insert({e.mem_key, e.id});
            time_tree.insert({e.time_key, e.id});
            planned += pages_of(e, e.level);
        }
    }
    void free_pages(Entry &e)
    {
        for (uint64_t p = e.first_page; p < e.first_page + e.n_pages; p++) page_used[p] = 0;
        used_pages -= e.n_pages;
        e.stored = false;
        e.n_pages = 0;
    }
    void drop(Entry &e)                        // Evict: out of both indices, pages returned
    {
        unfile(e);
        if (e.stored) free_pages(e);
        if (e.level != kDropped) used_time -= e.time;
        e.level = kDropped;
        evictions++;
    }
    // First fit over the arena as it is; returns pages_total when no run of `need` pages is free.
    uint64_t first_fit(uint64_t need) const
    {
        uint64_t run = 0;
        for (uint64_t i = 0; i < page_used.size(); i++) {
            run = page_used[i] ? 0 : run + 1;
            if (run == need) return i + 1 - need;
        }
        return page_used.size();
    }
    uint64_t budget_pages() const { return cfg.mem_budget_bytes / cfg.page_bytes; }
    uint64_t step_pages() const { return std::max<uint64_t>(1, cfg.step_bytes / cfg.page_bytes); }
};

namespace {

// SelectMax of Alg. 3 (see the reading above): the entry that gives way under the tighter constraint.
Entry *select_victim(daf_store *s, bool mem_tighter)
{
    auto &tree = mem_tighter ? s->mem_tree : s->time_tree;
    Entry *best = nullptr;
    for (auto it = tree.begin(); it != tree.end(); ++it) {
        Entry &e = s->entries[it->second];
        if (!best) {
            best = &e;
            continue;
        }
        // candidates that tie on the primary key: the other constraint decides
        const double k0 = mem_tighter ? best->mem_key : best->time_key, k1 = mem_tighter ? e.mem_key : e.time_key;
        if (k1 > k0) break;
        const double s0 = mem_tighter ? best->time_key : best->mem_key, s1 = mem_tighter ? e.time_key : e.mem_key;
        if (s1 < s0) best = &e;
    }
    return best;
}

// Brings UsedMem and UsedTime under the budgets (the while loop of Alg. 3).  Ids that lose their place are appended
// to `evicted`.
void enforce(daf_store *s, std::vector<uint64_t> *evicted)
{
    for (;;) {
        const uint64_t used = s->planned_pages(), cap = s->budget_pages();
        const bool over_mem = used > cap, over_time = s->used_time > s->cfg.time_budget;
        if (!over_mem && !over_time) return;
        // the tighter constraint: the smaller remaining proportion
        const double rem_mem = cap ? ((double)cap - (double)used) / (double)cap : -1.0;
        const double rem_time = s->cfg.time_budget > 0 ? (s->cfg.time_budget - s->used_time) / s->cfg.time_budget : -1.0;
        const bool mem_tighter = over_mem && (!over_time || rem_mem <= rem_time);
        Entry *v = select_victim(s, mem_tighter);
        if (!v) return;                                           // nothing left to give way
        if (mem_tighter && !v->stored && v->level != kDropped && v->level > 0) {
            s->unfile(*v);                                        // UpdateSize: one width down, keys refiled in both indices
            v->level--;
            s->file(*v);
            s->resizes++;
        } else {
            s->drop(*v);
            if (evicted) evicted->push_back(v->id);
        }
    }
}

uint32_t copy_out(const std::vector<uint64_t> &v, uint64_t *out, uint32_t *n)
{
    const uint32_t cap = n ? *n : 0;
    if (n) *n = (uint32_t)v.size();
    for (uint32_t i = 0; i < cap && i < v.size(); i++)
        if (out) out[i] = v[i];
    return (uint32_t)v.size();
}

}  // namespace

// What one activation occupies: window offsets, min, scale, packed codes, widths, each part rounded up to 16 bytes so
// that every part can start on the boundary the kernels ask for.
extern "C" uint64_t daf_store_bytes(uint64_t numel, uint32_t group_size, uint32_t width)
{
    if (group_size == 0 || width == 0) return 0;
    auto up16 = [](uint64_t v) { return (v + 15) & ~15ull; };
    const uint64_t groups = numel / group_size, windows = (numel + 16383) / 16384;
    return up16(8 * (windows + 1)) + 2 * up16(4 * groups) + up16(numel * width / 8) + up16(groups);
}

extern "C" daf_store *daf_store_create(const daf_store_config *cfg)
{
    if (!cfg || cfg->width_mask == 0 || (cfg->width_mask & ~0x116u)) return nullptr;
    daf_store *s = new (std::nothrow) daf_store();
    if (!s) return nullptr;
    s->cfg = *cfg;
    if (s->cfg.page_bytes == 0) s->cfg.page_bytes = 65536;
    if (s->cfg.step_bytes == 0) s->cfg.step_bytes = 100ull << 20;
    for (uint32_t b = 1; b <= 8; b <<= 1)
        if (cfg->width_mask & (1u << b)) s->widths.push_back(b);
    // the arena starts with one step (or the whole budget when that is smaller)
    s->page_used.assign(std::min(s->budget_pages(), s->step_pages()), 0);
    return s;
}

extern "C" void daf_store_destroy(daf_store *s) { delete s; }

extern "C" daf_status daf_store_estimate(daf_store *s, uint64_t id, uint64_t numel, uint32_t group_size, double importance,
                                         double time_cost, uint32_t *width, uint64_t *evicted_ids, uint32_t *n_evicted)
{
    if (!s || numel == 0 || group_size == 0 || numel % group_size || !(importance >= 0.0) || !(time_cost >= 0.0))
        return DAF_ERR_INVALID_ARG;
    auto it = s->entries.find(id);
    if (it != s->entries.end()) {                                 // a new iteration's estimate replaces the old entry
        Entry &old = it->second;
        s->unfile(old);
        if (old.stored) s->free_pages(old);
        if (old.level != kDropped) s->used_time -= old.time;
        s->entries.erase(it);
    }
    Entry e;
    e.id = id;
    e.numel = numel;
    e.group_size = group_size;
    e.importance = importance;
    e.time = time_cost;
    e.level = (uint32_t)s->widths.size() - 1;                     // start at the largest width, give way as needed
    s->entries[id] = e;
    s->used_time += time_cost;
    s->file(s->entries[id]);
    std::vector<uint64_t> evicted;
    enforce(s, &evicted);
    const Entry &now = s->entries[id];
    if (width) *width = now.level == kDropped ? 0u : s->widths[now.level];
    copy_out(evicted, evicted_ids, n_evicted);
    return DAF_OK;
}

extern "C" daf_status daf_store_width(const daf_store *s, uint64_t id, uint32_t *width, uint64_t *offset)
{
    if (!s) return DAF_ERR_INVALID_ARG;
    auto it = s->entries.find(id);
    if (it == s->entries.end()) return DAF_ERR_INVALID_ARG;
    if (width) *width = it->second.level == kDropped ? 0u : s->widths[it->second.level];
    if (offset) *offset = it->second.stored ? it->second.first_page * s->cfg.page_bytes : UINT64_MAX;
    return DAF_OK;
}

extern "C" daf_status daf_store_admit(daf_store *s, uint64_t id, double importance, uint32_t *width, uint64_t *offset,
                                      uint64_t *evicted_ids, uint32_t *n_evicted)
{
    if (!s || !(importance >= 0.0)) return DAF_ERR_INVALID_ARG;
    auto it = s->entries.find(id);
    if (it == s->entries.end()) return DAF_ERR_INVALID_ARG;
    Entry &e = it->second;
    std::vector<uint64_t> evicted;
    if (e.stored) return DAF_ERR_INVALID_ARG;                     // admitted twice without a release in between
    // UpdateKey in both indices with the importance just measured; an activation the estimate had dropped gets
    // another chance at the smallest width
    s->unfile(e);
    e.importance = importance;
    if (e.level == kDropped) {
        e.level = 0;
        s->used_time += e.time;
    }
    s->file(e);
    enforce(s, &evicted);
    if (e.level != kDropped) {
        // FirstFit over the free pages; the arena grows by a step (up to the budget) when nothing fits
        uint64_t need = s->pages_of(e, e.level), at = s->first_fit(need);
        while (at == s->page_used.size() && s->page_used.size() < s->budget_pages()) {
            s->page_used.resize(std::min<uint64_t>(s->budget_pages(), s->page_used.size() + s->step_pages()), 0);
            s->grows++;
            at = s->first_fit(need);
        }
        if (at == s->page_used.size()) {
            // the budget holds the bytes but not in one run (fragmentation): stored activations worth less per byte
            // than this one go, least valuable first, until a run opens up
            while (at == s->page_used.size()) {
                Entry *v = nullptr;
                for (const auto &kv : s->mem_tree) {
                    Entry &c = s->entries[kv.second];
                    if (kv.first > e.mem_key) break;
                    if (c.stored && c.id != id) {
                        v = &c;
                        break;
                    }
                }
                if (!v) break;
                s->drop(*v);
                evicted.push_back(v->id);
                at = s->first_fit(need);
            }
        }
        if (at == s->page_used.size()) {
            s->drop(e);                                           // no room at all
            evicted.push_back(id);
        } else {                                                  // InsertPage
            for (uint64_t p = at; p < at + need; p++) s->page_used[p] = 1;
            s->used_pages += need;
            e.stored = true;
            e.first_page = at;
            e.n_pages = need;
        }
    }
    if (width) *width = e.level == kDropped ? 0u : s->widths[e.level];
    if (offset) *offset = e.stored ? e.first_page * s->cfg.page_bytes : UINT64_MAX;
    copy_out(evicted, evicted_ids, n_evicted);
    return DAF_OK;
}

extern "C" daf_status daf_store_release(daf_store *s, uint64_t id)
{
    if (!s) return DAF_ERR_INVALID_ARG;
    auto it = s->entries.find(id);
    if (it == s->entries.end()) return DAF_ERR_INVALID_ARG;
    Entry &e = it->second;
    s->unfile(e);
    if (e.stored) s->free_pages(e);
    if (e.level != kDropped) s->used_time -= e.time;
    s->entries.erase(it);
    return DAF_OK;
}

extern "C" daf_status daf_store_set_budget(daf_store *s, uint64_t mem_budget_bytes, double time_budget, daf_store_move *moves,
                                           uint32_t *n_moves, uint64_t *evicted_ids, uint32_t *n_evicted)
{
    if (!s || !(time_budget >= 0.0)) return DAF_ERR_INVALID_ARG;
    s->cfg.mem_budget_bytes = mem_budget_bytes;
    s->cfg.time_budget = time_budget;
    std::vector<uint64_t> evicted;
    std::vector<daf_store_move> moved;
    enforce(s, &evicted);                             // the trees first: what no longer fits the budgets goes
    // then the arena: down in steps until it fits the new budget; what lies beyond the new end moves to the first
    // fit below it, or goes when there is none
    uint64_t target = s->page_used.size();
    while (target > s->budget_pages()) target = target > s->step_pages() ? target - s->step_pages() : s->budget_pages();
    if (target < s->page_used.size()) {
        std::vector<Entry *> beyond;
        for (auto &kv : s->entries)
            if (kv.second.stored && kv.second.first_page + kv.second.n_pages > target) beyond.push_back(&kv.second);
        std::sort(beyond.begin(), beyond.end(), [](const Entry *x, const Entry *y) { return x->importance > y->importance; });
        for (Entry *e : beyond) {
            const uint64_t old_first = e->first_page, need = e->n_pages;
            for (uint64_t p = old_first; p < old_first + need; p++) s->page_used[p] = 0;
            uint64_t run = 0, at = target;                        // first fit below the new end
            for (uint64_t i = 0; i < target; i++) {
                run = s->page_used[i] ? 0 : run + 1;
                if (run == need) {
                    at = i + 1 - need;
                    break;
                }
            }
            if (at == target) {
                s->used_pages -= need;
                e->stored = false;
                e->n_pages = 0;
                s->drop(*e);
                evicted.push_back(e->id);
            } else {
                for (uint64_t p = at; p < at + need; p++) s->page_used[p] = 1;
                e->first_page = at;
                moved.push_back(daf_store_move{e->id, old_first * s->cfg.page_bytes, at * s->cfg.page_bytes,
                                               need * s->cfg.page_bytes});
                s->moves++;
            }
        }
        s->page_used.resize(target);
        s->shrinks++;
    }
    const uint32_t cap = n_moves ? *n_moves : 0;
    if (n_moves) *n_moves = (uint32_t)moved.size();
    for (uint32_t i = 0; i < cap && i < moved.size(); i++)
        if (moves) moves[i] = moved[i];
    copy_out(evicted, evicted_ids, n_evicted);
    return DAF_OK;
}

extern "C" daf_status daf_store_get_stats(const daf_store *s, daf_store_stats *st)
{
    if (!s || !st) return DAF_ERR_INVALID_ARG;
    st->arena_bytes = s->page_used.size() * s->cfg.page_bytes;
    st->mem_budget_bytes = s->cfg.mem_budget_bytes;
    st->used_bytes = s->used_pages * s->cfg.page_bytes;
    st->planned_bytes = s->planned_pages() * s->cfg.page_bytes;
    st->time_budget = s->cfg.time_budget;
    st->used_time = s->used_time;
    st->entries = s->entries.size();
    st->kept = s->mem_tree.size();
    st->evictions = s->evictions;
    st->resizes = s->resizes;
    st->grows = s->grows;
    st->shrinks = s->shrinks;
    st->moves = s->moves;
    return DAF_OK;
}
