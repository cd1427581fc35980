"""Host tests of the importance-aware store (Sec. 3.4, Alg. 3 of the paper): hand-made scenarios whose outcome follows
from the policy's statement, and a step-by-step comparison with a reference that keeps no ordered index at all and
sorts the whole table whenever it needs a victim."""
import time

import numpy as np
import pytest

import paper_2507_07149_b200 as daf

PAGE = 65536
MB = 1 << 20


def nbytes(numel, G, b):
    up16 = lambda v: (v + 15) & ~15
    return up16(8 * ((numel + 16383) // 16384 + 1)) + 2 * up16(4 * (numel // G)) + up16(numel * b // 8) + up16(numel // G)


def test_size_model():
    assert daf.store_bytes(1 << 20, 256, 4) == 8 * 65 + 8 + 2 * 4 * 4096 + (1 << 19) + 4096 == nbytes(1 << 20, 256, 4)
    assert daf.store_bytes(32 * 3, 32, 1) == 16 + 2 * 16 + 16 + 16
    assert daf.store_bytes(1 << 20, 256, 0) == 0


def pages(numel, G, b, page=PAGE):
    return -(-nbytes(numel, G, b) // page)


class SortStore:
    """The same policy with plain lists: every victim is found by sorting all kept activations."""

    def __init__(self, mem, tbudget, widths=(1, 2, 4, 8), page=PAGE, step=100 * MB):
        self.mem, self.tb, self.widths, self.page, self.step = mem, tbudget, sorted(widths), page, step
        self.e = {}                                                 # id -> dict
        self.arena = [0] * min(mem // page, max(1, step // page))
        self.evictions = self.resizes = 0

    def _pages(self, a, level=None):
        level = a["level"] if level is None else level
        return pages(a["numel"], a["G"], self.widths[level], self.page)

    def _keys(self, a):
        size = float(max(1, self._pages(a, 0 if a["level"] is None else a["level"]) * self.page))
        return a["imp"] / size, a["imp"] / max(a["time"], 1e-30)

    def _kept(self):
        return [a for a in self.e.values() if a["level"] is not None]

    def _free(self, a):
        for p in range(a["first"], a["first"] + a["n"]):
            self.arena[p] = 0
        a["stored"], a["n"] = False, 0

    def _drop(self, a):
        if a["stored"]:
            self._free(a)
        a["level"] = None
        self.evictions += 1

    def _enforce(self, evicted):
        while True:
            kept = self._kept()
            used = sum(self._pages(a) for a in kept)
            used_t = sum(a["time"] for a in kept)
            cap = self.mem // self.page
            over_m, over_t = used > cap, used_t > self.tb
            if not over_m and not over_t:
                return
            rem_m = (cap - used) / cap if cap else -1.0
            rem_t = (self.tb - used_t) / self.tb if self.tb > 0 else -1.0
            mem_tighter = over_m and (not over_t or rem_m <= rem_t)
            if not kept:
                return
            order = (lambda a: (self._keys(a)[0], self._keys(a)[1], a["id"])) if mem_tighter else \
                    (lambda a: (self._keys(a)[1], self._keys(a)[0], a["id"]))
            v = sorted(kept, key=order)[0]
            if mem_tighter and not v["stored"] and v["level"] > 0:
                v["level"] -= 1
                self.resizes += 1
            else:
                self._drop(v)
                if evicted is not None:
                    evicted.append(v["id"])

    def _fit(self, need, limit=None):
        run = 0
        for i in range(len(self.arena) if limit is None else limit):
            run = 0 if self.arena[i] else run + 1
            if run == need:
                return i + 1 - need
        return None

    def estimate(self, ident, numel, G, imp, t, evicted=None):
        old = self.e.pop(ident, None)
        if old is not None and old["stored"]:
            self._free(old)
        self.e[ident] = dict(id=ident, numel=numel, G=G, imp=imp, time=t, level=len(self.widths) - 1, stored=False,
                             first=0, n=0)
        self._enforce(evicted)
        a = self.e[ident]
        return 0 if a["level"] is None else self.widths[a["level"]]

    def admit(self, ident, imp):
        a = self.e[ident]
        evicted = []
        a["imp"] = imp
        if a["level"] is None:
            a["level"] = 0
        self._enforce(evicted)
        if a["level"] is not None:
            need = self._pages(a)
            at = self._fit(need)
            cap = self.mem // self.page
            while at is None and len(self.arena) < cap:
                self.arena += [0] * (min(cap, len(self.arena) + max(1, self.step // self.page)) - len(self.arena))
                at = self._fit(need)
            while at is None:
                mine = self._keys(a)[0]
                cands = sorted((c for c in self._kept() if self._keys(c)[0] <= mine),
                               key=lambda c: (self._keys(c)[0], c["id"]))
                cands = [c for c in cands if c["stored"] and c["id"] != ident]
                if not cands:
                    break
                self._drop(cands[0])
                evicted.append(cands[0]["id"])
                at = self._fit(need)
            if at is None:
                self._drop(a)
                evicted.append(ident)
            else:
                for p in range(at, at + need):
                    self.arena[p] = 1
                a["stored"], a["first"], a["n"] = True, at, need
        return (0 if a["level"] is None else self.widths[a["level"]],
                a["first"] * self.page if a["stored"] else None, evicted)

    def release(self, ident):
        a = self.e.pop(ident)
        if a["stored"]:
            self._free(a)

    def set_budget(self, mem, tb):
        self.mem, self.tb = mem, tb
        evicted, moves = [], []
        self._enforce(evicted)
        cap, step = mem // self.page, max(1, self.step // self.page)
        target = len(self.arena)
        while target > cap:
            target = target - step if target > step else cap
        if target < len(self.arena):
            beyond = [a for a in self.e.values() if a["stored"] and a["first"] + a["n"] > target]
            for a in sorted(beyond, key=lambda a: (-a["imp"], a["id"])):
                old, need = a["first"], a["n"]
                for p in range(old, old + need):
                    self.arena[p] = 0
                at = self._fit(need, target)
                if at is None:
                    a["stored"], a["n"] = False, 0
                    self._drop(a)
                    evicted.append(a["id"])
                else:
                    for p in range(at, at + need):
                        self.arena[p] = 1
                    a["first"] = at
                    moves.append((a["id"], old * self.page, at * self.page, need * self.page))
            del self.arena[target:]
        return moves, evicted


def test_everything_fits_at_the_largest_width_first_fit_in_order():
    st = daf.Store(64 * MB, 100.0, step_bytes=16 * MB)
    n = 1 << 20
    for i in range(4):
        assert st.estimate(i, n, 256, 1.0 + i, 1.0) == 8
    at = 0
    for i in range(4):
        w, off, ev = st.admit(i, 1.0 + i)
        assert (w, off, ev) == (8, at, [])
        at += pages(n, 256, 8) * PAGE
    s = st.stats()
    assert s["used_bytes"] == at and s["planned_bytes"] == at and s["kept"] == 4 and s["arena_bytes"] == 16 * MB
    assert s["evictions"] == 0 and s["resizes"] == 0 and s["used_time"] == 4.0


def test_memory_pressure_lowers_the_least_valuable_width_by_width():
    n, G = 1 << 22, 256
    # budget: two activations at 8 bits plus one at 2 bits
    budget = (2 * pages(n, G, 8) + pages(n, G, 2)) * PAGE
    st = daf.Store(budget, 100.0)
    assert st.estimate(0, n, G, 9.0, 1.0) == 8
    assert st.estimate(1, n, G, 5.0, 1.0) == 8
    assert st.estimate(2, n, G, 1.0, 1.0) == 2                      # 8 -> 4 -> 2 and then it fits
    assert [st.width(i)[0] for i in range(3)] == [8, 8, 2]
    assert st.stats()["resizes"] == 2 and st.stats()["evictions"] == 0
    # a fourth, most valuable one: the least valuable per byte keeps giving way; at width 2 activation 2 is worth
    # 1 / 17 pages against 5 / 65 pages for activation 1, so activation 2 goes first (2 -> 1), then ...
    assert st.estimate(3, n, G, 20.0, 1.0) == 8
    ref = SortStore(budget, 100.0)
    for i, imp in enumerate((9.0, 5.0, 1.0, 20.0)):
        ref.estimate(i, n, G, imp, 1.0)
    got = [st.width(i)[0] for i in range(4)]
    assert got == [0 if a["level"] is None else ref.widths[a["level"]] for a in (ref.e[i] for i in range(4))]
    assert got[3] == 8 and got[0] >= got[1] >= got[2]
    assert st.stats()["planned_bytes"] <= budget


def test_time_pressure_evicts_by_importance_per_time_and_leaves_widths_alone():
    n, G = 1 << 20, 256
    st = daf.Store(1 << 30, 3.0)
    # importance / time: 0 -> 4, 1 -> 1, 2 -> 2.5, 3 -> 3
    for i, (imp, t) in enumerate(((4.0, 1.0), (2.0, 2.0), (2.5, 1.0), (3.0, 1.0))):
        st.estimate(i, n, G, imp, t)
    assert [st.width(i)[0] for i in range(4)] == [8, 0, 8, 8]        # 5 units of time > 3: activation 1 goes, 3 are left
    assert st.stats()["used_time"] == 3.0 and st.stats()["evictions"] == 1 and st.stats()["resizes"] == 0


def test_the_constraint_with_less_room_left_decides():
    n, G = 1 << 22, 256
    p8 = pages(n, G, 8)
    # three activations: memory over by little (3 p8 against 2.9 p8), time over by a lot (3 against 1.5)
    st = daf.Store(int(2.9 * p8) * PAGE, 1.5)
    st.estimate(0, n, G, 3.0, 1.0)
    st.estimate(1, n, G, 2.0, 1.0)
    st.estimate(2, n, G, 1.0, 1.0)
    # time is the tighter constraint both times: activation 2, then activation 1, are evicted outright; nothing resized
    assert [st.width(i)[0] for i in range(3)] == [8, 0, 0]
    assert st.stats()["resizes"] == 0
    # the other way round: time nearly fits, memory far over: widths go down instead
    st = daf.Store(int(1.2 * p8) * PAGE, 2.9)
    st.estimate(0, n, G, 3.0, 1.0)
    st.estimate(1, n, G, 2.0, 1.0)
    st.estimate(2, n, G, 1.0, 1.0)
    # (a width step halves an activation's size and so doubles its importance per byte: the victim changes as
    # the loop goes on, and no activation is dropped while another could still shrink)
    w = [st.width(i)[0] for i in range(3)]
    assert st.stats()["resizes"] > 0 and st.stats()["planned_bytes"] <= int(1.2 * p8) * PAGE
    assert sum(1 for x in w if x) >= 2 and w[0] >= w[1] >= w[2]


def test_admit_updates_keys_stored_activations_are_evicted_not_resized():
    n, G = 1 << 22, 256
    p8 = pages(n, G, 8)
    st = daf.Store(2 * p8 * PAGE, 100.0)
    st.estimate(0, n, G, 5.0, 1.0)
    st.estimate(1, n, G, 4.0, 1.0)
    assert st.admit(0, 5.0) == (8, 0, [])
    assert st.admit(1, 0.5) == (8, p8 * PAGE, [])                     # measured importance lower than estimated: still fits
    # a third one arrives that was not in the estimate; it is worth more than activation 1, which sits in pages and so
    # cannot shrink: it is evicted, and the newcomer takes its pages
    gone = []
    st.estimate(2, n, G, 3.0, 1.0, gone)                             # 2 is unplaced, worth 3 > 0.5 -> the victim is 1
    assert gone == [1]                                               # ... and the caller is told
    assert st.width(1) == (0, None)
    assert st.admit(2, 3.0) == (8, p8 * PAGE, [])
    s = st.stats()
    assert s["evictions"] == 1 and s["resizes"] == 0 and s["kept"] == 2
    # release returns the pages
    st.release(0)
    assert st.stats()["used_bytes"] == p8 * PAGE
    with pytest.raises(daf.DafError):
        st.release(0)
    with pytest.raises(daf.DafError):
        st.admit(2, 1.0)                                             # twice without a release


def test_arena_grows_and_shrinks_in_steps_and_reports_moves():
    n, G = 1 << 24, 256                                              # 16 Mi elements at 8 bits: ~16.6 MB each
    p8 = pages(n, G, 8)
    st = daf.Store(1000 * MB, 1e9)                                   # default step: 100 MB
    assert st.stats()["arena_bytes"] == 100 * MB
    for i in range(8):
        st.estimate(i, n, G, 1.0 + i, 1.0)
    offs = {}
    for i in range(8):
        w, off, ev = st.admit(i, 1.0 + i)
        assert w == 8 and ev == []
        offs[i] = off
    assert st.stats()["arena_bytes"] == 200 * MB and st.stats()["grows"] == 1   # 8 x 16.6 MB needs a second step
    assert offs[6] >= 100 * MB - p8 * PAGE                           # the later ones lie in the second step
    # free two in the first step, then lower the budget to 100 MB: what lies beyond the new end moves into the holes
    # (most important first) and the rest is evicted
    st.release(0)
    st.release(1)
    moves, evicted = st.set_budget(100 * MB, 1e9)
    s = st.stats()
    assert s["arena_bytes"] == 100 * MB and s["shrinks"] == 1
    assert s["used_bytes"] <= 100 * MB and s["planned_bytes"] <= 100 * MB
    beyond = [i for i in range(2, 8) if offs[i] + p8 * PAGE > 100 * MB]
    assert sorted([m[0] for m in moves] + [e for e in evicted if e in beyond]) == beyond
    for ident, src, dst, nb in moves:
        assert src == offs[ident] and dst + nb <= 100 * MB and nb == p8 * PAGE
        assert st.width(ident) == (8, dst)
    assert {m[2] for m in moves} <= {0, p8 * PAGE}                   # the two holes
    # no two kept activations overlap
    spans = sorted((st.width(i)[1], st.width(i)[1] + p8 * PAGE) for i in range(2, 8) if st.width(i)[1] is not None)
    assert all(a[1] <= b[0] for a, b in zip(spans, spans[1:]))
    # raising the budget again lets the arena grow by a step at the next allocation that needs it
    st.set_budget(1000 * MB, 1e9)
    for i in range(10, 16):
        st.estimate(i, n, G, 50.0, 1.0)
        st.admit(i, 50.0)
    assert st.stats()["arena_bytes"] == 200 * MB


def test_bad_arguments():
    with pytest.raises(daf.DafError):
        daf.Store(1 << 20, 1.0, widths=())
    st = daf.Store(1 << 24, 1.0)
    for args in ((0, 0, 256, 1.0, 1.0), (0, 1000, 256, 1.0, 1.0), (0, 1024, 256, -1.0, 1.0), (0, 1024, 256, 1.0, float("nan")),
                 (0, 1024, 0, 1.0, 1.0)):
        with pytest.raises(daf.DafError):
            st.estimate(*args)
    with pytest.raises(daf.DafError):
        st.admit(7, 1.0)
    with pytest.raises(daf.DafError):
        st.width(7)


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_random_scenarios_match_the_sort_based_reference(seed):
    """Several iterations of estimate / admit / release with budgets that change in between, sizes and importances
    drawn so that both constraints bind and ties occur; the two implementations must agree on every answer."""
    rng = np.random.default_rng(seed)
    page, step = 4096, 64 * 4096
    mem, tb = 700 * 4096, 24.0
    st = daf.Store(mem, tb, widths=(2, 4, 8) if seed == 1 else (1, 2, 4, 8), page_bytes=page, step_bytes=step)
    ref = SortStore(mem, tb, widths=(2, 4, 8) if seed == 1 else (1, 2, 4, 8), page=page, step=step)
    n_act = 40
    for it in range(6):
        numel = (rng.integers(1, 40, n_act) * 4096).tolist()
        imp = (rng.integers(0, 12, n_act) / 4.0).tolist()               # few distinct values: ties on purpose
        tcost = (rng.integers(1, 5, n_act) / 2.0).tolist()
        for i in range(n_act):
            gone, want_gone = [], []
            assert st.estimate(i, numel[i], 128, imp[i], tcost[i], gone) == \
                ref.estimate(i, numel[i], 128, imp[i], tcost[i], want_gone)
            assert gone == want_gone
        assert [st.width(i)[0] for i in range(n_act)] == \
            [0 if ref.e[i]["level"] is None else ref.widths[ref.e[i]["level"]] for i in range(n_act)]
        live = []
        for i in range(n_act):
            measured = float(rng.integers(0, 12)) / 4.0
            assert st.admit(i, measured) == ref.admit(i, measured), (it, i)
            live.append(i)
            if rng.random() < 0.15 and live:                            # something is consumed early
                j = live.pop(int(rng.integers(len(live))))
                st.release(j)
                ref.release(j)
            if i == n_act // 2:                                         # the budget changes in mid-iteration
                mem = int(rng.integers(200, 900)) * 4096
                tb = float(rng.integers(10, 40))
                got, want = st.set_budget(mem, tb), ref.set_budget(mem, tb)
                assert got == want, (it, "set_budget")
        s = st.stats()
        assert s["used_bytes"] == sum(ref.arena) * page and s["arena_bytes"] == len(ref.arena) * page
        assert s["evictions"] == ref.evictions and s["resizes"] == ref.resizes
        assert s["planned_bytes"] <= mem and s["used_time"] <= tb
        for i in live:
            st.release(i)
            ref.release(i)
        assert st.stats()["used_bytes"] == 0 and st.stats()["entries"] == 0


def test_ordered_indices_scale_where_sorting_does_not():
    """20,000 activations under a budget that forces thousands of victims: with the two trees each victim costs a
    few tree operations.  (The sort-based reference takes minutes at this size; 300 activations of it are timed
    for the ratio only.)"""
    rng = np.random.default_rng(7)
    n_act = 20000
    numel = (rng.integers(1, 64, n_act) * 16384).tolist()
    imp = rng.random(n_act).tolist()
    total8 = sum(pages(n, 256, 8) for n in numel) * PAGE
    st = daf.Store(total8 // 6, n_act * 0.4, step_bytes=total8)
    t0 = time.perf_counter()
    for i in range(n_act):
        st.estimate(i, numel[i], 256, imp[i], 1.0)
    dt_tree = time.perf_counter() - t0
    s = st.stats()
    assert s["planned_bytes"] <= total8 // 6 and s["used_time"] <= n_act * 0.4
    assert s["evictions"] + s["resizes"] > n_act
    # what is kept is worth more per byte than what was dropped, up to the width steps: the least valuable kept
    # activation at the smallest width is not below the most valuable dropped one ... checked on importance per page
    kept = [(imp[i] / pages(numel[i], 256, st.width(i)[0])) for i in range(0, n_act, 50) if st.width(i)[0]]
    assert kept and min(kept) > 0
    small = 300
    ref = SortStore(sum(pages(n, 256, 8) for n in numel[:small]) * PAGE // 6, small * 0.4, step=total8)
    t0 = time.perf_counter()
    for i in range(small):
        ref.estimate(i, numel[i], 256, imp[i], 1.0)
    dt_sort = time.perf_counter() - t0
    assert dt_tree < 5.0
    print(f"tree: {n_act} activations in {dt_tree:.3f} s; sorting: {small} in {dt_sort:.3f} s")
