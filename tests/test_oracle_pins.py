"""Pins for the CPU oracle: each stage is checked against something other than itself --
published known-answer vectors, numpy library routines, closed forms, brute force on tiny
inputs, float64 evaluations of Eq. 1 and worked vectors stored under tests/golden/."""
import heapq
import itertools
import os

import numpy as np
import pytest

import oracle

HEX = lambda a: [f"{int(v):08x}" for v in np.asarray(a).view(np.uint32).reshape(-1)]


def _sections(path):
    out, cur = {}, None
    for line in open(path):
        line = line.rstrip("\n")
        if not line or line.startswith("#"):
            continue
        if line.startswith("["):
            cur = line.strip("[]")
            out[cur] = []
        else:
            out[cur].append(line.split())
    return out


@pytest.fixture(scope="module")
def worked(golden_dir):
    return _sections(os.path.join(golden_dir, "worked_vectors.txt"))


def _ramp():
    return (np.arange(32, dtype=np.float32) * np.float32(0.1)).astype(np.float32)


# ------------------------------------------------------------------ Philox
def test_philox_known_answer_vectors(golden_dir):
    rows = [l.split() for l in open(os.path.join(golden_dir, "philox4x32_10_kat.txt")) if not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(t, 16) for t in r]
        got = oracle.philox4x32_10(v[0:4], v[4:6])
        assert [int(g) for g in got] == v[6:10]


def test_philox_single_round_by_hand():
    # one round on ctr=(1,2,3,4), key=(5,6): products taken with Python integers
    p0, p1 = 0xD2511F53 * 1, 0xCD9E8D57 * 3
    want = [(p1 >> 32) ^ 2 ^ 5, p1 & 0xFFFFFFFF, (p0 >> 32) ^ 4 ^ 6, p0 & 0xFFFFFFFF]
    ctr, key = oracle.philox_round([1, 2, 3, 4], [5, 6])
    assert [int(c) for c in ctr] == want
    assert [int(k) for k in key] == [(5 + 0x9E3779B9) & 0xFFFFFFFF, (6 + 0xBB67AE85) & 0xFFFFFFFF]


def test_r15_is_a_function_of_seed_and_element_index(worked):
    want = [int(t, 16) for t in worked["r15 seed=0 elements 0..11"][0]]
    assert [oracle.r15(0, j) for j in range(12)] == want
    # lanes of one Philox block: element j uses 16-bit lane j&7 of block j>>3, top 15 bits
    for seed, blk in ((0, 0), (7, 3), (2**40 + 5, 2**33 + 1)):
        o = oracle.philox4x32_10([blk & 0xFFFFFFFF, blk >> 32, 0, 0], [seed & 0xFFFFFFFF, seed >> 32])
        halves = []
        for w in o:
            halves += [int(w) & 0xFFFF, int(w) >> 16]
        assert [oracle.r15(seed, 8 * blk + e) for e in range(8)] == [h >> 1 for h in halves]


def test_r15_is_uniform_enough():
    r = np.array([oracle.r15(123, j) for j in range(1 << 15)], np.float64)
    assert r.min() >= 0 and r.max() < 2**15
    assert abs(r.mean() - (2**15 - 1) / 2) < 4 * 2**15 / np.sqrt(12 * r.size)


# ------------------------------------------------------------------ 16-bit conversions
def test_half_conversions_against_numpy():
    allh = np.arange(1 << 16, dtype=np.uint16)
    want = allh.view(np.float16).astype(np.float32)
    got = oracle.widen(allh.view(np.float16))
    finite = np.isfinite(want)
    assert np.array_equal(got.view(np.uint32)[finite], want.view(np.uint32)[finite])
    rng = np.random.default_rng(0)
    f = np.concatenate([rng.standard_normal(20000).astype(np.float32) * np.float32(10.0) ** rng.integers(-9, 6, 20000),
                        want[finite], np.float32([65504, 65519.99, 65520, 1e9, 2**-24, 2**-25, 2**-25 * 1.0001,
                                                  2**-14, 2**-14 * 0.9999, 0.0, -0.0])]).astype(np.float32)
    with np.errstate(over="ignore"):
        ref = f.astype(np.float16).view(np.uint16)
    got = np.array([oracle.lib().daf_oracle_float_to_half(float(v)) for v in f], np.uint16)
    assert np.array_equal(got, ref)


def test_bf16_conversions_against_torch():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(1)
    f = (rng.standard_normal(50000) * 10.0 ** rng.integers(-20, 20, 50000)).astype(np.float32)
    ref = torch.from_numpy(f).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle.lib().daf_oracle_float_to_bf16(float(v)) for v in f], np.uint16)
    assert np.array_equal(got, ref)
    back = oracle.widen(ref, dtype="bf16")
    want = torch.from_numpy(ref.view(np.int16)).view(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(back.view(np.uint32), want.view(np.uint32))


# ------------------------------------------------------------------ stats
@pytest.mark.parametrize("G", [32, 64, 256, 1024])
def test_stats_against_numpy_min_max(G):
    rng = np.random.default_rng(G)
    x = (rng.standard_normal(G * 37) * 10.0 ** rng.integers(-3, 3, G * 37)).astype(np.float32)
    mn, mx, R = oracle.stats(x, G)
    xr = x.reshape(-1, G)
    assert np.array_equal(mn, xr.min(1)) and np.array_equal(mx, xr.max(1))
    assert np.array_equal(R, (xr.max(1) - xr.min(1)).astype(np.float32))


def test_stats_signed_zero_and_degenerate_groups():
    x = np.zeros(96, np.float32)
    x[0:32] = [0.0, -0.0] * 16                 # min must be -0.0, max +0.0
    x[32:64] = -0.0                            # all -0.0
    x[64:96] = np.float32(1.0)
    x[65] = np.float32(1.0) + np.float32(2.0 ** -23)
    mn, mx, R = oracle.stats(x, 32)
    assert HEX(mn) == ["80000000", "80000000", "3f800000"]
    assert HEX(mx) == ["00000000", "80000000", "3f800001"]
    assert R[0] == 0 and R[1] == 0 and R[2] == np.float32(2.0 ** -23)
    tiny = np.zeros(32, np.float32)
    tiny[3] = np.float32(2.0 ** -119)          # range below 2^-118 counts as constant
    assert oracle.stats(tiny, 32)[2][0] == 0
    tiny[3] = np.float32(2.0 ** -118)
    assert oracle.stats(tiny, 32)[2][0] == np.float32(2.0 ** -118)


def test_stats_rejects_non_finite():
    x = np.ones(32, np.float32)
    x[5] = np.inf
    with pytest.raises(oracle.OracleError):
        oracle.stats(x, 32)
    x[5] = np.nan
    with pytest.raises(oracle.OracleError):
        oracle.stats(x, 32)
    x[5] = np.float32(3e38)
    x[6] = np.float32(-3e38)                   # finite values, infinite range
    with pytest.raises(oracle.OracleError):
        oracle.stats(x, 32)


# ------------------------------------------------------------------ bit choice
def test_raise_factors(worked):
    for b_lo, b_hi, hx in worked["raise factors b_lo b_hi hex"]:
        b_lo, b_hi = int(b_lo), int(b_hi)
        got = oracle.raise_factor(b_lo, b_hi)
        assert HEX(got)[0] == hx
        c = lambda b: 1.0 / (2.0 ** b - 1.0) ** 2
        assert abs(float(got) - np.sqrt((c(b_lo) - c(b_hi)) / (b_hi - b_lo))) < 1e-7


def test_bit_choice_worked_example(worked):
    sec = worked["bit choice: widths 1 2 4 8, budget 3, one window"]
    R = np.float32([float(t) for t in sec[0][1:]])
    want = [int(t) for t in sec[1][1:]]
    assert list(oracle.choose_bits(R, len(R), [1, 2, 4, 8], 3.0)) == want


def _heap_greedy(R, widths, beta_q8):
    """Independent sequential restatement: a max-heap holding each group's next raise."""
    n, S = len(R), sorted(widths)
    rem = ((beta_q8 * n) >> 8) - S[0] * n
    level = [0] * n

    def entry(g, k):
        v = np.float32(np.sqrt((1 / (2.0 ** S[k] - 1) ** 2 - 1 / (2.0 ** S[k + 1] - 1) ** 2) / (S[k + 1] - S[k])))
        key = int(np.float32(np.float32(R[g]) * v).view(np.uint32))
        return (-key, k, g)

    heap = [entry(g, 0) for g in range(n)] if len(S) > 1 else []
    heapq.heapify(heap)
    while heap:
        _, k, g = heapq.heappop(heap)
        cost = S[k + 1] - S[k]
        if cost > rem:
            break
        rem -= cost
        level[g] = k + 1
        if k + 2 < len(S):
            heapq.heappush(heap, entry(g, k + 1))
    return [S[l] for l in level]


@pytest.mark.parametrize("widths", [(1, 2, 4, 8), (2, 4, 8), (1, 8), (4,), (1, 2), (2, 8), (1, 4, 8)])
def test_bit_choice_equals_heap_greedy(widths):
    rng = np.random.default_rng(sum(widths))
    for trial in range(60):
        n = int(rng.integers(1, 70))
        kind = trial % 4
        if kind == 0:
            R = rng.random(n).astype(np.float32) * np.float32(10)
        elif kind == 1:
            R = (10.0 ** rng.uniform(-3, 3, n)).astype(np.float32)
        elif kind == 2:
            R = rng.choice(np.float32([0, 1, 2, 6, 6, 6]), n).astype(np.float32)      # many ties, zeros
        else:
            R = np.full(n, 6, np.float32)
        beta = float(rng.choice([min(widths), min(widths) + 0.37, 2.5, 3.0, 4.0, 5.75, 8.0]))
        if beta < min(widths):
            continue
        got = oracle.choose_bits(R, n, widths, beta)
        assert list(got) == _heap_greedy(R, widths, int(np.floor(np.float32(beta) * 256)))
        assert int(got.sum()) <= (int(np.floor(beta * 256)) * n) >> 8          # budget never exceeded


def test_bit_choice_two_widths_is_optimal_by_brute_force():
    rng = np.random.default_rng(5)
    c = lambda b: 1.0 / (2.0 ** b - 1.0) ** 2
    for widths in ((2, 4), (1, 8), (4, 8)):
        for _ in range(20):
            n = int(rng.integers(2, 9))
            R = (rng.random(n) * 5 + 0.1).astype(np.float32)
            beta = float(rng.uniform(widths[0], widths[1]))
            T = (int(np.floor(np.float32(beta) * 256)) * n) >> 8
            got = oracle.choose_bits(R, n, widths, beta)
            best = min((sum(float(R[g]) ** 2 * c(a[g]) for g in range(n)), a)
                       for a in itertools.product(widths, repeat=n) if sum(a) <= T)
            err = sum(float(R[g]) ** 2 * c(int(got[g])) for g in range(n))
            assert err <= best[0] * (1 + 1e-6)
            assert int(got.sum()) <= T


def test_bit_choice_special_cases():
    rng = np.random.default_rng(9)
    R = (rng.random(64) + 1).astype(np.float32)                 # distinct, within a factor of two
    assert set(oracle.choose_bits(R, 64, [1, 2, 4, 8], 1.0)) == {1}
    assert set(oracle.choose_bits(R, 64, [1, 2, 4, 8], 8.0)) == {8}
    assert set(oracle.choose_bits(R, 64, [2, 4, 8], 4.0)) == {4}
    b = oracle.choose_bits(R, 64, [1, 2, 4, 8], 3.0)            # half at 2, half at 4: the larger ranges get 4
    assert sorted(b) == [2] * 32 + [4] * 32
    assert R[b == 4].min() > R[b == 2].max()
    with pytest.raises(oracle.OracleError):
        oracle.choose_bits(R, 64, [2, 4], 1.5)                  # budget below the smallest width
    # ties: equal ranges are raised in group order
    b = oracle.choose_bits(np.full(8, 6, np.float32), 8, [1, 2], 1.5)
    assert list(b) == [2, 2, 2, 2, 1, 1, 1, 1]
    # windows are independent: the last window may be short
    R2 = np.concatenate([R, R[:10]])
    b2 = oracle.choose_bits(R2, 64, [1, 2, 4, 8], 3.0)
    assert np.array_equal(b2[:64], oracle.choose_bits(R, 64, [1, 2, 4, 8], 3.0))
    assert np.array_equal(b2[64:], oracle.choose_bits(R[:10], 10, [1, 2, 4, 8], 3.0))


def test_bit_choice_monotone_in_range():
    rng = np.random.default_rng(11)
    for _ in range(30):
        R = (10.0 ** rng.uniform(-2, 2, 64)).astype(np.float32)
        b = oracle.choose_bits(R, 64, [1, 2, 4, 8], float(rng.choice([2.0, 2.5, 3.0, 4.0, 5.0])))
        order = np.argsort(R, kind="stable")
        assert np.all(np.diff(b[order].astype(int)) >= 0)       # a larger range never gets fewer bits


# ------------------------------------------------------------------ group parameters and codes
def test_group_params_are_ieee_divisions():
    R = np.float32([0.0, 1.5, 3.1000001, 6.0, 1e-30, 1e30])
    for b in (1, 2, 4, 8):
        scale, inv = oracle.group_params(R, np.full(R.size, b, np.uint8))
        L = np.float32(2 ** b - 1)
        with np.errstate(divide="ignore", invalid="ignore"):
            assert np.array_equal(scale[1:], (R / L)[1:]) and np.array_equal(inv[1:], (L / R)[1:])
        assert scale[0] == 0 and inv[0] == 0


def test_float_to_uint_offset_trick_closed_form():
    # Eq. 5: bits(X) | 0x4B000000 is the float 2^23 + X, so subtracting 2^23 gives float(X) ...
    X = np.concatenate([np.arange(256), np.random.default_rng(0).integers(0, 2**23, 10000)]).astype(np.uint32)
    assert np.array_equal((X | np.uint32(0x4B000000)).view(np.float32) - np.float32(2**23), X.astype(np.float32))
    # ... and read backwards with offset 256: for s in [256, 512) the mantissa field is (s - 256) * 2^15
    s = np.float32(256) + np.random.default_rng(1).integers(0, 2**23, 10000).astype(np.float32) * np.float32(2.0**-15)
    assert np.array_equal(s.view(np.uint32) - np.uint32(0x43800000), ((s.astype(np.float64) - 256) * 2**15).astype(np.uint32))


def test_codes_scalar_example(worked):
    sec = dict((r[0], r[1]) for r in worked["scalar mn=0 mx=1.5 width=4 x=0.75"])
    scale, inv = oracle.group_params(np.float32([1.5]), np.uint8([4]))
    assert HEX(scale)[0] == sec["scale"] and HEX(inv)[0] == sec["inv"]
    s = np.float32(np.float64(0.75) * np.float64(inv[0]) + 256.0)
    assert HEX(s)[0] == sec["s"] and int(s.view(np.uint32)) - 0x43800000 == int(sec["fixed"])
    x = np.zeros(32, np.float32)
    x[0], x[1] = 0.75, 1.5
    mn, inv32, bits = np.float32([0]), inv, np.uint8([4])
    for r, want in ((0, 7), (0x3FFF, 7), (0x4000, 8), (0x7FFF, 8)):
        q = oracle.codes_r15(x, 32, mn, inv32, bits, np.full(32, r, np.uint16))
        assert q[0] == want and q[1] == 15 and q[2] == 0


def test_codes_mean_over_all_offsets_is_exact():
    """Summed over all 2^15 rounding offsets the code equals the fixed-point value exactly,
    so the stochastic code is unbiased on the 2^-15 grid, and that value is Eq. 1's quotient."""
    rng = np.random.default_rng(3)
    r_all = np.arange(1 << 15, dtype=np.uint16)
    for b in (1, 2, 4, 8):
        L = 2 ** b - 1
        mn, R = np.float32(rng.normal()), np.float32(rng.random() * 7 + 0.01)
        scale, inv = oracle.group_params(np.float32([R]), np.uint8([b]))
        xs = (mn + R * rng.random(6).astype(np.float32)).astype(np.float32)
        xs = np.clip(xs, mn, np.float32(mn + R))
        for xv in xs:
            x = np.full(1 << 15, xv, np.float32)
            q = oracle.codes_r15(x, 1 << 15, np.float32([mn]), inv, np.uint8([b]), r_all).astype(np.int64)
            t = (np.float64(xv) - np.float64(mn)) / (np.float64(R) / L)          # Eq. 1 in float64
            fixed = int(q.sum())
            if t < L - 1e-3:                                                    # away from the clamp
                assert abs(fixed / 2**15 - t) <= 2**-15 + 4 * L * 2**-23
                assert set(np.unique(q)) <= {int(np.floor(fixed / 2**15)), int(np.floor(fixed / 2**15)) + 1}
            assert q.max() <= L


@pytest.mark.parametrize("b", [1, 2, 4, 8])
def test_nearest_codes_against_eq1_in_float64(b):
    rng = np.random.default_rng(b)
    G, ng = 64, 200
    x = (rng.standard_normal(G * ng) * 3).astype(np.float32)
    mn, mx, R = oracle.stats(x, G)
    bits = np.full(ng, b, np.uint8)
    scale, inv = oracle.group_params(R, bits)
    q = oracle.codes(x, G, mn, inv, bits, rounding=oracle.ROUND_NEAREST)
    L = 2 ** b - 1
    t = (x.astype(np.float64) - np.repeat(mn, G)) / (np.repeat(R.astype(np.float64), G) / L)
    want = np.minimum(np.floor(t + 0.5), L)
    near_tie = np.abs(t - np.floor(t) - 0.5) < 2.0 ** -14 + 4 * L * 2.0 ** -23
    assert np.array_equal(q[~near_tie], want[~near_tie].astype(np.uint8))
    assert np.all(np.abs(q[near_tie].astype(np.int64) - want[near_tie]) <= 1)
    # error bound of round-to-nearest: |x_hat - x| <= scale/2 (1 + 2^-12) + a rounding of the result
    xh = oracle.decode(q, G, mn, scale)
    bound = np.repeat(scale, G).astype(np.float64) / 2 * (1 + 2.0 ** -12) + 2.0 ** -23 * np.repeat(np.maximum(np.abs(mn), np.abs(mx)), G)
    assert np.all(np.abs(xh.astype(np.float64) - x) <= bound)


def test_stochastic_rounding_is_unbiased_over_seeds():
    rng = np.random.default_rng(17)
    G, ng, K = 32, 8, 1024
    x = rng.standard_normal(G * ng).astype(np.float32)
    mn, mx, R = oracle.stats(x, G)
    bits = np.full(ng, 2, np.uint8)
    scale, inv = oracle.group_params(R, bits)
    acc = np.zeros(x.size, np.float64)
    for seed in range(K):
        acc += oracle.decode(oracle.codes(x, G, mn, inv, bits, seed=seed), G, mn, scale)
    s = np.repeat(scale, G).astype(np.float64)
    assert np.all(np.abs(acc / K - x) <= 4 * (s / 2) / np.sqrt(K) + 2.0 ** -16 * s + 1e-6)


def test_worked_vectors(worked):
    x = _ramp()
    inp = dict((r[0], r[1]) for r in worked["input"])
    assert HEX(x[[1, 17, 31]]) == [inp["x1"], inp["x17"], inp["x31"]]
    for b in (4, 2):
        sec = dict((r[0], r[1:]) for r in worked[f"width {b}"])
        c = oracle.compress(x, 32, [b], float(b))
        assert HEX(c.scale)[0] == sec["scale"][0]
        _, _, R = oracle.stats(x, 32)
        assert HEX(oracle.group_params(R, np.uint8([b]))[1])[0] == sec["inv"][0]
        assert list(c.codes) == [int(t) for t in sec["codes_stochastic"]]
        assert c.packed.tobytes().hex() == sec["packed_stochastic"][0]
        y = oracle.decompress(c)
        assert HEX(y[31])[0] == sec["xhat31_stochastic"][0]
        if "xhat17_stochastic" in sec:
            assert HEX(y[17])[0] == sec["xhat17_stochastic"][0]
        cn = oracle.compress(x, 32, [b], float(b), rounding=oracle.ROUND_NEAREST)
        assert cn.packed.tobytes().hex() == sec["packed_nearest"][0]


# ------------------------------------------------------------------ offsets and packing
def test_offsets_against_numpy_cumsum():
    rng = np.random.default_rng(2)
    for G in (32, 64, 256, 4096):
        bits = rng.choice(np.uint8([1, 2, 4, 8]), 1000)
        off = oracle.offsets(bits, G)
        assert off[0] == 0 and np.array_equal(off[1:], np.cumsum(bits.astype(np.uint64) * G // 8))


@pytest.mark.parametrize("G", [32, 64, 256])
def test_pack_against_numpy_packbits(G):
    rng = np.random.default_rng(G)
    ng = 50
    bits = rng.choice(np.uint8([1, 2, 4, 8]), ng)
    codes = np.concatenate([rng.integers(0, 2 ** int(b), G) for b in bits]).astype(np.uint8)
    packed = oracle.pack(codes, G, bits)
    assert packed.size == int((bits.astype(np.int64) * G // 8).sum())            # no padding anywhere
    stream = []
    for g, b in enumerate(bits):
        cg = codes[g * G:(g + 1) * G]
        stream.append(((cg[:, None] >> np.arange(int(b))) & 1).astype(np.uint8).reshape(-1))   # LSB first
    want = np.packbits(np.concatenate(stream), bitorder="little")
    assert np.array_equal(packed, want)
    assert np.array_equal(oracle.unpack(packed, codes.size, G, bits), codes)
    # little-endian 32-bit words: code i sits at shift (i*b) mod 32
    g = int(np.argmax(bits == 4)) if (bits == 4).any() else None
    if g is not None:
        off = oracle.offsets(bits, G)
        words = packed[int(off[g]):int(off[g + 1])].view("<u4")
        cg = codes[g * G:(g + 1) * G].astype(np.uint32).reshape(-1, 8)
        assert np.array_equal(words, (cg << (4 * np.arange(8, dtype=np.uint32))).sum(1).astype(np.uint32))


def test_pack_width8_is_identity():
    codes = np.random.default_rng(0).integers(0, 256, 128).astype(np.uint8)
    assert np.array_equal(oracle.pack(codes, 64, np.uint8([8, 8])), codes)


# ------------------------------------------------------------------ decode and whole path
def test_decode_closed_forms():
    mn, scale = np.float32([-1.25, 3.0]), np.float32([0.5, 0.0])
    q = np.zeros(64, np.uint8)
    q[1], q[2] = 3, 255
    y = oracle.decode(q, 32, mn, scale)
    assert y[0] == mn[0] and y[1] == np.float32(0.25) and y[2] == np.float32(-1.25 + 127.5)
    assert np.all(y[32:] == 3.0)                                   # scale 0: every code decodes to the minimum
    # fused multiply-add: one rounding (differs from multiply-then-add on this input)
    mn, scale = np.float32([1.0]), np.float32([1.0 + 2.0 ** -23])
    q = np.full(32, 3, np.uint8)
    want = np.float32(np.float64(3) * np.float64(scale[0]) + 1.0)
    assert oracle.decode(q, 32, mn, scale)[0] == want


@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
def test_constant_groups_round_trip_exactly(dtype):
    f32_to_bf16_bits = oracle.to_bf16_bits                       # the oracle's own conversion builds the oracle's input
    vals = np.float32([0.0, -0.0, 1.0, -3.5, 6.0, 1024.0, 2.0 ** -10, -65504.0])
    x = np.repeat(vals, 64)
    if dtype == "f16":
        a, kw = x.astype(np.float16), {}
    elif dtype == "bf16":
        a, kw = f32_to_bf16_bits(x), {"dtype": "bf16"}
    else:
        a, kw = x, {}
    c = oracle.compress(a, 64, [1, 2, 4, 8], 3.0, **kw)
    assert np.all(c.scale == 0) and np.all(c.codes == 0)
    y = oracle.decompress(c)
    # a constant group decodes to its minimum; -0.0 comes back as +0.0 (numerically equal)
    want = a.copy()
    if dtype == "f32":
        want[64:128] = 0.0
        assert np.array_equal(y.view(np.uint32), want.view(np.uint32))
    else:
        want = want.view(np.uint16).copy()
        want[64:128] = 0
        assert np.array_equal(y.view(np.uint16), want)


def test_whole_path_invariants_and_shard_invariance():
    rng = np.random.default_rng(21)
    G, We = 64, 1024
    n = We * 5 + G * 3                                             # ragged last window
    x = (rng.standard_normal(n) * np.repeat(10.0 ** rng.uniform(-2, 2, n // G), G)).astype(np.float32)
    for widths, beta in (((1, 2, 4, 8), 3.0), ((2, 4, 8), 4.0), ((1, 2, 4, 8), 2.5), ((4,), 4.0)):
        c = oracle.compress(x, G, widths, beta, window_elems=We, seed=5)
        W = We // G
        assert c.packed.size == int((c.bits.astype(np.int64) * G // 8).sum()) == int(c.window_offsets[-1])
        for w in range(-(-c.bits.size // W)):                      # average width per window within budget
            bw = c.bits[w * W:(w + 1) * W]
            assert bw.sum() <= (int(np.floor(beta * 256)) * bw.size) >> 8
        assert c.packed.size <= oracle.packed_capacity(n, G, We, beta)
        assert np.array_equal(oracle.unpack(c.packed, n, G, c.bits), c.codes)
        y = oracle.decompress(c)
        s = np.repeat(c.scale, G).astype(np.float64)
        assert np.all(np.abs(y.astype(np.float64) - x) <= s * (1 + 2.0 ** -12) + 2.0 ** -22 * np.abs(x) + 1e-30)
        # a window-aligned slice with elem_index_base set reproduces the same bytes
        lo, hi = 2 * We, 4 * We
        cs = oracle.compress(x[lo:hi], G, widths, beta, window_elems=We, seed=5, base=lo)
        assert np.array_equal(cs.bits, c.bits[lo // G:hi // G])
        assert np.array_equal(cs.packed, c.packed[int(c.window_offsets[2]):int(c.window_offsets[4])])
        assert np.array_equal(cs.mn, c.mn[lo // G:hi // G]) and np.array_equal(cs.scale, c.scale[lo // G:hi // G])


def test_compress_argument_checks():
    x = np.zeros(96, np.float32)
    with pytest.raises(oracle.OracleError):
        oracle.compress(x, 48, [4], 4.0)           # group size not a multiple of 32
    with pytest.raises(oracle.OracleError):
        oracle.compress(x, 64, [4], 4.0)           # numel not a multiple of the group size
    with pytest.raises(oracle.OracleError):
        oracle.compress(x, 32, [4], 3.0)           # budget below the smallest width


def test_relu_by_hand():
    """The producer fused in front of the compression (Sec. 3.2.3): negatives and -0 give +0."""
    a = np.array([-1.5, -0.0, 0.0, 2.5, -1e-30, 1e-30], np.float32)
    want = np.array([0.0, 0.0, 0.0, 2.5, 0.0, 1e-30], np.float32)
    assert np.array_equal(oracle.relu(a).view(np.uint32), want.view(np.uint32))
    assert np.array_equal(oracle.relu(a.astype(np.float16)).view(np.uint16), want.astype(np.float16).view(np.uint16))
    b = np.array([0xBFC0, 0x8000, 0x0000, 0x4020, 0x8001], np.uint16)          # bf16 -1.5, -0, +0, 2.5, a negative subnormal
    assert np.array_equal(oracle.relu(b, "bf16"), np.array([0, 0, 0, 0x4020, 0], np.uint16))


def test_relu6_by_hand():
    a = np.array([-1.5, -0.0, 0.0, 2.5, 6.0, 6.5, 1e30, -1e30], np.float32)
    want = np.array([0.0, 0.0, 0.0, 2.5, 6.0, 6.0, 6.0, 0.0], np.float32)
    assert np.array_equal(oracle.relu6(a).view(np.uint32), want.view(np.uint32))
    assert np.array_equal(oracle.relu6(a.astype(np.float16)).view(np.uint16), want.astype(np.float16).view(np.uint16))
    b = np.array([0xBFC0, 0x8000, 0x0000, 0x4020, 0x40C0, 0x40C1, 0x7F00], np.uint16)   # -1.5 -0 +0 2.5 6 6.03 huge
    assert np.array_equal(oracle.relu6(b, "bf16"), np.array([0, 0, 0, 0x4020, 0x40C0, 0x40C0, 0x40C0], np.uint16))


def test_gelu_and_its_derivative_against_closed_forms_and_a_library():
    """GELU(x) = x Phi(x): values that follow from the normal distribution, the two reflection identities, the
    derivative against a central difference, and torch's float64 GELU with its autograd derivative."""
    x = np.concatenate([np.linspace(-9, 9, 2001), [0.0, 1.0, -1.0, 1e-8, -1e-8, 20.0, -20.0]])
    y, d = oracle.gelu(x), oracle.gelu_grad(x)
    assert oracle.gelu([0.0])[0] == 0.0 and oracle.gelu_grad([0.0])[0] == 0.5
    assert abs(oracle.gelu([1.0])[0] - 0.8413447460685429) < 1e-15           # Phi(1)
    assert abs(oracle.gelu([-1.0])[0] + 0.15865525393145707) < 1e-15         # -(1 - Phi(1))
    assert np.allclose(y - oracle.gelu(-x), x, rtol=0, atol=1e-14)          # Phi(x) + Phi(-x) = 1
    assert np.allclose(d + oracle.gelu_grad(-x), 1.0, rtol=0, atol=1e-14)
    assert oracle.gelu([20.0])[0] == 20.0 and abs(oracle.gelu([-20.0])[0]) < 1e-80
    h = 1e-5
    num = (oracle.gelu(x + h) - oracle.gelu(x - h)) / (2 * h)
    assert np.allclose(num, d, rtol=0, atol=1e-9)
    torch = pytest.importorskip("torch")
    t = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    ty = torch.nn.functional.gelu(t)
    ty.sum().backward()
    assert np.allclose(ty.detach().numpy(), y, rtol=1e-13, atol=1e-15)    # (the library loses the far negative tail)
    assert np.allclose(t.grad.numpy(), d, rtol=0, atol=1e-14)


def test_packed_capacity_is_a_tight_bound():
    """The capacity formula (what the budget guarantees per window) against what the oracle's own compress produces: never
    exceeded on data with wildly different ranges, and met exactly when the budget is an allowed width."""
    rng = np.random.default_rng(2)
    for G, We, n_groups in ((32, 4096, 300), (256, 16384, 150), (1024, 8192, 21), (128, 16384, 129)):
        n = G * n_groups
        x = (rng.standard_normal(n) * np.repeat(10.0 ** rng.uniform(-4, 4, n_groups), G)).astype(np.float32)
        for beta in (1.0, 1.5, 2.0, 2.75, 3.0, 4.0, 5.5, 8.0):
            cap = oracle.packed_capacity(n, G, We, beta)
            got = oracle.compress(x, G, (1, 2, 4, 8), beta, window_elems=We).packed.size
            assert got <= cap, (G, We, beta)
            if beta in (1.0, 2.0, 4.0, 8.0):
                flat = oracle.compress(np.tile(np.linspace(-1, 1, G, dtype=np.float32), n_groups), G, (1, 2, 4, 8), beta,
                                       window_elems=We).packed.size
                assert flat == cap == n * int(beta) // 8
            # by hand: every window of n_w groups may spend floor(beta * 256) * n_w / 256 bits per group-unit
            W = We // G
            full, last = divmod(n_groups, W)
            q8 = int(np.floor(beta * 256))
            assert cap == full * ((q8 * W) >> 8) * G // 8 + ((q8 * last) >> 8) * G // 8
