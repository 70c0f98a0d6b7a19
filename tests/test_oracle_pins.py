"""Pins for the CPU oracle: closed forms, exact rational brute force, invariants and
special cases that reduce to library routines.  None of these restate the oracle's
own code path; a dropped term, wrong sign, off-by-one or transposed operand in the
oracle fails at least one of them."""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle import Params

RNG = np.random.default_rng(20260523)


# ----------------------------------------------------------------------------- Eq. 1

def test_mass_eq1_closed_form_dyadic():
    # weights that are exact in fp32 and in 36-bit fixed point: the mass is the exact ratio
    eps = 2.0 ** -10
    u = np.array([1.0, 3.0, -5.0, 0.0, 4.0 - eps, float("nan")], dtype=np.float32)
    A, SA, m = oracle.mass(u, eps)
    w = [Fraction(1) + Fraction(eps), Fraction(3) + Fraction(eps), Fraction(eps), Fraction(eps), Fraction(4),
         Fraction(eps)]
    tot = sum(w)
    for t in range(len(u)):
        assert Fraction(int(A[t]), SA) == w[t] / tot            # fixed point kept the ratios exactly
        assert m[t] == np.float32(float(w[t] / tot))            # one rounding to fp32
    assert int(A.sum()) == SA


def test_mass_sums_to_one_and_floor():
    for T in (1, 7, 4096, 131072):
        u = RNG.standard_normal(T).astype(np.float32)
        A, SA, m = oracle.mass(u, 1e-8)
        assert abs(float(m.astype(np.float64).sum()) - 1.0) <= T * 2.0 ** -24
        assert (m > 0).all() or (A == 0).any()
        assert int(A.max()) >= 2 ** 35 and int(A.max()) < 2 ** 36
        # negative scores carry only epsilon: all equal, and the smallest
        neg = u <= 0
        if neg.any():
            assert len(np.unique(m[neg])) == 1 and m[neg][0] == m.min()


def test_mass_scale_invariance_power_of_two():
    u = np.abs(RNG.standard_normal(257)).astype(np.float32) + 0.5
    A1, S1, m1 = oracle.mass(u, 0.0 + 2.0 ** -40)
    A2, S2, m2 = oracle.mass(u * np.float32(1024.0), 2.0 ** -30)
    assert (A1 == A2).all() and S1 == S2 and (m1 == m2).all()


# ----------------------------------------------------------------------------- cuts

def _brute_cuts(w, S):
    """Exact rational statement: b_k = min{t : c(t) >= k/S} with 1-based t, k = 1..S-1."""
    T = len(w)
    tot = sum(w)
    out = {0, T}
    for k in range(1, S):
        c = Fraction(0)
        for t in range(1, T + 1):
            c += w[t - 1]
            if c / tot >= Fraction(k, S):
                if 0 < t < T:
                    out.add(t)
                break
    return sorted(out)


@pytest.mark.parametrize("seed", range(40))
def test_cuts_match_exact_rational_brute_force(seed):
    rng = np.random.default_rng(seed)
    T = int(rng.integers(2, 65))
    S = int(rng.integers(1, 13))
    # small integer scores; eps = 2^-12 keeps every weight exact in fp32 and in fixed point
    eps = 2.0 ** -12
    u = rng.integers(-3, 40, size=T).astype(np.float32)
    if seed % 5 == 0:
        u[int(rng.integers(0, T))] = 4000.0          # one spike crossing several thresholds
    w = [Fraction(max(float(x), 0.0)) + Fraction(eps) for x in u]
    A, SA, m = oracle.mass(u, eps)
    Hm, _ = oracle.history_mass(A, SA, m, np.zeros(T, np.float32), 0.9, 1.0)
    got = oracle.cuts(oracle.prefix(Hm), S)
    assert got.tolist() == _brute_cuts(w, S)


def test_cuts_uniform_mass_closed_form():
    for T, S in ((100, 10), (4096, 8), (60, 3), (64, 64)):
        u = np.full(T, 0.25, dtype=np.float32)
        A, SA, m = oracle.mass(u, 1e-8)
        Hm, _ = oracle.history_mass(A, SA, m, np.zeros(T, np.float32), 0.9, 1.0)
        b = oracle.cuts(oracle.prefix(Hm), S)
        assert b.tolist() == [k * (T // S) for k in range(S + 1)]


def test_cuts_spike_dedup_and_single_segment():
    T = 50
    u = np.full(T, 1e-3, dtype=np.float32)
    u[20] = 100.0                                      # holds > 99.9 % of the mass
    A, SA, m = oracle.mass(u, 1e-8)
    Hm, _ = oracle.history_mass(A, SA, m, np.zeros(T, np.float32), 0.9, 1.0)
    C = oracle.prefix(Hm)
    assert oracle.cuts(C, 10).tolist() == [0, 21, T]   # one cut right after the spike, no empty segments
    assert oracle.cuts(C, 1).tolist() == [0, T]
    u[:] = 1e-3
    u[T - 1] = 100.0                                   # spike on the last token: its cut would be T, dropped
    A, SA, m = oracle.mass(u, 1e-8)
    Hm, _ = oracle.history_mass(A, SA, m, np.zeros(T, np.float32), 0.9, 1.0)
    assert oracle.cuts(oracle.prefix(Hm), 4).tolist() == [0, T]


# ----------------------------------------------------------------------------- merge / split

@pytest.mark.parametrize("seed", range(60))
def test_merge_split_invariants(seed):
    rng = np.random.default_rng(1000 + seed)
    T = int(rng.integers(1, 3000))
    n_cut = int(rng.integers(0, 30))
    raw = sorted({0, T} | {int(x) for x in rng.integers(1, max(T, 2), size=n_cut) if 0 < x < T})
    l_min = int(rng.integers(1, 40))
    l_max = int(rng.choice([0, 2 * l_min, 2 * l_min + 7, 256, 1000]))
    b = oracle.merge_split(np.array(raw, np.int32), l_min, l_max)
    lens = np.diff(b)
    assert b[0] == 0 and b[-1] == T and (lens > 0).all()             # cover, disjoint, ordered
    if T >= l_min and (l_max == 0 or l_max >= 2 * l_min):
        assert (lens >= l_min).all()
    if l_max > 0:
        assert (lens <= l_max).all()
    if l_max == 0:
        assert set(b.tolist()) <= set(raw)                            # merging only removes boundaries
    # every boundary that survives merging is a raw boundary; split pieces are near-equal
    merged = [x for x in b.tolist() if x in set(raw)]
    for a, e in zip(merged[:-1], merged[1:]):
        inner = [x for x in b.tolist() if a <= x <= e]
        pl = np.diff(inner)
        assert pl.max() - pl.min() <= 1
        assert list(pl) == sorted(pl, reverse=True)                   # larger pieces first
        if l_max > 0:
            assert len(pl) == -(-(e - a) // l_max) or (e - a) <= l_max


def test_merge_split_examples():
    # forward absorb: 5+5+10 -> 20 when l_min = 16; tail 4 folds left
    assert oracle.merge_split(np.array([0, 5, 10, 20, 40, 44], np.int32), 16, 0).tolist() == [0, 20, 44]
    # a single short segment stays
    assert oracle.merge_split(np.array([0, 7], np.int32), 16, 256).tolist() == [0, 7]
    # split 1000 with l_max 256 -> 4 pieces of 250
    assert oracle.merge_split(np.array([0, 1000], np.int32), 16, 256).tolist() == [0, 250, 500, 750, 1000]
    # 10 into l_max 4 -> ceil(10/4)=3 pieces 4,3,3
    assert oracle.merge_split(np.array([0, 10], np.int32), 1, 4).tolist() == [0, 4, 7, 10]


# ----------------------------------------------------------------------------- quotas

def _prefix_from_masses(masses, lens):
    """Cumulative integer mass with each segment's mass spread evenly over its tokens."""
    Hm = np.concatenate([np.full(L, M // L, dtype=np.uint64) for M, L in zip(masses, lens)])
    return np.cumsum(Hm, dtype=np.uint64)


def test_quota_formula_worked_example():
    # two long segments with masses 1:3, q_min = 1, budget 102: 1 + round(100/4) and 1 + round(300/4)
    lens = [400, 400]
    C = _prefix_from_masses([400 * 2 ** 20, 1200 * 2 ** 20], lens)
    q = oracle.quotas(C, np.array([0, 400, 800], np.int32), 1, 102)
    assert q.tolist() == [26, 76]
    # clipping: shares 1+3, 1+91 -> clipped to 10, 1+6; the deficit of 82 is handed out one token
    # per visit, heaviest segment with room first: 41 to each of the two long segments
    lens = [300, 10, 300]
    C = _prefix_from_masses([300 * 2 ** 20, 9000 * 2 ** 20, 600 * 2 ** 20], lens)
    q = oracle.quotas(C, np.array([0, 300, 310, 610], np.int32), 1, 103)
    assert q.tolist() == [45, 10, 48]
    # budget below the minima: minima are given up lightest first (ties: higher index)
    C = _prefix_from_masses([100 * 2 ** 20, 100 * 2 ** 20, 300 * 2 ** 20], [100, 100, 100])
    assert oracle.quotas(C, np.array([0, 100, 200, 300], np.int32), 2, 4).tolist() == [1, 1, 2]
    assert oracle.quotas(C, np.array([0, 100, 200, 300], np.int32), 2, 1).tolist() == [0, 0, 1]


@pytest.mark.parametrize("seed", range(60))
def test_quota_invariants(seed):
    rng = np.random.default_rng(2000 + seed)
    n_seg = int(rng.integers(1, 40))
    lens = rng.integers(1, 300, size=n_seg)
    masses = (rng.integers(1, 1000, size=n_seg).astype(np.int64) * lens) << 10
    C = _prefix_from_masses(masses.tolist(), lens.tolist())
    bounds = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    T = int(bounds[-1])
    q_min = int(rng.integers(0, 5))
    Bq = int(rng.integers(0, T + 1))
    q = oracle.quotas(C, bounds, q_min, Bq)
    qmin = np.minimum(q_min, lens)
    assert q.sum() == Bq                                        # quotas sum to the budget
    assert (q <= lens).all() and (q >= 0).all()
    if qmin.sum() <= Bq:
        assert (q >= qmin).all()                                 # minimum guarantee
        # proportional share up to rounding and the greedy correction
        M = np.diff(np.concatenate([[0], C[bounds[1:] - 1].astype(np.int64)]))
        share = (Bq - qmin.sum()) * M / M.sum()
        unclipped = q < lens
        if unclipped.all():
            assert np.abs(q - qmin - share).max() <= 1.5 + 1e-9


def test_quota_equal_segments_equal_quotas():
    lens = [100] * 8
    C = _prefix_from_masses([100 * 2 ** 20] * 8, lens)
    bounds = np.arange(0, 900, 100, dtype=np.int32)
    q = oracle.quotas(C, bounds, 1, 84)        # 84 = 8*10 + 4: the first four (ties by index) get one more
    assert q.tolist() == [11, 11, 11, 11, 10, 10, 10, 10]


def _quotas_of(masses, Bq, q_min=0, length=50):
    """Quotas of equally long segments (room everywhere) whose masses are in the given integer ratio."""
    lens = [length] * len(masses)
    C = _prefix_from_masses([m * length * 2 ** 20 for m in masses], lens)
    bounds = np.arange(0, length * (len(masses) + 1), length, dtype=np.int32)
    return oracle.quotas(C, bounds, q_min, Bq).tolist()


def test_quota_rounding_is_half_up_hand_worked():
    """Quota paragraph of the segmentation section, q_i = q_i^min + round(T_rem M_i / sum M): the rounding
    is to nearest with halves up.  Each case is worked by hand; floor, ceiling or halves-down would change
    the final quotas even after the adjustment step."""
    # masses 1:1:2, budget 2: shares 0.5, 0.5, 1 -> 1, 1, 1 (halves up), one too many; the surplus is taken
    # from the lightest segment, the higher index on a tie -> [1, 0, 1].  (Floor or halves-down: 0, 0, 1,
    # deficit 1 to the heaviest -> [0, 0, 2].)
    assert _quotas_of([1, 1, 2], 2) == [1, 0, 1]
    # masses 1:4, budget 3: shares 0.6 and 2.4 -> 1 and 2, already the budget.  (Ceiling: 1, 3 -> surplus from
    # the lightest -> [0, 3]; floor: 0, 2 -> deficit to the heaviest -> [0, 3].)
    assert _quotas_of([1, 4], 3) == [1, 2]
    # masses 1:2, budget 2: shares 2/3 and 4/3 -> 1, 1.  (Floor: 0, 1 -> [0, 2].)
    assert _quotas_of([1, 2], 2) == [1, 1]
    # with a minimum: q_min 2, masses 1:4, budget 7: remainder 3 shared as above on top of the minima
    assert _quotas_of([1, 4], 7, q_min=2) == [3, 4]


def test_quota_adjustment_order_hand_worked():
    """The adjustment that makes the quotas sum to the budget: a spare token goes to the heaviest segment
    first (lower index on a mass tie); a token too many is taken from the lightest first (higher index on
    a tie).  Room everywhere, so only the visiting order decides."""
    # masses 1:2:6, budget 2: shares 2/9, 4/9, 4/3 -> 0, 0, 1; the spare token goes to the heaviest
    assert _quotas_of([1, 2, 6], 2) == [0, 0, 2]
    # masses 1:2:2, budget 1: shares 0.2, 0.4, 0.4 -> 0, 0, 0; tie between the two heaviest -> lower index
    assert _quotas_of([1, 2, 2], 1) == [0, 1, 0]
    # masses 2:2:1, budget 1: the tie is between segments 0 and 1
    assert _quotas_of([2, 2, 1], 1) == [1, 0, 0]
    # surplus: masses 1:3, budget 2: shares 0.5, 1.5 -> 1, 2, one too many -> taken from the lightest
    assert _quotas_of([1, 3], 2) == [0, 2]
    # surplus with a tie among the lightest: masses 1:1:6, budget 4: shares 0.5, 0.5, 3 -> 1, 1, 3 -> the
    # higher index of the two lightest gives its token back
    assert _quotas_of([1, 1, 6], 4) == [1, 0, 3]
    # two spare tokens, three segments with room: one token per visit, heaviest first, then the next
    # masses 3:2:2 (sum 7), budget 5: shares 15/7 = 2.14, 10/7 = 1.43, 1.43 -> 2, 1, 1 -> spare 1 -> heaviest
    assert _quotas_of([3, 2, 2], 5) == [3, 1, 1]
    # masses 4:3:3 (sum 10), budget 4: shares 1.6, 1.2, 1.2 -> 2, 1, 1 = 4: nothing to adjust
    assert _quotas_of([4, 3, 3], 4) == [2, 1, 1]
    # masses 5:4:4 (sum 13), budget 5: shares 1.92, 1.54, 1.54 -> 2, 2, 2 = 6 -> surplus 1 from the lightest,
    # higher index on the tie
    assert _quotas_of([5, 4, 4], 5) == [2, 2, 1]


# ----------------------------------------------------------------------------- selection

def _key_order(g):
    """Library statement of the order: score descending, NaN last, ties by lower position."""
    g = np.asarray(g, dtype=np.float32)
    bits = g.view(np.uint32).astype(np.int64)
    key = np.where(bits >> 31 == 1, (~bits) & 0xFFFFFFFF, bits | 0x80000000)
    key = np.where(np.isnan(g), 0, key)
    return np.lexsort((np.arange(len(g)), -key))


@pytest.mark.parametrize("seed", range(20))
def test_single_segment_is_global_topk(seed):
    rng = np.random.default_rng(3000 + seed)
    T = int(rng.integers(2, 5000))
    Tk = int(rng.integers(1, T))
    g = rng.standard_normal(T).astype(np.float32)
    if seed % 3 == 0:
        g = np.round(g * 2) / 2                         # many ties
    if seed % 4 == 0:
        g[rng.integers(0, T, size=3)] = np.nan
        g[rng.integers(0, T, size=3)] = -0.0
        g[rng.integers(0, T, size=3)] = np.inf
    prm = Params(n_segments=1, l_min=1, l_max=0, q_min=0, n_sink=0, n_last=0, ema_beta=1.0)
    res = oracle.select_unit(np.abs(g), g, None, Tk, prm)
    assert res.n_seg == 1 and res.quotas.tolist() == [Tk] and res.n_backfill == 0
    assert res.keep_idx.tolist() == sorted(_key_order(g)[:Tk].tolist())
    # and against torch.topk on the values where no ties / NaN are involved
    if seed % 3 != 0 and seed % 4 != 0:
        assert set(res.keep_idx.tolist()) == set(torch.topk(torch.from_numpy(g), Tk).indices.tolist())


@pytest.mark.parametrize("seed", range(30))
def test_segmented_select_brute_force(seed):
    rng = np.random.default_rng(4000 + seed)
    T = int(rng.integers(8, 64))
    n_seg = int(rng.integers(1, 6))
    inner = sorted(set(rng.integers(1, T, size=n_seg - 1).tolist()))
    bounds = np.array([0] + inner + [T], np.int32)
    lens = np.diff(bounds)
    q = np.array([int(rng.integers(0, L + 1)) for L in lens], np.int32)
    g = rng.integers(-4, 5, size=T).astype(np.float32)           # heavy ties
    ns, nl = int(rng.integers(0, 3)), int(rng.integers(0, 4))
    chosen = set()
    for i in range(len(q)):
        a, b = int(bounds[i]), int(bounds[i + 1])
        chosen |= set(sorted(range(a, b), key=lambda t: (-g[t], t))[:q[i]])
    must = set(range(ns)) | set(range(T - nl, T))
    union = chosen | must
    Tk = int(q.sum()) + ns + nl
    if Tk > T:
        return
    rest = sorted(set(range(T)) - union, key=lambda t: (-g[t], t))
    want = sorted(union | set(rest[:Tk - len(union)]))
    keep, r = oracle.select(g, bounds, q, ns, nl, Tk)
    assert keep.tolist() == want and r == Tk - len(union)


# ----------------------------------------------------------------------------- EMA

def test_ema_closed_form_two_tokens():
    eps = 2.0 ** -30
    u = np.array([0.25, 0.75], np.float32)
    A, SA, m = oracle.mass(u, eps)
    Hm, c = oracle.history_mass(A, SA, m, np.array([0.5, 0.5], np.float32), 0.5, 0.5)
    np.testing.assert_allclose(c, [0.375, 0.625], rtol=1e-6)
    np.testing.assert_allclose(Hm.astype(np.float64) / 2 ** 36, [0.3125, 0.6875], rtol=1e-6)
    # lambda = 0: the credit becomes the current mass
    _, c0 = oracle.history_mass(A, SA, m, np.array([0.9, 0.1], np.float32), 0.0, 0.5)
    assert (c0 == m).all()


def test_ema_weights_and_normalised_credit_exact_rationals():
    """EMA paragraph of the segmentation section / Algorithm 1 step 2:
    c <- lambda c + (1 - lambda) m,  m_used = beta m + (1 - beta) normalize(c).
    Three tokens, lambda = 1/2, beta = 3/4, an old credit that does not sum to one.  The expected values are
    exact rationals; swapping beta with 1 - beta, or using c without normalising it, moves them by far more
    than the allowance (a few units of 2^-36 for the fixed-point images)."""
    eps = 2.0 ** -30
    u = np.array([1.0, 2.0, 5.0], np.float32)
    c_old = np.array([1.0, 0.25, 0.75], np.float32)               # sums to 2
    lam, beta = 0.5, 0.75
    A, SA, m = oracle.mass(u, eps)
    Hm, c = oracle.history_mass(A, SA, m, c_old, lam, beta)
    w = [Fraction(float(x)) + Fraction(eps) for x in u]
    W = sum(w)
    m_exact = [x / W for x in w]
    for t in range(3):
        assert m[t] == np.float32(float(m_exact[t]))
    # credit: both products are exact (powers of two), the sum is rounded once to fp32
    c_want = [np.float32(float(Fraction(1, 2) * Fraction(float(c_old[t])) + Fraction(1, 2) * Fraction(float(m[t]))))
              for t in range(3)]
    assert c.tolist() == [float(x) for x in c_want]
    assert abs(float(sum(Fraction(float(x)) for x in c)) - 1.5) < 1e-6          # not normalised: sums to 1 + 1/2
    C = sum(Fraction(float(x)) for x in c)
    for t in range(3):
        h = Fraction(3, 4) * m_exact[t] + Fraction(1, 4) * Fraction(float(c[t])) / C
        want = int(h * 2 ** 36)
        assert abs(int(Hm[t]) - want) <= 16, (t, int(Hm[t]), want)
        swapped = int((Fraction(1, 4) * m_exact[t] + Fraction(3, 4) * Fraction(float(c[t])) / C) * 2 ** 36)
        unnormalised = int((Fraction(3, 4) * m_exact[t] + Fraction(1, 4) * Fraction(float(c[t]))) * 2 ** 36)
        assert abs(swapped - want) > 2 ** 20 and abs(unnormalised - want) > 2 ** 20   # the pin can tell them apart
    # the mixed mass sums to one (beta + (1 - beta)) up to the floors
    assert abs(int(Hm.sum()) - 2 ** 36) <= 64


def test_must_keep_suffix_shrinks_before_sinks():
    """Algorithm 1 step 5: the must-keep set is inserted first; when the budget is short the recent suffix
    gives way before the sinks do."""
    assert oracle.must_keep(100, 10, 4, 16) == (4, 6)
    assert oracle.must_keep(100, 3, 4, 16) == (3, 0)
    assert oracle.must_keep(12, 11, 4, 16) == (4, 7)
    assert oracle.must_keep(100, 40, 4, 16) == (4, 16)
    assert oracle.must_keep(100, 4, 4, 16) == (4, 0)
    assert oracle.must_keep(100, 5, 0, 16) == (0, 5)
    # through the whole unit: budget 6 with 4 sinks and 16 recent tokens keeps the 4 sinks and the last 2
    T = 200
    u = np.linspace(1.0, 2.0, T).astype(np.float32)
    g = np.zeros(T, np.float32); g[50:150] = 1.0                    # the scores would choose the middle
    res = oracle.select_unit(u, g, None, 6, Params(n_segments=1, l_min=1, l_max=0, q_min=0, ema_beta=1.0))
    assert res.keep_idx.tolist() == [0, 1, 2, 3, T - 2, T - 1] and res.quotas.tolist() == [0]


def test_reciprocal_normalisation_matches_exact_division():
    """The oracle normalises by multiplying with the once-rounded reciprocal of the total.  Against the
    definition floor(A_t 2^36 / SA) evaluated with exact integers: the product A_t * fl(1 / SA) * 2^36 carries
    a relative error below 2^-52, i.e. below 2^-16 of one unit of the image for any A_t < 2^36, so the two can
    only differ when the exact quotient lies within 2^-16 of an integer: expected on none of 5000 random
    tokens, and never by more than one unit."""
    rng = np.random.default_rng(99)
    T = 5000
    u = np.exp(2.0 * rng.standard_normal(T)).astype(np.float32)
    A, SA, m = oracle.mass(u, 1e-8)
    Hm, _ = oracle.history_mass(A, SA, m, np.zeros(T, np.float32), 0.9, 1.0)
    exact = np.array([(int(a) << 36) // SA for a in A], dtype=np.int64)
    diff = Hm.astype(np.int64) - exact
    assert np.abs(diff).max() <= 1
    assert int((diff != 0).sum()) == 0
    # and the reported fp32 mass is the correctly rounded exact ratio except where double rounding bites
    m_exact = np.array([np.float32(float(Fraction(int(a), SA))) for a in A])
    assert int((m != m_exact).sum()) <= 2


def test_ema_unit_beta_is_ema_off_and_first_event_is_neutral():
    T, Tk = 1500, 400
    u = np.abs(RNG.standard_normal(T)).astype(np.float32) ** 3
    junk = RNG.random(T).astype(np.float32)
    off = oracle.select_unit(u, u, junk, Tk, Params(ema_beta=1.0))
    off2 = oracle.select_unit(u, u, None, Tk, Params(ema_beta=1.0, ema_lambda=0.3))
    assert (off.credit == junk).all()                                     # credit untouched
    assert off.bounds.tolist() == off2.bounds.tolist() and (off.keep_idx == off2.keep_idx).all()
    # first event, zero credit: normalize(c) = m, so the mixed mass equals m up to rounding
    A, SA, m = oracle.mass(u, 1e-8)
    H1, _ = oracle.history_mass(A, SA, m, np.zeros(T, np.float32), 0.9, 1.0)
    H9, c = oracle.history_mass(A, SA, m, np.zeros(T, np.float32), 0.9, 0.9)
    assert np.abs(H1.astype(np.int64) - H9.astype(np.int64)).max() <= 2 ** 36 * 1e-6 * m.max() + 2
    np.testing.assert_allclose(c, (np.float32(1.0) - np.float32(0.9)) * m, rtol=2e-7)
    # credit rows travel with their tokens, zero beyond the budget
    on = oracle.select_unit(u, u, None, Tk, Params(ema_beta=0.9))
    assert (on.credit[:Tk] == c[on.keep_idx]).all() and (on.credit[Tk:] == 0).all()


def test_ema_history_moves_boundaries_toward_past_mass():
    T = 1024
    past = np.zeros(T, np.float32); past[:128] = 1.0 / 128            # history says: mass at the front
    u = np.zeros(T, np.float32); u[-128:] = 1.0                        # now: mass at the back
    A, SA, m = oracle.mass(u, 1e-8)
    H_now, _ = oracle.history_mass(A, SA, m, past, 0.9, 1.0)
    H_mix, _ = oracle.history_mass(A, SA, m, past, 0.9, 0.5)
    first_now = oracle.cuts(oracle.prefix(H_now), 4)[1]
    first_mix = oracle.cuts(oracle.prefix(H_mix), 4)[1]
    assert first_now > T - 128 and first_mix <= 128


# ----------------------------------------------------------------------------- whole unit

@pytest.mark.parametrize("seed", range(25))
def test_unit_invariants(seed):
    rng = np.random.default_rng(5000 + seed)
    T = int(rng.integers(40, 6000))
    Tk = int(rng.integers(1, T))
    prm = Params(n_segments=int(rng.integers(1, 20)), l_min=int(rng.integers(1, 32)),
                 l_max=int(rng.choice([0, 64, 256])), q_min=int(rng.integers(0, 4)),
                 n_sink=int(rng.integers(0, 6)), n_last=int(rng.integers(0, 20)),
                 ema_beta=float(rng.choice([1.0, 0.9])))
    if prm.l_max and prm.l_max < 2 * prm.l_min:
        prm.l_max = 2 * prm.l_min
    u = (np.abs(rng.standard_normal(T)) ** 4).astype(np.float32)
    g = rng.standard_normal(T).astype(np.float32)
    res = oracle.select_unit(u, g, None, Tk, prm)
    k = res.keep_idx
    assert len(k) == Tk and (np.diff(k) > 0).all() and k[0] >= 0 and k[-1] < T
    ns, nl = oracle.must_keep(T, Tk, prm.n_sink, prm.n_last)
    assert set(range(ns)) <= set(k.tolist()) and set(range(T - nl, T)) <= set(k.tolist())
    assert ns == min(prm.n_sink, Tk) and nl == min(prm.n_last, Tk - ns, T - ns)   # sinks before suffix
    assert res.quotas.sum() == Tk - ns - nl
    lens = np.diff(res.bounds)
    assert res.bounds[0] == 0 and res.bounds[-1] == T and (res.quotas <= lens).all()
    kept_per_seg = np.histogram(k, bins=res.bounds)[0]
    assert (kept_per_seg >= res.quotas).all()            # each segment keeps at least its quota
    if np.minimum(prm.q_min, lens).sum() <= Tk - ns - nl:
        assert (kept_per_seg >= np.minimum(prm.q_min, lens)).all()   # no region wiped out


def test_segment_count_smoke_range_at_paper_operating_point():
    # Attention-like mass at T ~ 1.1-1.5 K, segment mass 0.1, lengths 16/256: the paper's
    # diagnostics table reports 7-10 segments of mean length 131-148.  Weak pin: a range.
    for seed in range(8):
        rng = np.random.default_rng(6000 + seed)
        T = int(rng.integers(1100, 1500))
        u = np.exp(1.5 * rng.standard_normal(T)).astype(np.float32)
        u[:4] += 50.0
        u[-64:] *= 4.0
        res = oracle.select_unit(u, u, None, 512, Params())
        assert 5 <= res.n_seg <= 14, res.n_seg
        assert 80 <= T / res.n_seg <= 260


# ----------------------------------------------------------------------------- gather

def test_gather_equals_dense_indexing():
    rng = np.random.default_rng(7)
    L, P, page, H, D, T, Tk = 2, 40, 16, 3, 128, 150, 37
    k = rng.integers(0, 65536, size=(L, P, page, H, D)).astype(np.uint16)
    v = rng.integers(0, 65536, size=(L, P, page, H, D)).astype(np.uint16)
    perm = rng.permutation(P).astype(np.int32)
    table = perm[:10]
    dst = perm[10:13]
    k0, v0 = k.copy(), v.copy()
    slots = table[np.arange(T) // page] * page + np.arange(T) % page
    for l in range(L):
        for h in range(H):
            keep = np.sort(rng.choice(T, size=Tk, replace=False)).astype(np.int32)
            dense_k = k0[l].reshape(-1, H, D)[slots, h]          # [T][D] dense view of this head
            dense_v = v0[l].reshape(-1, H, D)[slots, h]
            oracle.gather_unit(k, v, l, h, table, dst, keep)
            dslots = dst[np.arange(Tk) // page] * page + np.arange(Tk) % page
            assert (k[l].reshape(-1, H, D)[dslots, h] == dense_k[keep]).all()
            assert (v[l].reshape(-1, H, D)[dslots, h] == dense_v[keep]).all()
    # source pages untouched, nothing outside the destination pages written
    mask = np.ones(P, bool); mask[dst] = False
    assert (k[:, mask] == k0[:, mask]).all() and (v[:, mask] == v0[:, mask]).all()


# ----------------------------------------------------------------------------- scorers

def _tiny_cache(rng, L=1, H=2, T=200, P=20, D=128):
    x = torch.from_numpy(rng.standard_normal((L, P, 16, H, D)).astype(np.float32)).to(torch.bfloat16)
    pages = x.view(torch.int16).numpy().view(np.uint16)
    table = rng.permutation(P).astype(np.int32)[: (T + 15) // 16]
    slots = table[np.arange(T) // 16] * 16 + np.arange(T) % 16
    dense = x.float().double().reshape(L, -1, H, D)[:, slots]     # [L][T][H][D]
    return pages, table, dense


def test_tova_single_row_is_library_softmax():
    rng = np.random.default_rng(11)
    pages, table, dense = _tiny_cache(rng)
    T, D = dense.shape[1], 128
    q = torch.from_numpy(rng.standard_normal((1, 1, D)).astype(np.float32)).to(torch.bfloat16)
    for h in range(2):
        u = oracle.score_tova(pages, 0, h, table, T, q.view(torch.int16).numpy().view(np.uint16), 1, 1, True)
        ref = torch.softmax(dense[0, :, h] @ q.double().reshape(D) / np.sqrt(D), dim=0)
        np.testing.assert_allclose(u, ref.numpy(), rtol=2e-7, atol=0)
        assert abs(float(u.astype(np.float64).sum()) - 1.0) < 1e-6


def test_tova_permuting_the_tokens_permutes_the_scores():
    """With one query that sees every token the usage is a softmax over the cache: a function of the set of
    keys, so storing the same keys in another order returns the same scores in that order."""
    rng = np.random.default_rng(14)
    pages, table, dense = _tiny_cache(rng, T=192, P=16)
    T, D, H = 192, 128, 2
    q = torch.from_numpy(rng.standard_normal((1, 1, D)).astype(np.float32)).to(torch.bfloat16)
    qn = q.view(torch.int16).numpy().view(np.uint16)
    perm = rng.permutation(T)
    slots = table[np.arange(T) // 16] * 16 + np.arange(T) % 16
    flat = pages.reshape(1, -1, H, D)
    moved = np.zeros_like(flat)
    table2 = np.arange(T // 16, dtype=np.int32)                       # the permuted cache lives in pages 0..11
    moved[0, np.arange(T)] = flat[0, slots[perm]]                     # new position i holds old token perm[i]
    moved = moved.reshape(pages.shape)
    for h in range(H):
        u = oracle.score_tova(pages, 0, h, table, T, qn, 1, 1, True)
        u2 = oracle.score_tova(moved, 0, h, table2, T, qn, 1, 1, True)
        np.testing.assert_allclose(u2, u[perm], rtol=1e-6, atol=0)
        assert not np.allclose(u2, u, rtol=1e-3)                      # (the permutation did move something)


def test_tova_window_group_mean_and_causal_padding():
    rng = np.random.default_rng(12)
    pages, table, dense = _tiny_cache(rng, T=120, P=12)
    T, D, G, W = 120, 128, 3, 5
    q = torch.from_numpy((rng.standard_normal((G, W, D)) * 2).astype(np.float32)).to(torch.bfloat16)
    qn = q.view(torch.int16).numpy().view(np.uint16)
    K = dense[0, :, 1]
    # non-causal: plain mean of G*W library softmaxes
    u = oracle.score_tova(pages, 0, 1, table, T, qn, G, W, False)
    ref = torch.softmax(q.double().reshape(G * W, D) @ K.T / np.sqrt(D), dim=1).mean(0)
    np.testing.assert_allclose(u, ref.numpy(), rtol=3e-7)
    # causal: window query j sees tokens t <= T-W+j; unseen pairs take the window maximum
    u = oracle.score_tova(pages, 0, 1, table, T, qn, G, W, True)
    probs = torch.zeros(G, W, T, dtype=torch.float64)
    for j in range(W):
        n = T - W + j + 1
        probs[:, j, :n] = torch.softmax(q.double()[:, j] @ K[:n].T / np.sqrt(D), dim=1)
    pmax = probs.max()
    seen = torch.arange(T)[None, :] <= (T - W + torch.arange(W))[:, None]
    ref = torch.where(seen[None], probs, pmax).mean((0, 1))
    np.testing.assert_allclose(u, ref.numpy(), rtol=3e-7)
    assert np.allclose(u[: T - W + 1], probs.mean((0, 1))[: T - W + 1].numpy(), rtol=3e-7)
    # identical rows collapse to one softmax
    q1 = q[:1, :1].expand(G, W, D).contiguous()
    u1 = oracle.score_tova(pages, 0, 1, table, T, q1.view(torch.int16).numpy().view(np.uint16), G, W, False)
    r1 = torch.softmax(K @ q1.double()[0, 0] / np.sqrt(D), dim=0)
    np.testing.assert_allclose(u1, r1.numpy(), rtol=3e-7)


def test_keydiff_is_negative_cosine_to_mean_key():
    rng = np.random.default_rng(13)
    pages, table, dense = _tiny_cache(rng, T=333, P=30)
    for h in range(2):
        K = dense[0, :, h]
        g = oracle.score_keydiff(pages, 0, h, table, 333)
        ref = -torch.nn.functional.cosine_similarity(K, K.mean(0, keepdim=True), dim=1)
        np.testing.assert_allclose(g, ref.numpy(), rtol=1e-6, atol=1e-7)
    # closed forms: identical keys -> -1; a key orthogonal to the mean -> 0; opposite -> +1
    L, P, H, D = 1, 1, 1, 128
    x = torch.zeros((L, P, 16, H, D))
    x[0, 0, :, 0, 0] = 2.0
    pg = x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    g = oracle.score_keydiff(pg, 0, 0, np.array([0], np.int32), 16)
    assert (g == -1.0).all()
    x[0, 0, 3, 0, :] = 0.0; x[0, 0, 3, 0, 5] = 7.0             # orthogonal to the mean direction... almost
    x[0, 0, 4, 0, 0] = -0.5                                     # opposite
    pg = x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    g = oracle.score_keydiff(pg, 0, 0, np.array([0], np.int32), 16)
    mu = x[0, 0, :, 0].double().mean(0)
    assert abs(g[3] + float(7.0 * mu[5] / (7.0 * mu.norm()))) < 1e-6
    assert g[4] > 0.9 and g[0] < -0.9


def _u16(t):
    return t.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def _expected_logits(K, mean, cov):
    """l_t = mu.k_t / sqrt(D) + k_t^T Sigma k_t / (2 D), by library matrix products in fp64."""
    D = K.shape[1]
    return K @ mean / np.sqrt(D) + ((K @ cov) * K).sum(1) / (2 * D)


def test_expected_attention_is_the_gaussian_expectation_of_the_attention_weight():
    """The logit the scorer exponentiates is log E[exp(q.k / sqrt(D))] for q ~ N(mu, Sigma) (the idea the paper's
    expected-attention scorer is named for): checked against a Monte-Carlo mean over sampled queries, which knows
    nothing of the closed form.  With uniform values the score is softmax(logit) + eps times the value norm."""
    rng = np.random.default_rng(31)
    T, D = 48, 128
    pages_k, table, dense = _tiny_cache(rng, T=T, P=4, H=1)
    K = dense[0, :, 0].numpy() * 0.5
    pages_k = _u16(torch.from_numpy(pages_k.view(np.int16)).view(torch.bfloat16).float() * 0.5)   # keys halved: tame variance
    A = rng.standard_normal((D, 6)) * 0.6
    cov = torch.from_numpy(A @ A.T + 0.25 * np.eye(D)).to(torch.bfloat16)
    mean = rng.standard_normal(D).astype(np.float32) * 0.5
    cov64 = cov.double().numpy()
    # values: every row the same vector of norm 5 (3, 4, 0, ...)
    v = torch.zeros((1, 4, 16, 1, D)); v[..., 0] = 3.0; v[..., 1] = 4.0
    eps = 0.01
    g = oracle.score_expected(pages_k, _u16(v), 0, 0, table, T, mean[None], _u16(cov)[None], eps)
    # Monte Carlo: q = mu + C z with C C^T = Sigma (Sigma as the scorer reads it, after rounding to bf16, symmetrised)
    sym = (cov64 + cov64.T) / 2
    w, U = np.linalg.eigh(sym)
    C = U * np.sqrt(np.clip(w, 0, None))
    n = 400_000
    z = rng.standard_normal((n, D))
    q = mean.astype(np.float64) + z @ C.T
    mc = np.exp(q @ K.T / np.sqrt(D))                    # [n][T]
    est, se = mc.mean(0), mc.std(0) / np.sqrt(n)
    closed = np.exp(_expected_logits(K, mean.astype(np.float64), sym))
    assert (np.abs(est - closed) < 6 * se + 1e-12).all()
    assert (se / closed < 0.02).all()                    # (the estimate is sharp enough to tell 1/2 from 1 in the quadratic term)
    ref = (closed / closed.sum() + eps) * 5.0
    np.testing.assert_allclose(g, ref, rtol=2e-6)


def test_expected_attention_special_cases():
    rng = np.random.default_rng(32)
    T, D, H = 150, 128, 2
    pages_k, table, dense = _tiny_cache(rng, T=T, P=12, H=H)
    pages_v, _, dense_v = _tiny_cache(np.random.default_rng(33), T=T, P=12, H=H)
    slots = table[np.arange(T) // 16] * 16 + np.arange(T) % 16
    V = torch.from_numpy(pages_v.view(np.int16)).view(torch.bfloat16).double().reshape(1, -1, H, D)[0, slots]   # values through this cache's table
    h = 1
    K = dense[0, :, h].numpy()
    vnorm = V[:, h].norm(dim=1).numpy()
    mu = torch.from_numpy(rng.standard_normal(D).astype(np.float32)).to(torch.bfloat16)
    zero = np.zeros((1, D, D), np.uint16)
    # zero covariance: the softmax of one query, i.e. the TOVA score of the query mu (another routine of the oracle,
    # itself pinned to the library softmax), times the value norm
    g0 = oracle.score_expected(pages_k, pages_v, 0, h, table, T, mu.float().numpy()[None], zero, 0.0)
    u = oracle.score_tova(pages_k, 0, h, table, T, _u16(mu).reshape(1, 1, D), 1, 1, False)
    np.testing.assert_allclose(g0, u.astype(np.float64) * vnorm, rtol=3e-6)
    # eps is added before the value norm multiplies
    g1 = oracle.score_expected(pages_k, pages_v, 0, h, table, T, mu.float().numpy()[None], zero, 0.25)
    np.testing.assert_allclose(g1, (u.astype(np.float64) + 0.25) * vnorm, rtol=3e-6)
    # isotropic covariance s^2 I: logit = mu.k / sqrt(D) + s^2 |k|^2 / (2 D)
    s2 = 0.75
    iso = _u16(torch.eye(D) * s2)[None]
    g2 = oracle.score_expected(pages_k, pages_v, 0, h, table, T, mu.float().numpy()[None], iso, 0.0)
    lg = K @ mu.double().numpy() / np.sqrt(D) + s2 * (K * K).sum(1) / (2 * D)
    ref = np.exp(lg - lg.max()); ref /= ref.sum()
    np.testing.assert_allclose(g2, ref * vnorm, rtol=3e-6)
    # a general covariance against library matrix products; only its symmetric part matters
    Cm = torch.from_numpy(rng.standard_normal((D, D)) * 0.05).to(torch.bfloat16)
    g3 = oracle.score_expected(pages_k, pages_v, 0, h, table, T, mu.float().numpy()[None], _u16(Cm)[None], 0.0)
    lg = _expected_logits(K, mu.double().numpy(), Cm.double().numpy())
    ref = np.exp(lg - lg.max()); ref /= ref.sum()
    np.testing.assert_allclose(g3, ref * vnorm, rtol=3e-6)
    g3t = oracle.score_expected(pages_k, pages_v, 0, h, table, T, mu.float().numpy()[None], _u16(Cm.T.contiguous())[None], 0.0)
    np.testing.assert_allclose(g3t, g3, rtol=1e-6)
    # group: the mean of the heads' softmaxes (not a softmax of mean logits); identical heads collapse
    mu_b = torch.from_numpy(rng.standard_normal(D).astype(np.float32) * 3).to(torch.bfloat16)
    gg = oracle.score_expected(pages_k, pages_v, 0, h, table, T, np.stack([mu.float().numpy(), mu_b.float().numpy()]),
                               np.concatenate([iso, zero]), 0.0)
    ub = oracle.score_tova(pages_k, 0, h, table, T, _u16(mu_b).reshape(1, 1, D), 1, 1, False)
    np.testing.assert_allclose(gg, (g2 / vnorm + ub) / 2 * vnorm, rtol=5e-6)
    same = oracle.score_expected(pages_k, pages_v, 0, h, table, T, np.stack([mu.float().numpy()] * 3),
                                 np.concatenate([iso] * 3), 0.0)
    np.testing.assert_allclose(same, g2, rtol=1e-6)


# ----------------------------------------------------------------------------- usage smoothing, decoupled signals

def test_usage_smoothing_hand_computed_and_library_pooling():
    # small integers: every partial sum and quotient by 4-bit-exact divisors is exact
    u = np.array([4, 8, 0, 12, 16, 4], np.float32)
    assert oracle.smooth_usage(u, 1).tolist() == u.tolist()
    assert oracle.smooth_usage(u, 3).tolist() == [np.float32(x) / np.float32(3) for x in (12, 12, 20, 28, 32, 20)]
    want5 = [np.float32(x) / np.float32(5) for x in (12, 24, 40, 40, 32, 32)]
    assert oracle.smooth_usage(u, 5).tolist() == want5
    # a window wider than the sequence still divides by k
    assert oracle.smooth_usage(np.array([3, 6], np.float32), 7).tolist() == [np.float32(9) / np.float32(7)] * 2
    # against a library's zero-padded average pooling (stride 1, padding k // 2)
    rng = np.random.default_rng(5)
    x = np.exp(rng.standard_normal(1000)).astype(np.float32)
    for k in (3, 5, 7, 9):
        ref = torch.nn.functional.avg_pool1d(torch.from_numpy(x).double()[None, None], k, stride=1, padding=k // 2)[0, 0]
        np.testing.assert_allclose(oracle.smooth_usage(x, k), ref.numpy(), rtol=2e-6)
    with pytest.raises(ValueError):
        oracle.smooth_usage(x, 4)


def _event_inputs(rng, T=300, W=4, Hq=4, H=2):
    pages, table, dense = _tiny_cache(rng, T=T, P=T // 16 + 12)
    q = torch.randn((1, 1, Hq, W, 128)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    dst = np.arange(T // 16 + 2, T // 16 + 2 + 4, dtype=np.int32)[None]
    return pages, table, q, dst


def test_smoothing_changes_the_mass_only_and_decoupled_signals_split_roles():
    """Smoothing and a separate usage signal act on the mass (hence on segments and quotas);
    inside a segment tokens are still ranked by the base score g."""
    rng = np.random.default_rng(31)
    torch.manual_seed(31)
    T, Tk = 300, 64
    pages, table, q, dst = _event_inputs(rng, T=T)
    prm = Params(n_segments=6, l_min=8, l_max=0, q_min=1, n_sink=2, n_last=4, ema_lambda=0.9, ema_beta=1.0, eps=1e-8)
    lens = np.array([T], np.int32)
    tab = table[None].copy()
    credit = np.zeros((1, 1, 2, T), np.float32)

    def run(**kw):
        return oracle.compress(pages.copy(), pages.copy(), tab.copy(), lens.copy(), q, credit.copy(), Tk, prm,
                               kw.pop("scorer", oracle.SCORER_TOVA), dst, n_q_heads=4, do_gather=False, **kw)

    base = run()
    pooled = run(pool_kernel=5)
    for unit in base:
        g = base[unit].scores
        assert (pooled[unit].scores == g).all()                                  # g is not smoothed
        assert (pooled[unit].usage == oracle.smooth_usage(g, 5)).all()
        _, _, m = oracle.mass(oracle.smooth_usage(g, 5), prm.eps)
        assert (pooled[unit].mass == m).all()
        # selection inside each segment of the pooled run is the top-q of g there
        r = pooled[unit]
        for i in range(r.n_seg):
            a, b = r.bounds[i], r.bounds[i + 1]
            order = sorted(range(a, b), key=lambda t: (-g[t], t))[: r.quotas[i]]
            assert set(order) <= set(r.keep_idx.tolist())
    # decoupled: mass from the window attention, ranking from the key-only score
    dec = run(scorer=oracle.SCORER_KEYDIFF, decoupled=True)
    kd = run(scorer=oracle.SCORER_KEYDIFF)
    for unit in base:
        assert (dec[unit].usage == base[unit].scores).all() and (dec[unit].scores == kd[unit].scores).all()
        assert (dec[unit].bounds == base[unit].bounds).all() and (dec[unit].quotas == base[unit].quotas).all()
        r, g = dec[unit], kd[unit].scores
        for i in range(r.n_seg):
            a, b = r.bounds[i], r.bounds[i + 1]
            order = sorted(range(a, b), key=lambda t: (-g[t], t))[: r.quotas[i]]
            assert set(order) <= set(r.keep_idx.tolist())
    # the expected-attention scorer as base score: alone (u = g) and with the window attention as the mass signal
    stats = dict(q_mean=rng.standard_normal((1, 1, 4, 128)).astype(np.float32),
                 q_cov=_u16(torch.from_numpy(rng.standard_normal((1, 1, 4, 128, 128)) * 0.05)), score_eps=0.01)
    ex = run(scorer=oracle.SCORER_EXPECTED, **stats)
    exd = run(scorer=oracle.SCORER_EXPECTED, decoupled=True, **stats)
    for (l, b, h) in base:
        want = oracle.score_expected(pages, pages, l, h, tab[b], T, stats["q_mean"][l, b, 2 * h:2 * h + 2],
                                     stats["q_cov"][l, b, 2 * h:2 * h + 2], 0.01)
        assert (ex[(l, b, h)].scores == want).all() and (ex[(l, b, h)].usage == want).all()
        assert (exd[(l, b, h)].scores == want).all() and (exd[(l, b, h)].usage == base[(l, b, h)].scores).all()
        assert (exd[(l, b, h)].bounds == base[(l, b, h)].bounds).all()
    # an external usage signal plays the same role
    ext_g = rng.standard_normal((1, 1, 2, T)).astype(np.float32)
    ext_u = np.exp(rng.standard_normal((1, 1, 2, T))).astype(np.float32)
    both = run(scorer=oracle.SCORER_EXTERNAL, ext_scores=ext_g, ext_usage=ext_u)
    only_u = run(scorer=oracle.SCORER_EXTERNAL, ext_scores=ext_u)
    for unit in both:
        assert (both[unit].bounds == only_u[unit].bounds).all() and (both[unit].quotas == only_u[unit].quotas).all()
        assert (both[unit].mass == only_u[unit].mass).all()


# ----------------------------------------------------------------------------- component ablations

def test_ablation_fixed_length_segments_and_length_proportional_quotas():
    """The two component ablations of the paper's ablation table: segments of equal length, and a
    budget shared by segment length instead of mass."""
    rng = np.random.default_rng(77)
    T, Tk, S = 1200, 300, 10
    u = np.exp(2.0 * rng.standard_normal(T)).astype(np.float32)
    base = dict(n_segments=S, l_min=1, l_max=0, q_min=1, n_sink=0, n_last=0, ema_beta=1.0)
    # fixed-length: S divides T, so every boundary is k T / S whatever the mass looks like
    r = oracle.select_unit(u, u, None, Tk, Params(fixed_segments=True, **base))
    assert r.bounds.tolist() == [k * T // S for k in range(S + 1)]
    r2 = oracle.select_unit(np.roll(u, 123), None, None, Tk, Params(fixed_segments=True, **base))
    assert r2.bounds.tolist() == r.bounds.tolist() and r2.quotas.tolist() != r.quotas.tolist()  # quotas still follow the mass
    # S does not divide T: floor(k T / S), then the usual merge of short pieces
    r3 = oracle.select_unit(u[:1003], None, None, Tk, Params(fixed_segments=True, **base))
    assert r3.bounds.tolist() == [k * 1003 // S for k in range(S + 1)]
    r4 = oracle.select_unit(u[:1003], None, None, Tk, Params(fixed_segments=True, **{**base, "l_min": 150}))
    assert r4.bounds[0] == 0 and r4.bounds[-1] == 1003 and (np.diff(r4.bounds) >= 150).all()
    # length-proportional quotas: equal lengths -> equal quotas, however skewed the mass is
    r5 = oracle.select_unit(u, None, None, Tk, Params(fixed_segments=True, uniform_quotas=True, **base))
    assert r5.quotas.tolist() == [Tk // S] * S
    # with mass-quantile segments of different lengths: quotas follow the lengths within one token and sum to the budget
    r6 = oracle.select_unit(u, None, None, Tk, Params(uniform_quotas=True, **base))
    L = np.diff(r6.bounds)
    assert r6.quotas.sum() == Tk and (np.abs(r6.quotas - Tk * L / T) <= 1.0 + 1e-9).all()
    assert (r6.bounds == oracle.select_unit(u, None, None, Tk, Params(**base)).bounds).all()   # segments unchanged
    # inside a segment the pick is still the top-q of the scores
    for i in range(r6.n_seg):
        a, b = r6.bounds[i], r6.bounds[i + 1]
        top = sorted(range(a, b), key=lambda t: (-u[t], t))[: r6.quotas[i]]
        assert set(top) <= set(r6.keep_idx.tolist())


def test_retained_iou_closed_forms():
    Tk = 8
    assert oracle.retained_iou(np.arange(Tk), Tk, Tk) == np.float32(1.0)                 # the same set twice
    assert oracle.retained_iou(np.arange(Tk, 2 * Tk), Tk, Tk) == np.float32(0.0)         # only new tokens kept
    keep = np.array([0, 2, 4, 6, 8, 9, 10, 11])                                          # four old, four new
    assert oracle.retained_iou(keep, Tk, Tk) == np.float32(4) / np.float32(12)
    assert oracle.retained_iou(keep, 0, Tk) == np.float32(0.0)                           # no previous event
    assert oracle.retained_iou(keep, 5, Tk) == np.float32(3) / np.float32(10)            # a smaller previous budget


# ----------------------------------------------------------------------------- stored results

def test_oracle_reproduces_the_stored_small_case():
    """tests/golden/select_unit_small.json was written by tests/golden/make_golden.py from the oracle alone; an
    accidental change to the oracle's arithmetic or tie rules shows up here."""
    import importlib.util
    import json
    import os
    here = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(here, "make_golden.py"))
    mg = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mg)
    gold = json.load(open(os.path.join(here, "select_unit_small.json")))
    prm = Params(**gold["params"])
    credit = np.zeros(gold["T"], np.float32)
    for event, want in enumerate(gold["events"]):
        n = want["n_tokens"]
        u = mg.scores(event, n)
        r = oracle.select_unit(u, u, credit[:n], gold["Tk"], prm)
        assert r.bounds.tolist() == want["bounds"] and r.quotas.tolist() == want["quotas"]
        assert r.keep_idx.tolist() == want["keep_idx"] and r.n_backfill == want["n_backfill"]
        assert [int(v) for v in r.mass[:8].view(np.uint32)] == want["mass_bits_first8"]
        assert [int(v) for v in r.credit[:8].view(np.uint32)] == want["credit_bits_first8"]
        credit = np.zeros(gold["Tk"] + gold["append"], np.float32)
        credit[: gold["Tk"]] = r.credit[: gold["Tk"]]
