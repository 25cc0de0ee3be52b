"""Pins for the oracle's RNG, advantages, selection and compaction (CPU only)."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import SEL_DET, SEL_RPC, SEL_URS, compact, grpo_adv, philox4x32_10, select
from oracle.nat_oracle import urs_threshold

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ Philox
def _kat():
    rows = []
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            v = [int(x, 16) for x in line.split()]
            rows.append((v[:4], v[4:6], v[6:]))
    return rows


def _philox_bigint(c, k):
    """Independent restatement with Python integers (arbiter for both sides)."""
    c = list(c)
    k = list(k)
    for r in range(10):
        if r:
            k = [(k[0] + 0x9E3779B9) % 2**32, (k[1] + 0xBB67AE85) % 2**32]
        a = 0xD2511F53 * c[0]
        b = 0xCD9E8D57 * c[2]
        c = [(b >> 32) ^ c[1] ^ k[0], b % 2**32, (a >> 32) ^ c[3] ^ k[1], a % 2**32]
    return c


def test_philox_known_answers():
    rows = _kat()
    assert len(rows) == 3
    for c, k, want in rows:
        got = [int(x) for x in philox4x32_10(*c, *k)]
        assert got == want
        assert _philox_bigint(c, k) == want


def test_philox_vectorised_matches_bigint():
    rng = np.random.default_rng(5)
    C = rng.integers(0, 2**32, size=(64, 4), dtype=np.uint64)
    K = rng.integers(0, 2**32, size=(64, 2), dtype=np.uint64)
    out = philox4x32_10(C[:, 0], C[:, 1], C[:, 2], C[:, 3], K[:, 0], K[:, 1])
    for j in range(64):
        want = _philox_bigint([int(x) for x in C[j]], [int(x) for x in K[j]])
        assert [int(o[j]) for o in out] == want


# --------------------------------------------------------------- advantages
def test_adv_binary_closed_form():
    # k ones among G: mu = k/G, sigma = sqrt(k (G-k)) / G   (Eq. grpo-adv)
    G, eps = 8, 1e-6
    for k in range(G + 1):
        R = np.array([1.0] * k + [0.0] * (G - k), dtype=np.float32)
        adv = grpo_adv(R, 1, G, eps)
        sigma = math.sqrt(k * (G - k)) / G
        hi = (1 - k / G) / (sigma + eps)
        lo = (0 - k / G) / (sigma + eps)
        want = np.array([hi] * k + [lo] * (G - k))
        if k in (0, G):
            assert np.all(adv == 0.0)
        else:
            np.testing.assert_allclose(adv, want, rtol=2e-7)


def test_adv_matches_numpy_zscore_and_sums_to_zero():
    rng = np.random.default_rng(1)
    P, G, eps = 5, 6, 1e-6
    R = rng.normal(size=P * G).astype(np.float32)
    adv = grpo_adv(R, P, G, eps).reshape(P, G)
    R2 = R.astype(np.float64).reshape(P, G)
    want = (R2 - R2.mean(1, keepdims=True)) / (R2.std(1, ddof=0, keepdims=True) + eps)
    np.testing.assert_allclose(adv, want, rtol=3e-7, atol=1e-7)
    assert np.all(np.abs(adv.sum(1)) < 1e-5)
    # groups are independent: changing one group leaves the others untouched
    R3 = R.copy()
    R3[:G] += 3.0
    adv3 = grpo_adv(R3, P, G, eps).reshape(P, G)
    assert np.array_equal(adv3[1:], adv[1:])


# ---------------------------------------------------------------- selection
def _cu(T):
    return np.concatenate([[0], np.cumsum(T)]).astype(np.int32)


def test_rpc_uniform_cutoff_closed_forms():
    # q(l) = 1/T  =>  p_t = (T-t+1)/T,  sum_t p_t = (T+1)/2   (uniform cutoff)
    T = np.array([1, 2, 7, 64, 1000])
    mask, pi, cut = select(SEL_RPC, _cu(T), min_cut=1, seed=3)
    cu = _cu(T)
    for i, Ti in enumerate(T):
        p = pi[cu[i]:cu[i + 1]]
        t = np.arange(1, Ti + 1)
        want = ((Ti - t + 1).astype(np.float32) / np.float32(Ti))
        assert np.array_equal(p, want)
        assert p[0] == 1.0 and np.all(np.diff(p) <= 0) and p[-1] > 0
        assert abs(float(p.astype(np.float64).sum()) - (Ti + 1) / 2) < 1e-4 * Ti
        assert 1 <= cut[i] <= Ti
        assert np.array_equal(mask[cu[i]:cu[i + 1]], (t <= cut[i]).astype(np.uint8))


def test_rpc_minimum_cutoff_closed_forms():
    # p_t = 1 (t <= C), (T-t+1)/(T-C+1) (t > C); E[L] = (C+T)/2; 1/p bounded
    C = 100
    T = np.array([30, 100, 101, 250, 8192])
    cu = _cu(T)
    mask, pi, cut = select(SEL_RPC, cu, min_cut=C, seed=11, offset=5)
    for i, Ti in enumerate(T):
        Ci = min(C, Ti)
        p = pi[cu[i]:cu[i + 1]].astype(np.float64)
        t = np.arange(1, Ti + 1)
        want = np.where(t <= Ci, 1.0, (Ti - t + 1) / (Ti - Ci + 1))
        np.testing.assert_allclose(p, want, rtol=6e-8)
        assert abs(p.sum() - (Ci + Ti) / 2) < 1e-4 * Ti
        late = t > Ci      # the weight bound is stated for the positions past the mandatory prefix
        assert np.all(1.0 / p[late] <= (Ti - Ci + 1) / (Ti - t[late] + 1) * (1 + 1e-6))
        assert Ci <= cut[i] <= Ti
    # a response shorter than C is kept whole with pi = 1
    assert cut[0] == 30 and np.all(pi[:30] == 1.0) and np.all(mask[:30] == 1)


def test_rpc_cut_law_exact_enumeration():
    """Pr(L >= t) over every value of the 64-bit draw's quotient equals pi_t.

    L = C + floor(u n / 2^64): the quotient takes each value j in {0..n-1} for
    ceil((j+1) 2^64 / n) - ceil(j 2^64 / n) values of u, so the law is uniform
    to within 2^-64 * n; rational arithmetic checks the survival function.
    """
    for T, C in [(9, 1), (40, 10), (13, 13)]:
        n = T - C + 1
        counts = [-((-(j + 1) * 2**64) // n) - (-((-j * 2**64) // n)) for j in range(n)]
        assert sum(counts) == 2**64
        _, pi, _ = select(SEL_RPC, _cu([T]), min_cut=C)
        for t in range(1, T + 1):
            surv = Fraction(sum(c for j, c in enumerate(counts) if C + j >= t), 2**64)
            want = Fraction(1) if t <= C else Fraction(T - t + 1, n)
            assert abs(surv - want) <= Fraction(n, 2**64)
            assert abs(float(pi[t - 1]) - float(want)) <= 6e-8 * float(want)


def test_rpc_cut_mean_over_seeds():
    # E[L]/T = 1/2 + C/(2T)   (Appendix B.2)
    T, C, S = 400, 100, 3000
    cu = _cu([T] * 8)
    cuts = np.concatenate([select(SEL_RPC, cu, min_cut=C, seed=s)[2] for s in range(S // 8)])
    mean = cuts.mean() / T
    want = 0.5 + C / (2 * T)
    sd = math.sqrt(((T - C + 1) ** 2 - 1) / 12) / T / math.sqrt(len(cuts))
    assert abs(mean - want) < 4 * sd
    assert cuts.min() >= C and cuts.max() <= T
    # distinct responses and distinct seeds give distinct draws
    assert len(np.unique(cuts)) > 200


def test_urs_threshold_and_pi():
    assert urs_threshold(1.0) == 2**32
    assert urs_threshold(0.5) == 2**31
    assert urs_threshold(1e-12) == 1
    with pytest.raises(ValueError):
        urs_threshold(0.0)
    T = np.array([5, 64, 333])
    for p in (0.25, 0.5, 0.75):
        mask, pi, cut = select(SEL_URS, _cu(T), p=p, seed=9)
        assert cut is None
        assert np.all(pi == np.float32(p))
    mask, pi, _ = select(SEL_URS, _cu(T), p=1.0, seed=9)
    assert np.all(mask == 1) and np.all(pi == 1.0)      # full-token case


def test_urs_frequency_matches_p():
    # E[m / pi] = 1 (Proposition 1): binomial z-test with fixed seeds
    T = np.array([4096] * 16)
    for p in (0.25, 0.5, 0.9):
        mask, pi, _ = select(SEL_URS, _cu(T), p=p, seed=123, offset=7)
        n = mask.size
        z = (mask.sum() - n * p) / math.sqrt(n * p * (1 - p))
        assert abs(z) < 4.0
        est = (mask / pi.astype(np.float64)).mean()
        assert abs(est - 1.0) < 4.0 * math.sqrt((1 - p) / p / n)


def test_urs_keying():
    """Draws depend on (seed, offset, response, position) and on nothing else."""
    T = np.array([37, 64, 21])
    cu = _cu(T)
    base, _, _ = select(SEL_URS, cu, p=0.5, seed=42, offset=1)
    # response 1 in isolation but with the same global index => same bits
    k0, k1, off = 42, 0, 1
    t0 = np.arange(64, dtype=np.uint64)
    words = philox4x32_10(t0 >> np.uint64(2), 1, 0, off, k0, k1)
    x = np.choose((t0 & np.uint64(3)).astype(np.int64), words)
    assert np.array_equal(base[cu[1]:cu[2]], (x < 2**31).astype(np.uint8))
    other_seed, _, _ = select(SEL_URS, cu, p=0.5, seed=43, offset=1)
    other_off, _, _ = select(SEL_URS, cu, p=0.5, seed=42, offset=2)
    hi_off, _, _ = select(SEL_URS, cu, p=0.5, seed=42, offset=1 + (1 << 32))
    assert not np.array_equal(base, other_seed)
    assert not np.array_equal(base, other_off)
    assert not np.array_equal(base, hi_off)
    # the prefix of a longer response equals the shorter response's draws
    longer, _, _ = select(SEL_URS, _cu([50, 64, 21]), p=0.5, seed=42, offset=1)
    assert np.array_equal(longer[:37], base[:37])


def test_det_truncation():
    T = np.array([1, 2, 9, 100])
    cu = _cu(T)
    mask, pi, cut = select(SEL_DET, cu, beta=0.5)
    assert list(cut) == [1, 1, 4, 50]
    assert np.all(pi == 1.0)
    for i in range(len(T)):
        assert mask[cu[i]:cu[i + 1]].sum() == cut[i]
        assert np.all(mask[cu[i]:cu[i] + cut[i]] == 1)


def test_empty_responses():
    cu = _cu([0, 5, 0, 3, 0])
    for mode in (SEL_URS, SEL_RPC, SEL_DET):
        mask, pi, cut = select(mode, cu, p=0.5, min_cut=2, beta=0.5, seed=1)
        assert mask.shape == (8,)
        if cut is not None:
            assert cut[0] == 0 and cut[2] == 0 and cut[4] == 0
        si, sr, so, n = compact(mask, cu)
        assert n == int(mask.sum()) and so[0] == 0 and so[1] == 0 and so[-1] == n


# --------------------------------------------------------------- compaction
def test_compact_brute_force_and_segments():
    rng = np.random.default_rng(2)
    T = rng.integers(1, 50, size=12)
    cu = _cu(T)
    mask = (rng.random(cu[-1]) < 0.4).astype(np.uint8)
    si, sr, so, n = compact(mask, cu)
    assert n == mask.sum()
    assert np.array_equal(si, np.nonzero(mask)[0])
    resp_of = np.repeat(np.arange(len(T)), T)
    assert np.array_equal(sr, resp_of[si])
    for i in range(len(T)):
        assert so[i + 1] - so[i] == mask[cu[i]:cu[i + 1]].sum()
    # prefix modes: the kept tokens of response i are [cu_i, cu_i + L_i)
    mask, _, cut = select(SEL_RPC, cu, min_cut=3, seed=4)
    si, sr, so, n = compact(mask, cu)
    want = np.concatenate([np.arange(cu[i], cu[i] + cut[i]) for i in range(len(T))])
    assert np.array_equal(si, want)
    assert n == cut.sum()


# ------------------------------------------------- general survival schedules
from oracle import select_survival  # noqa: E402


def _geometric_schedule(T, rho, floor):
    p = np.maximum(rho ** np.arange(T), floor).astype(np.float32)
    p[0] = 1.0
    return p


def test_survival_selection_is_a_prefix_with_the_scheduled_law():
    rng = np.random.default_rng(7)
    T = np.array([1, 5, 64, 300, 0, 17])
    cu = _cu(T)
    surv = np.concatenate([_geometric_schedule(t, 0.97, 0.05) for t in T if t > 0])
    mask, cut = select_survival(cu, surv, seed=3, offset=1)
    for i, Ti in enumerate(T):
        m = mask[cu[i]:cu[i + 1]]
        assert m.sum() == cut[i] and np.all(m[:cut[i]] == 1) and np.all(m[cut[i]:] == 0)
        assert (cut[i] >= 1) == (Ti > 0)
    # frequencies over many responses: Pr(L >= t) = surv_t (binomial z-test, fixed seeds)
    Tn, R = 40, 4000
    p = _geometric_schedule(Tn, 0.9, 0.02)
    cuR = _cu([Tn] * R)
    maskR, cutR = select_survival(cuR, np.tile(p, R), seed=11)
    freq = maskR.reshape(R, Tn).mean(0)
    z = (freq - p) / np.sqrt(np.maximum(p * (1 - p), 1e-12) / R)
    assert np.abs(z[1:]).max() < 4.5 and freq[0] == 1.0
    # the uniform-cutoff schedule (T-t+1)/T gives a uniform cut: E[L] = (T+1)/2
    pu = ((Tn - np.arange(Tn)) / Tn).astype(np.float32)
    _, cutU = select_survival(cuR, np.tile(pu, R), seed=12)
    assert abs(cutU.mean() - (Tn + 1) / 2) < 4 * math.sqrt((Tn ** 2 - 1) / 12 / R)
    with pytest.raises(ValueError):
        select_survival(_cu([3]), np.array([1.0, 0.5, 0.7], dtype=np.float32))


def test_survival_draw_boundaries_are_exact():
    """u = k 2^-24 is kept iff k < ceil(p 2^24): checked at the two draws around the
    boundary, found by scanning seeds for responses whose draw lands there."""
    p_t = np.float32(0.3)
    bound = math.ceil(float(p_t) * 2 ** 24)          # number of 24-bit draws with u < p
    assert abs(bound / 2 ** 24 - float(p_t)) < 2 ** -24
    surv = np.array([1.0, p_t], dtype=np.float32)
    from oracle.philox import philox4x32_10 as ph
    seen = {True: 0, False: 0}
    for seed in range(400):
        x0 = int(ph(0, 0, 2, 0, seed, 0)[0])
        k = x0 >> 8
        mask, cut = select_survival(_cu([2]), surv, seed=seed)
        assert (cut[0] == 2) == (k < bound)
        seen[k < bound] += 1
    assert seen[True] > 50 and seen[False] > 150
    # the comparison itself at the boundary, in float32 as the kernels do it
    assert np.float32(bound - 1) * np.float32(2.0 ** -24) < p_t
    assert not (np.float32(bound) * np.float32(2.0 ** -24) < p_t)


# ------------------------------------------------------- packing of the prefixes
def test_gather_scatter_rows():
    from oracle import gather_rows, scatter_rows
    rng = np.random.default_rng(4)
    T = rng.integers(1, 40, size=9)
    cu = _cu(T)
    x = rng.normal(size=(cu[-1], 6)).astype(np.float32)
    mask, _, cut = select(SEL_RPC, cu, min_cut=2, seed=8)
    si, sr, so, n = compact(mask, cu)
    g = gather_rows(x, si)
    assert np.array_equal(g, x[si])                                   # library indexing
    # under RPC the packed rows are the prefixes, and sel_offsets are their cu_seqlens
    for i in range(len(T)):
        assert np.array_equal(g[so[i]:so[i + 1]], x[cu[i]:cu[i] + cut[i]])
    s = scatter_rows(g, si, cu[-1])
    assert np.array_equal(s, x * mask[:, None])
    assert scatter_rows(g[:0], si[:0], 5).shape == (5, 6)


# ------------------------------------------------------ sharding by response
def test_resp_base_makes_a_shard_draw_the_whole_batch_masks():
    """A shard that passes the global index of its first response realises, for its own
    responses, exactly the mask, pi and cut the whole batch realises (Section 3.1: masks
    of different responses are drawn independently, so this is what keeps Proposition 1
    valid response by response under data-parallel sharding)."""
    T = np.array([37, 0, 64, 21, 5, 90, 1, 12])
    cu = _cu(T)
    for mode, kw in ((SEL_URS, dict(p=0.5)), (SEL_RPC, dict(min_cut=4)), (SEL_DET, dict(beta=0.5))):
        mask, pi, cut = select(mode, cu, seed=9, offset=3, **kw)
        for lo, hi in ((0, 3), (3, 8), (5, 6)):
            m2, p2, c2 = select(mode, _cu(T[lo:hi]), seed=9, offset=3, resp_base=lo, **kw)
            assert np.array_equal(m2, mask[cu[lo]:cu[hi]])
            assert np.array_equal(p2.view(np.uint32), pi[cu[lo]:cu[hi]].view(np.uint32))
            if cut is not None:
                assert np.array_equal(c2, cut[lo:hi])
        # without the base the shard would reuse the draws of responses 0..: a different mask
        if mode != SEL_DET:
            m3, _, _ = select(mode, _cu(T[3:8]), seed=9, offset=3, **kw)
            assert not np.array_equal(m3, mask[cu[3]:cu[8]])
    surv = np.concatenate([_geometric_schedule(t, 0.9, 0.05) for t in T if t > 0])
    ms, cs = select_survival(cu, surv, seed=2)
    m2, c2 = select_survival(_cu(T[3:8]), surv[cu[3]:], seed=2, resp_base=3)
    assert np.array_equal(m2, ms[cu[3]:]) and np.array_equal(c2, cs[3:])


# ------------------------------------------------------------ general cut laws
from oracle import cutlaw_counts, select_cutlaw  # noqa: E402


def test_cutlaw_survival_is_the_suffix_sum_of_q():
    """Eq. rpc-survival: p_t = sum_{l >= t} q(l), with p_1 = 1, p non-increasing and
    p_T = q(T) > 0, for a geometric and a random law, against rational arithmetic."""
    rng = np.random.default_rng(5)
    T = np.array([1, 7, 64, 0, 300, 33])
    cu = _cu(T)
    q = np.concatenate([(np.maximum(0.9 ** np.arange(t), 0.02) * rng.uniform(0.5, 1.0, t)) / 40
                        for t in T if t > 0])
    q = q.astype(np.float32)
    mask, pi, cut = select_cutlaw(cu, q, seed=1)
    k = cutlaw_counts(q)
    assert np.array_equal(k, np.floor(q.astype(np.float64) * 2.0 ** 32).astype(np.uint64))
    assert list(cutlaw_counts(np.array([1.0, 2.5, 0.5, -1.0, np.nan], dtype=np.float32))) == \
        [2 ** 32 - 1, 2 ** 32 - 1, 2 ** 31, 0, 0]
    for i, Ti in enumerate(T):
        if Ti == 0:
            assert cut[i] == 0
            continue
        p = pi[cu[i]:cu[i + 1]].astype(np.float64)
        kk = [int(x) for x in k[cu[i]:cu[i + 1]]]
        tot = sum(kk)
        for t in range(Ti):
            want = Fraction(sum(kk[t:]), tot)
            assert abs(Fraction(float(p[t])) - want) <= want * Fraction(1, 2 ** 24)
        assert p[0] == 1.0 and np.all(np.diff(p) <= 0) and p[-1] > 0
        # and against the law itself: float32 rounding of pi plus the 2^-32 quantum of
        # each of the (at most Ti) masses in the suffix
        qq = q[cu[i]:cu[i + 1]].astype(np.float64)
        np.testing.assert_allclose(p, np.cumsum(qq[::-1])[::-1] / qq.sum(), rtol=2e-7,
                                   atol=2 * Ti * 2.0 ** -32 / qq.sum())
        m = mask[cu[i]:cu[i + 1]]
        assert 1 <= cut[i] <= Ti and m[:cut[i]].all() and not m[cut[i]:].any()


def test_cutlaw_uniform_law_reproduces_the_uniform_cutoff_closed_form():
    # q = 1/T on every position (T a power of two, so the masses are exact):
    # pi_t = (T - t + 1) / T, bit for bit what the RPC mode writes for C = 1
    for Tn in (8, 64, 4096):
        cu = _cu([Tn, Tn])
        _, pi, _ = select_cutlaw(cu, np.full(2 * Tn, 1.0 / Tn, dtype=np.float32))
        _, pi_rpc, _ = select(SEL_RPC, cu, min_cut=1)
        assert np.array_equal(pi.view(np.uint32), pi_rpc.view(np.uint32))
    # a mandatory prefix C: zero mass before position C (App. B.2): pi = 1 for t <= C
    Tn, C = 64, 16
    q = np.zeros(Tn, dtype=np.float32)
    q[C - 1:] = 1.0 / 64
    _, pi, cut = select_cutlaw(_cu([Tn]), q, seed=3)
    _, pi_rpc, _ = select(SEL_RPC, _cu([Tn]), min_cut=C)
    assert np.array_equal(pi.view(np.uint32), pi_rpc.view(np.uint32)) and cut[0] >= C
    # scaling the whole law changes nothing
    _, pi2, cut2 = select_cutlaw(_cu([Tn]), q * np.float32(0.25), seed=3)
    assert np.array_equal(pi2, pi) and cut2[0] == cut[0]
    # no mass anywhere: the response is kept whole
    m0, p0, c0 = select_cutlaw(_cu([5]), np.zeros(5, dtype=np.float32))
    assert m0.all() and np.all(p0 == 1) and c0[0] == 5
    # masses after the last positive one: those tokens are never selected (pi = 0)
    m1, p1, c1 = select_cutlaw(_cu([4]), np.array([0.5, 0.5, 0.0, -1.0], dtype=np.float32))
    assert np.all(p1[2:] == 0) and not m1[2:].any() and c1[0] in (1, 2)


def test_cutlaw_draw_boundaries_and_frequencies():
    """L >= t iff floor(u S_1 / 2^64) < S_t: checked against the integer draw recomputed
    from the generator, and Pr(L = l) = q(l) over many responses (z-test, fixed seeds)."""
    from oracle.philox import philox4x32_10 as ph
    q = np.array([0.125, 0.25, 0.5, 0.125], dtype=np.float32)
    k = [int(x) for x in cutlaw_counts(q)]
    S = [sum(k[t:]) for t in range(4)]
    for seed in range(300):
        x0, x1, _, _ = ph(0, 7, 3, 0, seed, 0)
        r = (((int(x1) << 32) | int(x0)) * S[0]) >> 64
        want = sum(1 for t in range(4) if S[t] > r)
        _, _, cut = select_cutlaw(_cu([4]), q, seed=seed, resp_base=7)
        assert cut[0] == want
    R = 6000
    _, _, cuts = select_cutlaw(_cu([4] * R), np.tile(q, R), seed=13)
    freq = np.bincount(cuts, minlength=5)[1:] / R
    z = (freq - q) / np.sqrt(q * (1 - q) / R)
    assert np.abs(z).max() < 4.5


# ---------------------------------------------- draws: ranges, ends and strictness
def test_rpc_cut_reaches_both_ends_with_the_uniform_frequency():
    """L_i is uniform on {C..T}: both ends are attained and every value has frequency
    1/(T - C + 1) (z-test over 8000 responses, fixed seed).  A cut law that never reaches T
    would leave the last token with inclusion probability 0 < p_{i,T}."""
    T, C, R = 7, 3, 8000
    _, pi, cuts = select(SEL_RPC, _cu([T] * R), min_cut=C, seed=17)
    n = T - C + 1
    freq = np.bincount(cuts, minlength=T + 1)[C:] / R
    assert cuts.min() == C and cuts.max() == T
    z = (freq - 1.0 / n) / math.sqrt((1.0 / n) * (1 - 1.0 / n) / R)
    assert np.abs(z).max() < 4.5
    # and the realised frequency of keeping token t is pi_t
    kept = (np.arange(1, T + 1)[None, :] <= cuts[:, None]).mean(0)
    p = pi[:T].astype(np.float64)
    zz = (kept - p) / np.sqrt(np.maximum(p * (1 - p), 1e-12) / R)
    assert np.abs(zz[C:]).max() < 4.5 and np.all(kept[:C] == 1.0)


def test_survival_draw_is_24_bit_and_the_comparison_strict():
    """Each response's schedule is built from its own draw, recomputed here from the
    generator: with p_2 = k 2^-24 (k the 24-bit draw itself) the token is NOT kept
    (u < p fails at equality), with p_2 = (k + 1) 2^-24 it is.  A coarser draw, or a
    non-strict comparison, flips one of the two."""
    from oracle.philox import philox4x32_10 as ph
    B = 64
    x0 = ph(0, np.arange(B), 2, 0, 5, 0)[0]
    k = (x0 >> np.uint64(8)).astype(np.int64)
    assert (k % 2 == 1).sum() > 10 and (k % 2 == 0).sum() > 10      # both parities occur
    cu = _cu([2] * B)
    at = np.stack([np.ones(B), k * 2.0 ** -24], axis=1).astype(np.float32).ravel()
    above = np.stack([np.ones(B), (k + 1) * 2.0 ** -24], axis=1).astype(np.float32).ravel()
    ok = k > 0                                                       # a schedule must stay positive
    at[1::2][~ok] = 2.0 ** -24
    _, cut_at = select_survival(cu, at, seed=5)
    _, cut_above = select_survival(cu, above, seed=5)
    assert np.all(cut_at[ok] == 1) and np.all(cut_above == 2)


def test_cutlaw_unit_counts_make_every_cut_equally_likely():
    """Masses of one fixed-point quantum each (q = 2^-32): S = (T, .., 2, 1) and r is uniform
    on {0..T-1}, so L = T - r takes every value in {1..T} with probability 1/T; a non-strict
    comparison S_t >= r would never produce L = 1."""
    T, R = 4, 6000
    q = np.full(T * R, 2.0 ** -32, dtype=np.float32)
    mask, pi, cuts = select_cutlaw(_cu([T] * R), q, seed=23)
    assert np.array_equal(pi[:T], np.array([1.0, 0.75, 0.5, 0.25], dtype=np.float32))
    freq = np.bincount(cuts, minlength=T + 1)[1:] / R
    assert cuts.min() == 1 and cuts.max() == T
    z = (freq - 0.25) / math.sqrt(0.25 * 0.75 / R)
    assert np.abs(z).max() < 4.5


def test_rpc_draw_layout_is_the_documented_one():
    """The cut of response i comes from words 0 and 1 of the Philox block with counter
    (0, i, 1, offset_lo): u = x1 2^32 + x0 (the layout the C header documents and the CUDA
    kernels follow).  T - C + 1 = 2^40-scale ranges do not exist, so the high word decides L:
    using x0 twice, or the words swapped, changes the cuts."""
    from oracle.philox import philox4x32_10 as ph
    T, C = 32768, 1
    for seed in range(40):
        x0, x1, _, _ = ph(0, 3, 1, 9, seed, 0)
        u = (int(x1) << 32) | int(x0)
        want = C + ((u * (T - C + 1)) >> 64)
        _, _, cut = select(SEL_RPC, _cu([T]), min_cut=C, seed=seed, offset=9, resp_base=3)
        assert cut[0] == want
        assert want == C + ((int(x1) * (T - C + 1)) >> 32)      # the high word alone fixes L here
