"""Pins for the CPU oracle: values the paper prints, closed forms, brute force.

None of these tests touches the CUDA library.  Each check is chosen so that a
plausible slip in the oracle (a dropped term, a wrong sign or index, the wrong
Beta parameters) fails it.
"""
import itertools
import math
import os
from fractions import Fraction

import mpmath
import numpy as np
import pytest

from oracle import beta_codebook as bc
from oracle import pvq_oracle as po
from oracle import pvq_pyref as pr
from paper_2410_16926_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


_POINTS = {}


def pyramid_points(n, k):
    """All integer points with sum |p_i| = k, by exhaustive search of [-k,k]^n."""
    if (n, k) not in _POINTS:
        _POINTS[(n, k)] = [p for p in itertools.product(range(-k, k + 1), repeat=n)
                           if sum(map(abs, p)) == k]
    return _POINTS[(n, k)]


def hyp2f1_terminating(a, b, c, z):
    """2F1 for a non-positive integer a: the finite sum of Pochhammer ratios."""
    total, term, j = Fraction(0), Fraction(1), 0
    while True:
        total += term
        if a + j == 0 or b + j == 0:
            break
        term = term * Fraction((a + j) * (b + j), (c + j) * (j + 1)) * z
        j += 1
    return total


def binomial_count(n, k):
    """Textbook count of P(n,k): choose the s non-zero coordinates, their signs,
    and a composition of k into s positive parts."""
    if k == 0:
        return 1
    return sum((1 << s) * math.comb(n, s) * math.comb(k - 1, s - 1) for s in range(1, min(n, k) + 1))


# ----------------------------------------------------------------- count table

def test_paper_example_P_2_7_has_28_points():
    # Sec. 2.5, figure of P(2,7): 28 points, codes C(2,7) = [0, 27].
    with open(os.path.join(GOLDEN, "paper_values.txt")) as f:
        vals = dict(line.split("#")[0].split("=") for line in f if "=" in line.split("#")[0])
    assert pr.count(2, 7) == int(vals["N(2,7)"])
    assert int(po.code_to_int(po.count_table(2, 7, 1)[2, 7])) == int(vals["N(2,7)"])
    codes = sorted(pr.enumerate_point(list(p), 7) for p in pyramid_points(2, 7))
    assert codes == list(range(int(vals["code_min(2,7)"]), int(vals["code_max(2,7)"]) + 1))


def test_boundary_values():
    # Sec. 2.4: N(D,0) = 1 for all D >= 0 and N(0,K) = 0 for all K >= 1.
    t = po.count_table(12, 12, 2)
    for n in range(13):
        assert po.code_to_int(t[n, 0]) == 1 == pr.count(n, 0)
    for k in range(1, 13):
        assert po.code_to_int(t[0, k]) == 0 == pr.count(0, k)


@pytest.mark.parametrize("n,k", [(1, 1), (2, 7), (3, 4), (5, 3), (8, 8), (16, 18), (32, 22), (32, 50), (64, 96)])
def test_closed_form_hypergeometric(n, k):
    # Sec. 2.4: N(D,K) = 2D * 2F1(1-D, 1-K; 2; 2).
    exact = 2 * n * hyp2f1_terminating(1 - n, 1 - k, 2, 2)
    assert exact.denominator == 1
    assert pr.count(n, k) == exact.numerator
    assert pr.count(n, k) == binomial_count(n, k)
    W = (pr.count(n, k).bit_length() + 31) // 32
    assert po.code_to_int(po.count_table(n, k, W)[n, k]) == exact.numerator
    if n * k <= 64:
        mpmath.mp.dps = 60
        assert int(mpmath.nint(2 * n * mpmath.hyp2f1(1 - n, 1 - k, 2, 2))) == exact.numerator


@pytest.mark.parametrize("n,k", [(1, 5), (2, 7), (3, 4), (4, 5), (5, 3), (6, 3)])
def test_count_is_number_of_points(n, k):
    assert pr.count(n, k) == len(pyramid_points(n, k))


def test_table_first_row_and_column():
    # App. C.1 pseudocode: the one-dimensional row is all 2, the one-pulse column is 2d.
    t = po.count_table(40, 60, 4)
    for k in range(1, 61):
        assert po.code_to_int(t[1, k]) == 2
    for n in range(0, 41):
        assert po.code_to_int(t[n, 1]) == 2 * n


def test_c_table_equals_python_table():
    for (N, K, W) in [(32, 22, 2), (32, 50, 3), (64, 96, 6), (16, 18, 2)]:
        tc = po.count_table(N, K, W + 1)
        tp = pr.count_table(N, K)
        for n in range(N + 1):
            for k in range(K + 1):
                assert po.code_to_int(tc[n, k]) == tp[n][k]


def test_cumulative_identity():
    # App. C.2: sum_{j=1}^{m-1} N(d,k-j) = V(d,k-1) - V(d,k-m), V(d,k) = sum_{i=1}^k N(d,i).
    t = pr.count_table(9, 14)
    V = [[sum(row[1:k + 1]) for k in range(15)] for row in t]
    for d in range(10):
        for k in range(1, 15):
            for m in range(1, k + 1):
                assert sum(t[d][k - j] for j in range(1, m)) == V[d][k - 1] - V[d][k - m]


def test_telescoped_enumeration_identity():
    # Algorithm 2 rewritten with the cumulative counts of App. C.2, as the CUDA encoder uses it:
    # with U(n,k) = V(n,k) + V(n,k-1), V(n,k) = sum_{j<=k} N(n,j), the term of position i is
    # U(n,k_i) - U(n,k_{i+1}) for y_i <= 0 and U(n,k_i) - 2 V(n,k_{i+1}) for y_i > 0, so the code is
    # U(N-1,K) + sum_i [ U(n_i - 1, k_{i+1}) - (U or 2V)(n_i, k_{i+1}) ] with U(-1, .) = 0.
    rng = np.random.default_rng(3)
    for (N, K) in [(2, 7), (3, 4), (6, 4), (8, 11), (16, 18), (32, 50)]:
        t = pr.count_table(N, K)
        V = [[sum(row[:k + 1]) for k in range(K + 1)] for row in t]
        U = lambda n, k: 0 if n < 0 else V[n][k] + (V[n][k - 1] if k > 0 else 0)
        pts = pyramid_points(N, K) if N <= 3 else []
        for _ in range(200):
            cuts = np.sort(rng.integers(0, K + 1, size=N - 1))
            mags = np.diff(np.concatenate(([0], cuts, [K])))
            pts.append(tuple(int(m) * int(sg) for m, sg in zip(mags, rng.choice([-1, 1], size=N))))
        for y in pts:
            code, k = U(N - 1, K), K
            for i, yi in enumerate(y):
                n = N - 1 - i
                k -= abs(yi)
                code += U(n - 1, k) - (2 * V[n][k] if yi > 0 else U(n, k))
            assert k == 0 and code == pr.enumerate_point(list(y), K)


# -------------------------------------------------------------------- pulses K

@pytest.mark.parametrize("N,bits", [(32, 64), (32, 96), (64, 192), (16, 40), (8, 24), (128, 384)])
def test_max_pulses_is_largest_that_fits(N, bits):
    # Sec. 3.3 Step 2, checked with the binomial closed form rather than the recurrence.
    K = po.max_pulses(N, bits)
    assert K == pr.max_pulses(N, bits)
    assert binomial_count(N, K) <= (1 << bits) < binomial_count(N, K + 1)
    assert po.index_bits(N, K) == (binomial_count(N, K) - 1).bit_length() <= bits


def test_max_pulses_beyond_4096():
    # Step 2 with closed forms for tiny N: N(2,K) = 4K and N(3,K) = 4K^2 + 2, so the largest K
    # with N(3,K) <= 2^27 is floor(sqrt((2^27 - 2) / 4)) = 5792, and N(2,K) <= 2^14 gives 4096.
    assert po.max_pulses(3, 27) == math.isqrt(((1 << 27) - 2) // 4) == 5792
    assert po.max_pulses(2, 14) == 4096
    assert binomial_count(3, 5792) == 4 * 5792 ** 2 + 2 <= 1 << 27 < binomial_count(3, 5793)


def test_bits_per_weight_examples():
    # Sec. 4.1: group size 16 with a 40-bit direction code is 2.5 bits per weight; the
    # tables' 3.125 = 3 + 16/128, 3.25 = 3 + 4/16, 3.5 = 2.5 + 16/16, 3.88 ~ 3.5 + 6/16
    # only come out with both bit counts divided by the group size.
    def bpw(n, index_bits, amp_bits):
        return index_bits / n + amp_bits / n
    assert bpw(16, 40, 0) == 2.5
    assert bpw(128, 384, 16) == 3.125
    assert bpw(16, 48, 4) == 3.25
    assert bpw(16, 40, 16) == 3.5
    assert abs(bpw(16, 56, 6) - 3.88) < 0.01


# ------------------------------------------------------- enumeration bijection

@pytest.mark.parametrize("n,k", [(1, 3), (2, 7), (3, 4), (4, 5), (5, 3), (6, 4)])
def test_encode_is_a_bijection_and_decode_inverts_it(n, k):
    pts = pyramid_points(n, k)
    total = pr.count(n, k)
    seen = set()
    for p in pts:
        c = pr.enumerate_point(list(p), k)
        assert 0 <= c < total
        seen.add(c)
        y, ok = pr.deenumerate_code(c, n, k)
        assert ok and tuple(y) == p
        # the C oracle agrees on both directions
        cw = po.enumerate_point(p, k, 1)
        assert po.code_to_int(cw) == c
        yc, okc = po.deenumerate_code(cw, n, k)
        assert okc and tuple(yc.tolist()) == p
    assert seen == set(range(total))


def test_invalid_codes_are_flagged():
    n, k = 4, 5
    total = pr.count(n, k)
    for c in (total, total + 1, total + 57, (1 << 32) - 1):
        _, ok = pr.deenumerate_code(c, n, k)
        assert not ok
        _, okc = po.deenumerate_code(po.int_to_code(c, 1), n, k)
        assert not okc


def _decode_without_negative_update(c, N, K):
    """Algorithm 3 with the line after x_i <- -j left out (the slip the paper says
    the original description contains).  Only here to show the pins catch it."""
    t = pr.count_table(N, K)
    r, k, y = c, K, [0] * N
    for i in range(N):
        if k <= 0:
            break
        row = t[N - 1 - i]
        if r < row[k]:
            continue
        r -= row[k]
        j = 1
        while j < k and r >= 2 * row[k - j]:
            r -= 2 * row[k - j]
            j += 1
        if r < row[k - j]:
            y[i] = j
        else:
            y[i] = -j  # missing: r -= row[k - j]
        k -= j
    return y


def test_missing_update_breaks_only_points_with_a_negative_before_the_end():
    # Sec. 2.5 "Pyramid decoding" / remark under Algorithm 3: without the update after
    # x_i <- -j, decoding goes wrong only when a negative value is followed by more pulses.
    n, k = 4, 4
    exposed = broken = 0
    for p in pyramid_points(n, k):
        c = pr.enumerate_point(list(p), k)
        y = _decode_without_negative_update(c, n, k)
        first_neg = next((i for i, v in enumerate(p) if v < 0), None)
        k_after = None if first_neg is None else k - sum(abs(v) for v in p[:first_neg + 1])
        if first_neg is None or k_after == 0:
            assert tuple(y) == p          # no negative, or nothing left to decode after it
        else:
            exposed += 1
            broken += tuple(y) != p
    assert exposed > 0 and broken > exposed // 2


@pytest.mark.parametrize("N,K,W", [(128, 187, 12), (128, 386, 16), (256, 369, 24), (64, 3359, 16), (128, 6378, 32)])
def test_wide_codes_against_python_integers(N, K, W):
    """The C oracle's 32-limb integers at the group sizes and bit rates of the paper's grid
    (Sec. 4.1) against Python's: the enumeration of quantised Gaussian groups, and back."""
    rng = np.random.default_rng(N + K)
    total = pr.count_table(N, K)[N][K]
    assert (total.bit_length() + 31) // 32 <= W and total > 1 << (32 * (W - 1))
    for _ in range(6):
        x = rng.standard_normal(N).astype(np.float32)
        y = po.quantize_group(x, K)
        assert np.abs(y).sum() == K
        cw = po.enumerate_point(y, K, W)
        c = po.code_to_int(cw)
        assert c == pr.enumerate_point(y.tolist(), K) and 0 <= c < total
        y2, ok = po.deenumerate_code(cw, N, K)
        assert ok and np.array_equal(y, y2)
    for c in (0, total - 1):
        y, ok = po.deenumerate_code(po.int_to_code(c, W), N, K)
        assert ok and np.abs(y).sum() == K


def test_random_points_round_trip_at_config_sizes():
    rng = np.random.default_rng(7)
    for (N, K, W) in [(32, 22, 2), (32, 50, 3), (64, 96, 6)]:
        total = pr.count_table(N, K)[N][K]
        for _ in range(40):
            x = rng.standard_normal(N).astype(np.float32)
            y = po.quantize_group(x, K)
            assert np.abs(y).sum() == K
            cw = po.enumerate_point(y, K, W)
            c = po.code_to_int(cw)
            assert c == pr.enumerate_point(y.tolist(), K) and 0 <= c < total
            y2, ok = po.deenumerate_code(cw, N, K)
            assert ok and np.array_equal(y, y2)
        # the extremes of the code range decode to valid points too
        for c in (0, total - 1):
            y, ok = po.deenumerate_code(po.int_to_code(c, W), N, K)
            assert ok and np.abs(y).sum() == K
            assert po.code_to_int(po.enumerate_point(y, K, W)) == c


# ----------------------------------------------------------- direction (greedy)

def _nearest_on_pyramid_sqdist(a, k):
    """Exhaustive search over P(n,k) for the point nearest to the non-negative target a."""
    best = None
    for p in itertools.product(range(k + 1), repeat=len(a)):
        if sum(p) != k:
            continue
        d = sum((Fraction(float(ai)) - pi) ** 2 for ai, pi in zip(a, p))
        best = d if best is None or d < best else best
    return best


@pytest.mark.parametrize("n,k", [(2, 3), (3, 4), (4, 5), (5, 4), (6, 5)])
def test_greedy_matches_exhaustive_nearest_point(n, k):
    # Sec. 2.5: the vector is mapped to the closest point on the pyramid.
    rng = np.random.default_rng(100 * n + k)
    for trial in range(60):
        x = rng.standard_normal(n).astype(np.float32)
        if trial % 5 == 0:
            x = np.round(x * 2).astype(np.float32) / 2          # provoke equal residuals
        if not np.any(x):
            continue
        y = np.array(pr.quantize_group(x.tolist(), k))
        assert np.array_equal(y, po.quantize_group(x, k))
        assert np.abs(y).sum() == k
        assert all((yi == 0) or (yi < 0) == bool(np.signbit(xi)) for yi, xi in zip(y, x))
        l1 = pr.tree_sum(np.abs(x))
        a = [np.float32(np.float32(abs(v)) * np.float32(np.float32(k) / l1)) for v in x]
        d_greedy = sum((Fraction(float(ai)) - abs(int(yi))) ** 2 for ai, yi in zip(a, y))
        assert d_greedy == _nearest_on_pyramid_sqdist(a, k)


def test_lowest_index_wins_ties():
    # Four equal values, K = 6: floor gives one pulse each, the two pulses left over go to
    # the lowest indices.
    y = po.quantize_group(np.array([1, 1, 1, 1], dtype=np.float32), 6)
    assert y.tolist() == [2, 2, 1, 1]
    y = po.quantize_group(np.array([-1, 1, -1, 1], dtype=np.float32), 7)
    assert y.tolist() == [-2, 2, -2, 1]
    assert pr.quantize_group([1, 1, 1, 1], 6) == [2, 2, 1, 1]


def test_fixup_remove_branch_with_forced_start():
    # The floor start cannot overshoot, so the removal loop is exercised directly.
    m = np.array([3, 0, 2, 2], dtype=np.int32)          # sum 7, K = 5
    e = np.array([0.25, 0.9, 0.10, 0.10], dtype=np.float32)
    out = po.fixup(m, e, 5)
    # smallest residual among m>0 is 0.10 at index 2 (lowest index of the tie), then index 3
    assert out.tolist() == [3, 0, 1, 1]
    assert pr.fixup(m.tolist(), e.tolist(), 5) == [3, 0, 1, 1]
    m = np.array([1, 0, 0, 0], dtype=np.int32)          # add branch: K = 3
    e = np.array([0.2, 0.7, 0.7, 0.1], dtype=np.float32)
    assert po.fixup(m, e, 3).tolist() == [1, 1, 1, 0]


def test_deficit_is_below_group_size():
    # Sec. 2.5: the fix-up ends within T < D steps.
    rng = np.random.default_rng(3)
    for (N, K) in [(32, 22), (32, 50), (64, 96)]:
        for _ in range(200):
            x = rng.standard_normal(N).astype(np.float32)
            l1 = po.tree_sum_padded(np.abs(x))
            a = np.abs(x) * np.float32(np.float32(K) / l1)
            deficit = K - int(np.floor(a).sum())
            assert 0 <= deficit < N


def test_degenerate_groups():
    assert po.quantize_group(np.zeros(8, dtype=np.float32), 5).tolist() == [5, 0, 0, 0, 0, 0, 0, 0]
    x = np.zeros(8, dtype=np.float32)
    x[3] = -2.5
    assert po.quantize_group(x, 5).tolist() == [0, 0, 0, -5, 0, 0, 0, 0]
    x = np.array([-0.0, 1.0, 0.0, -1.0], dtype=np.float32)
    assert po.quantize_group(x, 4).tolist() == [0, 2, 0, -2]
    tiny = np.full(4, 1e-45, dtype=np.float32)            # K / l1 overflows: no direction
    assert po.quantize_group(tiny, 4).tolist() == [4, 0, 0, 0]
    assert pr.quantize_group(tiny.tolist(), 4) == [4, 0, 0, 0]


# ------------------------------------------------------------------ fp32 tree

def test_tree_sum_order():
    # (1e8 + 1) + (-1e8 + 1) is 0 in fp32 with adjacent pairs first; left-to-right gives 1.
    v = np.array([1e8, 1.0, -1e8, 1.0], dtype=np.float32)
    assert po.tree_sum_padded(v) == np.float32(0.0)
    assert pr.tree_sum(v) == np.float32(0.0)
    # contiguous halves: ((a+b)+(c+d)) + ((e+f)+(g+h))
    v = np.array([1.0, 2 ** -24, 2 ** -24, 2 ** -24, 2 ** -24, 2 ** -24, 2 ** -24, 2 ** -24], dtype=np.float32)
    h = np.float32
    expect = h(h(h(v[0] + v[1]) + h(v[2] + v[3])) + h(h(v[4] + v[5]) + h(v[6] + v[7])))
    assert po.tree_sum_padded(v) == expect
    # padding: 5 values behave as 8 with three zeros appended
    w = np.array([0.1, 0.2, 0.3, 0.4, 0.5], dtype=np.float32)
    assert po.tree_sum_padded(w) == h(h(h(w[0] + w[1]) + h(w[2] + w[3])) + w[4])


def test_tree_sum_close_to_exact():
    rng = np.random.default_rng(11)
    for n in (32, 64, 448):
        v = rng.standard_normal(n).astype(np.float32) ** 2
        s = float(po.tree_sum_padded(v))
        exact = math.fsum(float(a) for a in v)
        assert abs(s - exact) <= 10 * 2.0 ** -24 * exact


# ---------------------------------------------------------- amplitude codebook

@pytest.mark.parametrize("N,G,b", [(32, 16, 8), (32, 128, 4), (32, 448, 8), (64, 448, 6)])
def test_edges_are_the_quantiles(N, G, b):
    # CDF(edge_j) = j / 2^b with the regularised incomplete beta function from mpmath.
    e = bc.edges_f64(N, G, b)
    assert np.all(np.diff(e) > 0) and 0 < e[0] and e[-1] < 1
    mpmath.mp.dps = 40
    a, bb = bc.beta_params(N, G)
    L = 1 << b
    for j in (1, L // 4, L // 2, L - 1):
        cdf = mpmath.betainc(a, bb, 0, mpmath.mpf(float(e[j - 1])), regularized=True)
        assert abs(float(cdf) - j / L) < 1e-9
    assert np.all(np.diff(bc.edges_f32(N, G, b)) > 0)


@pytest.mark.parametrize("N,G,b", [(32, 16, 8), (32, 128, 4), (32, 448, 8), (64, 448, 6)])
def test_levels_are_the_probability_midpoints(N, G, b):
    # Sec. 3.4: dequantize(q) = PPF((q + 1/2) / 2^b), i.e. CDF(level_q) = (q + 1/2) / 2^b with
    # mpmath's regularised incomplete beta.  A midpoint of the two edges in the u domain, or
    # PPF(q / 2^b), lands in the same bin but misses this value by far more than the bound.
    lev = bc.levels_f64(N, G, b)
    mpmath.mp.dps = 40
    a, bb = bc.beta_params(N, G)
    L = 1 << b
    for q in (0, L // 4, L // 2, L - 1):
        cdf = mpmath.betainc(a, bb, 0, mpmath.mpf(float(lev[q])), regularized=True)
        assert abs(float(cdf) - (q + 0.5) / L) < 1e-9
    # the plausible mistakes, shown to fail the same check
    e = np.concatenate(([0.0], bc.edges_f64(N, G, b), [1.0]))
    for q in (L // 4, L // 2):
        for wrong in (0.5 * (e[q] + e[q + 1]), e[q]):
            cdf = mpmath.betainc(a, bb, 0, mpmath.mpf(float(wrong)), regularized=True)
            assert abs(float(cdf) - (q + 0.5) / L) > 1e-7  # a hundred times the bound above
    # the amplitude table is the square root of it, rounded once
    amp = bc.levels_amp_f32(N, G, b)
    assert np.array_equal(amp, np.sqrt(lev).astype(np.float32))


def test_uniform_and_power_special_cases():
    # Beta(1,1) is uniform; Beta(1,b) has PPF(p) = 1 - (1-p)^(1/b).  N=2 gives alpha = 1.
    e = bc.edges_f64(2, 2, 3)
    assert np.allclose(e, np.arange(1, 8) / 8, rtol=0, atol=1e-14)
    e = bc.edges_f64(2, 5, 3)
    assert np.allclose(e, 1 - (1 - np.arange(1, 8) / 8) ** (1 / 4), rtol=1e-12)


@pytest.mark.parametrize("N,G,b", [(32, 16, 8), (32, 128, 4), (64, 448, 6)])
def test_quantize_dequantize_identity(N, G, b):
    # Sec. 3.4: dequantize(q) is the probability midpoint of bin q, so it quantises back to q,
    # both by the threshold count and by floor(CDF * 2^b) taken literally.
    e32 = bc.edges_f32(N, G, b)
    lev = bc.levels_f64(N, G, b)
    q_thr = (lev.astype(np.float32)[:, None] >= e32[None, :]).sum(axis=1)
    assert q_thr.tolist() == list(range(1 << b))
    assert bc.quantize_cdf(lev, N, G, b).tolist() == list(range(1 << b))
    amp = bc.levels_amp_f32(N, G, b)
    assert np.allclose(amp.astype(np.float64) ** 2, lev, rtol=3e-7)


def test_threshold_count_equals_floor_of_cdf():
    rng = np.random.default_rng(5)
    N, G, b = 32, 128, 4
    u = rng.beta(*bc.beta_params(N, G), size=20000)
    e = bc.edges_f64(N, G, b)
    q_thr = (u[:, None] >= e[None, :]).sum(axis=1)
    assert np.array_equal(q_thr, bc.quantize_cdf(u, N, G, b))


def test_gaussian_rows_fill_all_bins_evenly():
    # Sec. 3.4 theorem (with the proof's parameters): on Gaussian rows every one of the 2^b
    # bins is hit with probability 2^-b.  The parameters printed in the theorem statement,
    # Beta(D/2, G(D-1)/2), visibly tilt the occupancy; so the check tells the two apart.
    rng = np.random.default_rng(9)
    N, G, b = 32, 16, 4
    w = rng.standard_normal((40000, G, N))
    ss = (w ** 2).sum(axis=2)
    u = ss / ss.sum(axis=1, keepdims=True)
    L = 1 << b

    def occupancy(edges):
        q = (u[..., None] >= edges).sum(axis=-1)
        return np.bincount(q.ravel(), minlength=L) / q.size

    occ = occupancy(bc.edges_f64(N, G, b))
    assert np.all(np.abs(occ - 1 / L) < 0.004)
    from scipy import stats
    wrong = stats.beta.ppf(np.arange(1, L) / L, N / 2, G * (N - 1) / 2)
    occ_wrong = occupancy(wrong)
    assert np.max(np.abs(occ_wrong - 1 / L)) > 0.008


# --------------------------------------------------------------- whole matrix

def _small_matrix(rows, cols, seed, sigma=0.02):
    rng = np.random.default_rng(seed)
    return (rng.standard_normal((rows, cols)) * sigma).astype(np.float32)


def test_matrix_encode_matches_per_group_python_reference():
    N, K, b = 8, 6, 3
    x = _small_matrix(5, 48, 1)
    G = x.shape[1] // N
    edges = bc.edges_f32(N, G, b)
    codes, sidx, rnorm = po.encode(x, N, K, b, edges, W=1)
    q = po.unpack_scale_idx(sidx, G, b)
    for r in range(x.shape[0]):
        ss = [pr.tree_sum(x[r, g * N:(g + 1) * N] * x[r, g * N:(g + 1) * N]) for g in range(G)]
        ss_row = pr.tree_sum_padded(ss)
        assert rnorm[r] == np.sqrt(ss_row, dtype=np.float32)
        for g in range(G):
            y = pr.quantize_group(x[r, g * N:(g + 1) * N].tolist(), K)
            assert po.code_to_int(codes[r, g]) == pr.enumerate_point(y, K)
            u = np.float32(ss[g] / ss_row)
            assert q[r, g] == int((u >= edges).sum())


def test_scale_index_stream_is_lsb_first():
    N, K, b = 8, 6, 3
    x = _small_matrix(2, 40, 2)          # G = 5 -> 15 bits -> 2 bytes, stride rounded to 4
    G = 5
    codes, sidx, rnorm = po.encode(x, N, K, b, bc.edges_f32(N, G, b), W=1)
    assert sidx.shape == (2, 4)
    q = po.unpack_scale_idx(sidx, G, b)
    for r in range(2):
        stream = sum(int(v) << (3 * g) for g, v in enumerate(q[r]))
        assert stream == int.from_bytes(sidx[r].tobytes(), "little")


def test_decode_reconstruction_properties():
    import torch
    N, K, b = 32, 50, 8
    x = _small_matrix(16, 512, 3)
    G = x.shape[1] // N
    edges, amp = bc.edges_f32(N, G, b), bc.levels_amp_f32(N, G, b)
    codes, sidx, rnorm = po.encode(x, N, K, b, edges)
    out_bits, status = po.decode(codes, sidx, rnorm, N, K, b, amp)
    assert status == 0
    out = (out_bits.astype(np.uint32) << 16).view(np.float32)
    q = po.unpack_scale_idx(sidx, G, b)
    for r in range(0, 16, 5):
        for g in range(0, G, 3):
            y, ok = po.deenumerate_code(codes[r, g], N, K)
            assert ok
            # direction: the decoded group is y scaled to the quantised amplitude
            target = y / np.sqrt(float((y.astype(np.int64) ** 2).sum())) * float(rnorm[r]) * float(amp[q[r, g]])
            ref = torch.tensor(target, dtype=torch.float32).to(torch.bfloat16).to(torch.float32).numpy()
            got = out[r, g * N:(g + 1) * N]
            assert np.all(np.abs(got - ref) <= np.abs(ref) * 2.0 ** -7 + 1e-30)
            # amplitude: the group's norm is the dequantised amplitude up to bf16 rounding
            assert abs(np.linalg.norm(got) - rnorm[r] * amp[q[r, g]]) <= 2.0 ** -8 * rnorm[r] * amp[q[r, g]]
    # row norm identity: the groups' energies add up to the stored row norm
    assert np.allclose(np.sqrt((x.astype(np.float64) ** 2).sum(axis=1)), rnorm, rtol=1e-6)
    # the codec is a sensible quantiser: about 3 bits per weight buys > 12 dB
    err = ((out - x) ** 2).sum() / (x ** 2).sum()
    assert err < 10 ** (-12 / 10)


def test_bf16_rounding_matches_torch():
    import torch
    # decode's last step rounds to bf16 (nearest even): drive it with y=(K,0,..), amp chosen freely
    N, K, b = 2, 1, 1
    rng = np.random.default_rng(4)
    vals = np.concatenate([rng.standard_normal(2000).astype(np.float32) * np.float32(3.0),
                           np.array([1.00390625, 1.01171875, 3.0e38, 1e-40, 0.0], dtype=np.float32)])
    codes = np.zeros((vals.size, 1, 1), dtype=np.uint32)            # code 0 -> y = (0,+1)? check below
    y0, ok = po.deenumerate_code(codes[0, 0], N, K)
    assert ok and np.abs(y0).sum() == 1
    sidx = np.zeros((vals.size, po.scale_row_stride(1, b)), dtype=np.uint8)
    levels = np.array([1.0, 1.0], dtype=np.float32)
    out_bits, _ = po.decode(codes, sidx, vals, N, K, b, levels)
    ref = torch.tensor(vals).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    pos = int(np.nonzero(y0)[0][0])
    assert np.array_equal(out_bits[:, pos], ref)


def test_zero_row_and_invalid_code():
    N, K, b = 8, 6, 3
    x = _small_matrix(3, 32, 6)
    x[1] = 0.0
    G = 4
    edges, amp = bc.edges_f32(N, G, b), bc.levels_amp_f32(N, G, b)
    codes, sidx, rnorm = po.encode(x, N, K, b, edges, W=1)
    assert rnorm[1] == 0 and np.all(po.unpack_scale_idx(sidx, G, b)[1] == 0)
    out_bits, status = po.decode(codes, sidx, rnorm, N, K, b, amp)
    assert status == 0 and np.all((out_bits[1] & 0x7FFF) == 0)
    codes[2, 1, 0] = pr.count(N, K)       # first invalid value
    out_bits, status = po.decode(codes, sidx, rnorm, N, K, b, amp)
    assert status == 1 and np.all(out_bits[2, 8:16] == 0) and np.any(out_bits[2, :8] != 0)


# ------------------------------------------------------------ rotation (Sec. 2.3, Step 1)

def _hadamard(n):
    h = np.array([[1.0]])
    while h.shape[0] < n:
        h = np.block([[h, h], [h, -h]])
    return h


@pytest.mark.parametrize("block,cols", [(4, 12), (16, 16), (64, 128), (256, 512)])
def test_rotation_is_the_hadamard_matrix_exactly_on_small_integers(block, cols):
    # power-of-four blocks scale by a power of two and small integers add without rounding:
    # the butterflies must then equal the matrix product bit for bit
    rng = np.random.default_rng(block)
    x = rng.integers(-8, 9, size=(5, cols)).astype(np.float32)
    s = (rng.integers(0, 2, size=block) * 2 - 1).astype(np.float32)
    got = po.rotate(x, block, s)
    xs = (x.reshape(5, cols // block, block) * s).astype(np.float64)
    want = (xs @ _hadamard(block)) / np.sqrt(block)
    assert np.array_equal(got.astype(np.float64), want.reshape(5, cols))


@pytest.mark.parametrize("block", [8, 32, 512])
def test_rotation_against_the_matrix_for_irrational_scales(block):
    rng = np.random.default_rng(7)
    x = rng.standard_normal((3, 2 * block)).astype(np.float32)
    s = (rng.integers(0, 2, size=block) * 2 - 1).astype(np.float32)
    got = po.rotate(x, block, s).astype(np.float64)
    want = ((x.reshape(3, 2, block) * s).astype(np.float64) @ _hadamard(block) / np.sqrt(block)).reshape(3, -1)
    assert np.max(np.abs(got - want)) < 1e-5 * np.sqrt(block)
    # orthogonal: norms are kept
    assert np.allclose(np.linalg.norm(got, axis=1), np.linalg.norm(x.astype(np.float64), axis=1), rtol=1e-5)


def test_rotation_twice_without_signs_is_the_identity():
    rng = np.random.default_rng(3)
    x = rng.integers(-20, 21, size=(4, 64)).astype(np.float32)
    ones = np.ones(16, dtype=np.float32)
    assert np.array_equal(po.rotate(po.rotate(x, 16, ones), 16, ones), x)      # H H = n I, exact here


def test_rotation_of_bf16_input_widens_exactly():
    from paper_2410_16926_b200 import inputs
    rng = np.random.default_rng(11)
    x = rng.standard_normal((2, 64)).astype(np.float32)
    xb = inputs.f32_to_bf16_bits(x)
    s = np.ones(64, dtype=np.float32)
    assert np.array_equal(po.rotate(xb, 64, s), po.rotate(inputs.bf16_bits_to_f32(xb), 64, s))


# --------------------------------------- 16-bit amplitudes and the least-squares amplitude

def test_binary16_conversion_matches_numpy_on_every_half_and_on_ties():
    # every binary16 value converts to itself; rounding of fp32 agrees with numpy's IEEE conversion
    for h in list(range(0, 0x7c01, 37)) + [0x0001, 0x03ff, 0x0400, 0x7bff, 0x7c00, 0x8001, 0xfbff]:
        f = np.array([h], dtype=np.uint16).view(np.float16)[0]
        assert po.f32_to_f16(np.float32(f)) == h
        assert np.float32(po.f16_to_f32(h)) == np.float32(f)
    rng = np.random.default_rng(16)
    vals = np.concatenate([rng.standard_normal(4000) * 10.0 ** rng.integers(-9, 6, 4000),
                           [65504.0, 65519.9, 65520.0, 1e9, 5.96e-8, 2.98e-8, 2.9802325e-8, 6.1e-5, 0.0, -0.0,
                            1.00048828125, 1.0009765625 + 2.0 ** -12]]).astype(np.float32)
    with np.errstate(over="ignore"):
        want = vals.astype(np.float16).view(np.uint16)
    got = np.array([po.f32_to_f16(v) for v in vals], dtype=np.uint16)
    assert np.array_equal(got, want)


def test_binary16_amplitudes_round_trip_the_group_norm():
    rng = np.random.default_rng(21)
    N, K, rows, cols = 32, 22, 6, 256
    x = (rng.standard_normal((rows, cols)) * 0.05).astype(np.float32)
    codes, sidx, rnorm = po.encode(x, N, K, 16)
    assert sidx.shape == (rows, 2 * (cols // N))                       # 16 bits per group
    amp16 = sidx.view(np.uint16).reshape(rows, cols // N)
    norms = np.sqrt((x.reshape(rows, -1, N).astype(np.float64) ** 2).sum(axis=2))
    got = amp16.view(np.float16).astype(np.float64)
    assert np.all(np.abs(got - norms) <= np.abs(norms) * 2.0 ** -11 + 1e-12)   # half an ulp of binary16 (+ fp32 sums)
    out, st = po.decode(codes, sidx, rnorm, N, K, 16)
    o = inputs.bf16_bits_to_f32(out).reshape(rows, -1, N).astype(np.float64)
    # decoded groups have the stored amplitude as their norm (up to bf16 rounding of the elements)
    assert st == 0 and np.allclose(np.sqrt((o ** 2).sum(axis=2)), got, rtol=6e-3)


def test_least_squares_amplitude_is_the_projection_and_beats_the_norm():
    rng = np.random.default_rng(22)
    N, K, rows, cols = 16, 18, 8, 128
    x = rng.standard_normal((rows, cols)).astype(np.float32)
    c0, s0, r0 = po.encode(x, N, K, 16, amp_mode=0)
    c1, s1, r1 = po.encode(x, N, K, 16, amp_mode=1)
    assert np.array_equal(c0, c1)                                      # the direction does not depend on it
    a0 = s0.view(np.uint16).view(np.float16).astype(np.float64).reshape(rows, -1)
    a1 = s1.view(np.uint16).view(np.float16).astype(np.float64).reshape(rows, -1)
    xg = x.reshape(rows, -1, N).astype(np.float64)
    for r in range(rows):
        for g in range(cols // N):
            y, ok = po.deenumerate_code(c0[r, g], N, K)
            yh = y / np.linalg.norm(y)
            proj = float(yh @ xg[r, g])                                # argmin_a ||x - a y_hat||
            assert abs(a1[r, g] - proj) <= abs(proj) * 2.0 ** -10
            assert np.linalg.norm(xg[r, g] - a1[r, g] * yh) <= np.linalg.norm(xg[r, g] - a0[r, g] * yh) + 1e-3
            assert a1[r, g] <= a0[r, g] * (1 + 2.0 ** -10)             # Cauchy-Schwarz


def test_least_squares_amplitude_with_the_quantile_codebook():
    rng = np.random.default_rng(23)
    N, K, b, rows, cols = 32, 22, 8, 4, 1024
    x = rng.standard_normal((rows, cols)).astype(np.float32)
    e = bc.edges_f32(N, cols // N, b)
    q0 = po.unpack_scale_idx(po.encode(x, N, K, b, e, amp_mode=0)[1], cols // N, b)
    q1 = po.unpack_scale_idx(po.encode(x, N, K, b, e, amp_mode=1)[1], cols // N, b)
    assert np.all(q1 <= q0) and np.mean(q1 < q0) > 0.5                 # smaller amplitudes, lower bins


# ------------------------------------------------ QSNR on a Gaussian source (Sec. 2.6, Fig. 3)

@pytest.mark.parametrize("N", [16, 32])
def test_qsnr_on_a_gaussian_source_sits_under_the_rate_distortion_bound(N):
    # A memoryless Gaussian source at R bits per sample cannot beat 6.02 R dB; a spherical code
    # of this size stays within a few dB of it, gains about 6 dB per bit, and the least-squares
    # amplitude is never worse than the norm.
    rng = np.random.default_rng(0)
    x = rng.standard_normal((128, 1024)).astype(np.float32)
    prev = None
    for bpw in (2.0, 3.0, 4.0):
        bits = int(bpw * N)
        K = po.max_pulses(N, bits)
        q = []
        for amp_mode in (0, 1):
            c, s, r = po.encode(x, N, K, 16, W=(bits + 31) // 32, amp_mode=amp_mode)
            out, _ = po.decode(c, s, r, N, K, 16)
            xh = inputs.bf16_bits_to_f32(out).astype(np.float64)
            q.append(10 * np.log10((x.astype(np.float64) ** 2).sum() / ((x - xh) ** 2).sum()))
        assert q[1] >= q[0] - 1e-9
        assert 6.02 * bpw - 2.6 < q[0] < 6.02 * (bpw + 16.0 / N)
        if prev is not None:
            assert 5.0 < q[0] - prev < 8.0          # per extra bit
        prev = q[0]
