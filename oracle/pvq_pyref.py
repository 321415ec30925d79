"""Pure-Python form of the oracle (Python ints, numpy.float32 scalars).

Test infrastructure only.  It restates the same passages of the paper as
pvq_oracle.c, with Python's unbounded integers instead of limb arrays, and is
used on small cases: to cross-check the C oracle and to run the brute-force
pins.  It shares no code with the CUDA library.

Passages followed: Sec. 2.4 (pyramid, count recurrence), Sec. 2.5 and
Algorithm 1 (direction, floor + greedy reading), Algorithm 2 (encoding),
Algorithm 3 (corrected decoding), Sec. 3.3 Step 2 (pulses K).
"""
from functools import lru_cache

import numpy as np

f32 = np.float32


@lru_cache(maxsize=None)
def count(n: int, k: int) -> int:
    """N(n,k) = |P(n,k)|, Sec. 2.4: N(n,0)=1, N(0,k>=1)=0,
    N(n,k) = N(n-1,k) + N(n,k-1) + N(n-1,k-1)."""
    if k == 0:
        return 1
    if n == 0:
        return 0
    return count(n - 1, k) + count(n, k - 1) + count(n - 1, k - 1)


def count_table(nmax: int, kmax: int):
    """Rows n = 0..nmax, columns k = 0..kmax, built bottom-up (no recursion depth)."""
    t = [[0] * (kmax + 1) for _ in range(nmax + 1)]
    for n in range(nmax + 1):
        for k in range(kmax + 1):
            if k == 0:
                t[n][k] = 1
            elif n == 0:
                t[n][k] = 0
            else:
                t[n][k] = t[n - 1][k] + t[n][k - 1] + t[n - 1][k - 1]
    return t


def index_bits(N: int, K: int) -> int:
    """ceil(log2 N(N,K)) on the integer itself."""
    v = count_table(N, K)[N][K]
    return (v - 1).bit_length()


def max_pulses(N: int, bits: int) -> int:
    """Sec. 3.3 Step 2: largest K with N(N,K) <= 2**bits."""
    K = 0
    while True:
        t = count_table(N, K + 1)
        if t[N][K + 1] > (1 << bits):
            return K
        K += 1


def tree_sum(v):
    """Balanced tree over contiguous halves, fp32, length a power of two."""
    v = [f32(a) for a in v]
    if len(v) == 1:
        return v[0]
    mid = len(v) // 2
    return f32(tree_sum(v[:mid]) + tree_sum(v[mid:]))


def tree_sum_padded(v):
    p = 1
    while p < len(v):
        p <<= 1
    return tree_sum(list(v) + [f32(0.0)] * (p - len(v)))


def fixup(m, e, K):
    """Greedy single-pulse add / remove, lowest index on equal residuals."""
    m = list(m)
    e = [f32(a) for a in e]
    while sum(m) < K:
        j = 0
        for i in range(1, len(m)):
            if e[i] > e[j]:
                j = i
        m[j] += 1
        e[j] = f32(e[j] - f32(1.0))
    while sum(m) > K:
        j = -1
        for i in range(len(m)):
            if m[i] > 0 and (j < 0 or e[i] < e[j]):
                j = i
        m[j] -= 1
        e[j] = f32(e[j] + f32(1.0))
    return m


def quantize_group(x, K):
    """x (fp32 values) -> y in P(N,K): l1 scale, floor, greedy fix-up, signs."""
    x = [f32(a) for a in x]
    N = len(x)
    l1 = tree_sum([f32(abs(a)) for a in x])
    with np.errstate(divide="ignore", over="ignore"):
        gsc = f32(f32(K) / l1)
    if not (l1 > 0) or not np.isfinite(gsc):
        return [K] + [0] * (N - 1)
    a = [f32(f32(abs(v)) * gsc) for v in x]
    f = [f32(np.floor(v)) for v in a]
    m = [int(v) for v in f]
    e = [f32(ai - fi) for ai, fi in zip(a, f)]
    m = fixup(m, e, K)
    return [-mi if np.signbit(xi) else mi for mi, xi in zip(m, x)]


def enumerate_point(y, K):
    """Algorithm 2: pyramid point -> code in [0, N(N,K)-1]."""
    N = len(y)
    assert sum(abs(v) for v in y) == K
    t = count_table(N, K)
    c, k = 0, K
    for i, v in enumerate(y):
        if k == 0:
            break
        d1 = N - 1 - i
        mag = abs(v)
        if mag >= 1:
            c += t[d1][k]
            c += 2 * sum(t[d1][k - j] for j in range(1, mag))
            if v < 0:
                c += t[d1][k - mag]
        k -= mag
    return c


def deenumerate_code(c, N, K):
    """Algorithm 3 (corrected): code -> (pyramid point, valid flag)."""
    t = count_table(N, K)
    r, k = c, K
    y = [0] * N
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
            y[i] = -j
            r -= row[k - j]
        k -= j
    return y, (r == 0 and k == 0)
