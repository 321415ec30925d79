"""Oracle for the amplitude codebook (Sec. 3.4 and Sec. 3.3 Step 5).

Test infrastructure only; shares no code with the CUDA library.

The normalised group energy u = s_g^2 / ||s||^2 of a Gaussian row follows
Beta(N/2, N(G-1)/2) (the result of the appendix proof and of Step 5; the
theorem statement prints other parameters, which the proof does not support).
A b-bit quantiser is  quantize(u) = floor(CDF(u) * 2^b)  and
dequantize(q) = PPF((q + 1/2) / 2^b).  Because the CDF is increasing,
floor(CDF(u) 2^b) = #{ j in 1..2^b-1 : u >= PPF(j / 2^b) }, so the quantiser is
stored as its 2^b - 1 inner bin edges; the paper's own implementation
(App. C.3) calls scipy.stats.beta for both functions, and so does this file.
Everything is fp64 and rounded once to fp32 at the end.
"""
import numpy as np
from scipy import stats


def beta_params(N: int, G: int):
    """(alpha, beta) of the law of u for group size N and G groups per row."""
    if G < 2:
        raise ValueError("the quantile codebook needs at least two groups per row")
    return 0.5 * N, 0.5 * N * (G - 1)


def edges_f64(N: int, G: int, scale_bits: int) -> np.ndarray:
    a, b = beta_params(N, G)
    L = 1 << scale_bits
    p = np.arange(1, L, dtype=np.float64) / L
    return stats.beta.ppf(p, a, b)


def levels_f64(N: int, G: int, scale_bits: int) -> np.ndarray:
    a, b = beta_params(N, G)
    L = 1 << scale_bits
    p = (np.arange(L, dtype=np.float64) + 0.5) / L
    return stats.beta.ppf(p, a, b)


def edges_f32(N: int, G: int, scale_bits: int) -> np.ndarray:
    """Bin edges in the u domain, ascending, 2^b - 1 values."""
    return edges_f64(N, G, scale_bits).astype(np.float32)


def levels_amp_f32(N: int, G: int, scale_bits: int) -> np.ndarray:
    """sqrt of the dequantised u: the factor that multiplies the row norm."""
    return np.sqrt(levels_f64(N, G, scale_bits)).astype(np.float32)


def quantize_cdf(u, N: int, G: int, scale_bits: int) -> np.ndarray:
    """The paper's formula taken literally: floor(CDF(u) * 2^b), clamped."""
    a, b = beta_params(N, G)
    L = 1 << scale_bits
    q = np.floor(stats.beta.cdf(np.asarray(u, dtype=np.float64), a, b) * L)
    return np.minimum(q, L - 1).astype(np.int64)
