"""ctypes front end of the C oracle (pvq_oracle.c).

Test infrastructure only: imported by tests, by the smoke check and by the
benchmark's CPU-baseline leg, never by the CUDA library or its binding.
Argument marshalling only; the arithmetic is in the C file.
"""
import ctypes as C

import numpy as np

from . import build as _build

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        i32, i64, vp = C.c_int, C.c_int64, C.c_void_p
        L.pvqo_count_table.argtypes = [i32, i32, i32, vp]
        L.pvqo_index_bits.argtypes = [i32, i32]
        L.pvqo_max_pulses.argtypes = [i32, i32]
        L.pvqo_tree_sum_padded.argtypes = [vp, i32]
        L.pvqo_tree_sum_padded.restype = C.c_float
        L.pvqo_fixup.argtypes = [vp, vp, i32, i32]
        L.pvqo_fixup.restype = None
        L.pvqo_quantize_group.argtypes = [vp, i32, i32, vp]
        L.pvqo_quantize_group.restype = None
        L.pvqo_enumerate.argtypes = [vp, i32, i32, i32, vp]
        L.pvqo_deenumerate.argtypes = [vp, i32, i32, i32, vp]
        L.pvqo_scale_row_stride.argtypes = [i64, i32]
        L.pvqo_scale_row_stride.restype = C.c_size_t
        L.pvqo_encode_amp.argtypes = [vp, i32, i64, i64, i64, i32, i32, i32, i32, i32, vp, vp, vp, vp, i32]
        L.pvqo_f32_to_f16.argtypes = [C.c_float]
        L.pvqo_f32_to_f16.restype = C.c_uint16
        L.pvqo_f16_to_f32.argtypes = [C.c_uint16]
        L.pvqo_f16_to_f32.restype = C.c_float
        L.pvqo_encode.argtypes = [vp, i32, i64, i64, i64, i32, i32, i32, i32, vp, vp, vp, vp, i32]
        L.pvqo_decode.argtypes = [vp, vp, vp, i64, i64, i32, i32, i32, i32, vp, vp, i64, vp, i32]
        L.pvqo_rotate.argtypes = [vp, i32, i64, i64, i64, i32, vp, vp]
        L.pvqo_threads.argtypes = []
        _lib = L
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def words_for_bits(bits: int) -> int:
    return (bits + 31) // 32


def count_table(nmax: int, kmax: int, W: int) -> np.ndarray:
    """uint32 [nmax+1][kmax+1][W], little-endian limbs of N(n,k)."""
    out = np.zeros((nmax + 1, kmax + 1, W), dtype=np.uint32)
    if lib().pvqo_count_table(nmax, kmax, W, _p(out)) != 0:
        raise OverflowError("N(n,k) does not fit %d words" % W)
    return out


def index_bits(N: int, K: int) -> int:
    return lib().pvqo_index_bits(N, K)


def max_pulses(N: int, bits: int) -> int:
    return lib().pvqo_max_pulses(N, bits)


def tree_sum_padded(v) -> np.float32:
    v = np.ascontiguousarray(v, dtype=np.float32)
    return np.float32(lib().pvqo_tree_sum_padded(_p(v), v.size))


def fixup(m, e, K: int):
    m = np.ascontiguousarray(m, dtype=np.int32).copy()
    e = np.ascontiguousarray(e, dtype=np.float32).copy()
    lib().pvqo_fixup(_p(m), _p(e), m.size, K)
    return m


def quantize_group(x, K: int) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    y = np.zeros(x.size, dtype=np.int32)
    lib().pvqo_quantize_group(_p(x), x.size, K, _p(y))
    return y


def enumerate_point(y, K: int, W: int) -> np.ndarray:
    y = np.ascontiguousarray(y, dtype=np.int32)
    code = np.zeros(W, dtype=np.uint32)
    if lib().pvqo_enumerate(_p(y), y.size, K, W, _p(code)) != 0:
        raise ValueError("not a point of P(N,K), or code too wide")
    return code


def deenumerate_code(code, N: int, K: int):
    code = np.ascontiguousarray(code, dtype=np.uint32)
    y = np.zeros(N, dtype=np.int32)
    ok = lib().pvqo_deenumerate(_p(code), N, K, code.size, _p(y))
    if ok < 0:
        raise ValueError("bad arguments")
    return y, bool(ok)


def scale_row_stride(G: int, scale_bits: int) -> int:
    return int(lib().pvqo_scale_row_stride(G, scale_bits))


def code_to_int(words) -> int:
    return sum(int(w) << (32 * i) for i, w in enumerate(np.asarray(words).tolist()))


def int_to_code(v: int, W: int) -> np.ndarray:
    return np.array([(v >> (32 * i)) & 0xFFFFFFFF for i in range(W)], dtype=np.uint32)


def f32_to_f16(f) -> int:
    return int(lib().pvqo_f32_to_f16(float(f)))


def f16_to_f32(h) -> float:
    return float(lib().pvqo_f16_to_f32(int(h)))


def encode(x: np.ndarray, N: int, K: int, scale_bits: int, edges: np.ndarray = None, W: int = None,
           nthreads: int = 0, amp_mode: int = 0):
    """x: 2-D float32 array, or uint16 array holding bf16 bit patterns.
    scale_bits 1..8 with the quantile `edges`, or 16 (binary16 amplitudes, no edges);
    amp_mode 0: amplitude ||x_g||, 1: least-squares amplitude of the chosen direction.
    Returns (codes uint32 [rows][G][W], scale_idx uint8 [rows][stride], row_norm f32 [rows])."""
    assert x.ndim == 2 and x.flags.c_contiguous
    if x.dtype == np.float32:
        dtype = 0
    elif x.dtype == np.uint16:
        dtype = 1
    else:
        raise TypeError("float32 or uint16 (bf16 bits)")
    rows, cols = x.shape
    G = cols // N
    if W is None:
        W = words_for_bits(index_bits(N, K))
    if scale_bits == 16:
        edges = np.zeros(1, dtype=np.float32)
    else:
        edges = np.ascontiguousarray(edges, dtype=np.float32)
        assert edges.size == (1 << scale_bits) - 1
    codes = np.zeros((rows, G, W), dtype=np.uint32)
    sidx = np.zeros((rows, scale_row_stride(G, scale_bits)), dtype=np.uint8)
    rnorm = np.zeros(rows, dtype=np.float32)
    rc = lib().pvqo_encode_amp(_p(x), dtype, rows, cols, cols, N, K, scale_bits, amp_mode, W, _p(edges),
                               _p(codes), _p(sidx), _p(rnorm), nthreads)
    if rc != 0:
        raise ValueError("oracle encode rejected its arguments")
    return codes, sidx, rnorm


def decode(codes: np.ndarray, sidx: np.ndarray, rnorm: np.ndarray, N: int, K: int,
           scale_bits: int, levels: np.ndarray = None, nthreads: int = 0):
    """Returns (bf16 bit patterns uint16 [rows][cols], status word)."""
    rows, G, W = codes.shape
    cols = G * N
    codes = np.ascontiguousarray(codes, dtype=np.uint32)
    sidx = np.ascontiguousarray(sidx, dtype=np.uint8)
    rnorm = np.ascontiguousarray(rnorm, dtype=np.float32)
    if scale_bits == 16:
        levels = np.zeros(1, dtype=np.float32)
    else:
        levels = np.ascontiguousarray(levels, dtype=np.float32)
        assert levels.size == (1 << scale_bits)
    assert sidx.shape == (rows, scale_row_stride(G, scale_bits))
    out = np.zeros((rows, cols), dtype=np.uint16)
    status = np.zeros(1, dtype=np.uint32)
    rc = lib().pvqo_decode(_p(codes), _p(sidx), _p(rnorm), rows, cols, N, K, scale_bits, W,
                           _p(levels), _p(out), cols, _p(status), nthreads)
    if rc != 0:
        raise ValueError("oracle decode rejected its arguments")
    return out, int(status[0])


def rotate(x: np.ndarray, block: int, signs: np.ndarray) -> np.ndarray:
    """Random-sign Hadamard rotation along the columns (Sec. 2.3 / Step 1): float32 [rows][cols]."""
    assert x.ndim == 2 and x.flags.c_contiguous
    dtype = 0 if x.dtype == np.float32 else 1
    assert x.dtype in (np.float32, np.uint16)
    signs = np.ascontiguousarray(signs, dtype=np.float32)
    assert signs.size == block
    out = np.zeros(x.shape, dtype=np.float32)
    if lib().pvqo_rotate(_p(x), dtype, x.shape[0], x.shape[1], x.shape[1], block, _p(signs), _p(out)) != 0:
        raise ValueError("oracle rotate rejected its arguments")
    return out


def unpack_scale_idx(sidx: np.ndarray, G: int, scale_bits: int) -> np.ndarray:
    """LSB-first bit stream per row -> int array [rows][G]."""
    bits = np.unpackbits(sidx, axis=1, bitorder="little")[:, :G * scale_bits]
    bits = bits.reshape(sidx.shape[0], G, scale_bits).astype(np.int64)
    return (bits << np.arange(scale_bits)).sum(axis=2)


def threads() -> int:
    return lib().pvqo_threads()
