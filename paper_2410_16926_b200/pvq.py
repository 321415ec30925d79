"""Thin Python binding of the PVQ C-ABI library (include/pvq.h).

Argument marshalling only: every function checks tensor device / dtype /
contiguity, passes raw device pointers and the current CUDA stream to the
library call of the same name, and raises on a non-zero status.  No arithmetic
of the codec happens here, and there is no fallback: a missing library is an
error.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# PVQ_B200_LIB selects another build of the same library, e.g. the bounds-checked one
# (libpvq_b200_debug.so, see pvq_debug_status in include/pvq.h).
LIB_PATH = os.environ.get("PVQ_B200_LIB") or os.path.join(_HERE, "libpvq_b200.so")

DTYPE_F32 = 0
DTYPE_BF16 = 1
STATUS_INVALID_CODE = 1
STATUS_STAGING_TIMEOUT = 2
STATUS_TABLE_MISMATCH = 4

_lib = None


class PvqError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        msg = lib().pvq_strerror(status).decode()
        if status == 5:
            msg += " (cudaError %d)" % lib().pvq_last_cuda_error()
        super().__init__("%s: %s" % (where, msg))


class MatrixDesc(C.Structure):
    """Mirror of pvq_matrix_desc."""
    _fields_ = [("d_x", C.c_void_p), ("d_out", C.c_void_p), ("d_codes", C.c_void_p),
                ("d_scale_idx", C.c_void_p), ("d_row_norm", C.c_void_p), ("d_edges", C.c_void_p),
                ("d_levels", C.c_void_p), ("rows", C.c_int64), ("cols", C.c_int64), ("ld", C.c_int64),
                ("ld_out", C.c_int64)]


def lib():
    """The loaded C library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("PVQ CUDA library not built: %s is missing "
                               "(run `python -m paper_2410_16926_b200.build`)" % LIB_PATH)
        L = C.CDLL(LIB_PATH)
        i32, i64, vp, sz = C.c_int, C.c_int64, C.c_void_p, C.c_size_t
        ip = C.POINTER(C.c_int)
        L.pvq_strerror.argtypes = [i32]
        L.pvq_strerror.restype = C.c_char_p
        L.pvq_last_cuda_error.argtypes = []
        L.pvq_index_bits.argtypes = [i32, i32, ip]
        L.pvq_max_pulses.argtypes = [i32, i32, ip]
        L.pvq_code_words.argtypes = [i32, i32, ip]
        L.pvq_count_table_bytes.argtypes = [i32, i32]
        L.pvq_count_table_bytes.restype = sz
        L.pvq_scale_row_stride.argtypes = [i64, i32]
        L.pvq_scale_row_stride.restype = sz
        L.pvq_build_count_table.argtypes = [i32, i32, vp, sz, vp]
        L.pvq_build_scale_codebook.argtypes = [i32, i64, i32, vp, vp, vp]
        L.pvq_encode.argtypes = [vp, i32, i64, i64, i64, i32, i32, i32, vp, vp, vp, vp, vp, vp]
        L.pvq_decode.argtypes = [vp, vp, vp, i64, i64, i32, i32, i32, vp, vp, vp, i64, vp, vp]
        L.pvq_roundtrip.argtypes = [vp, i32, i64, i64, i64, i32, i32, i32, vp, vp, vp, vp, i64, vp]
        L.pvq_encode_batched.argtypes = [C.POINTER(MatrixDesc), i32, i32, i32, i32, i32, vp, vp]
        L.pvq_decode_batched.argtypes = [C.POINTER(MatrixDesc), i32, i32, i32, i32, vp, vp, vp]
        L.pvq_encode_amp.argtypes = [vp, i32, i64, i64, i64, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp]
        L.pvq_rotate_encode.argtypes = [vp, i32, i64, i64, i64, i32, vp, i32, i32, i32, vp, vp, vp, vp, vp, vp]
        L.pvq_rotate_roundtrip.argtypes = [vp, i32, i64, i64, i64, i32, vp, i32, i32, i32, vp, vp, vp, vp, i64, vp]
        L.pvq_decode_static_table.argtypes = [vp, vp, vp, i64, i64, i32, i32, i32, vp, vp, i64, vp, vp]
        L.pvq_debug_status.argtypes = [vp]
        L.pvq_encode_status.argtypes = [vp]
        _lib = L
    return _lib


EXPORTS = ["pvq_strerror", "pvq_last_cuda_error", "pvq_index_bits", "pvq_max_pulses", "pvq_code_words",
           "pvq_count_table_bytes", "pvq_scale_row_stride", "pvq_build_count_table",
           "pvq_build_scale_codebook", "pvq_encode", "pvq_decode", "pvq_roundtrip", "pvq_encode_batched",
           "pvq_decode_batched", "pvq_decode_static_table", "pvq_rotate_encode", "pvq_rotate_roundtrip", "pvq_encode_amp",
           "pvq_debug_status", "pvq_encode_status"]


def _check(status, where):
    if status != 0:
        raise PvqError(status, where)


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t, dtype=None):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("expected a CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError("expected dtype %s, got %s" % (dtype, t.dtype))
    if not t.is_contiguous() and not (t.dim() == 2 and t.stride(1) == 1):
        raise ValueError("expected a row-major tensor")
    return C.c_void_p(t.data_ptr())


def _dtype_code(x):
    if x.dtype == torch.float32:
        return DTYPE_F32
    if x.dtype == torch.bfloat16:
        return DTYPE_BF16
    raise TypeError("input must be float32 or bfloat16")


def encode_status(word):
    """The status word of the encode-side calls of this thread (an int32 device tensor of one
    element, or None): a staging time-out is reported there."""
    _check(lib().pvq_encode_status(_ptr(word, torch.int32)), "pvq_encode_status")


def debug_status(word):
    """Bounds-checked build only: violations are ORed into `word` (an int32 device tensor of one
    element, zeroed by the caller) by every later call of this thread; None switches it off."""
    _check(lib().pvq_debug_status(_ptr(word, torch.int32)), "pvq_debug_status")


# ---- host helpers ---------------------------------------------------------------

def index_bits(N, K):
    out = C.c_int()
    _check(lib().pvq_index_bits(N, K, C.byref(out)), "pvq_index_bits")
    return out.value


def max_pulses(N, bits):
    out = C.c_int()
    _check(lib().pvq_max_pulses(N, bits, C.byref(out)), "pvq_max_pulses")
    return out.value


def code_words(N, K):
    out = C.c_int()
    _check(lib().pvq_code_words(N, K, C.byref(out)), "pvq_code_words")
    return out.value


def count_table_bytes(N, K):
    return int(lib().pvq_count_table_bytes(N, K))


def scale_row_stride(G, scale_bits):
    return int(lib().pvq_scale_row_stride(G, scale_bits))


# ---- set-up ---------------------------------------------------------------------

def build_count_table(N, K, device="cuda"):
    """The device table blob of pvq_build_count_table (flat int32): the count table N(n,k)
    followed by the rearranged copies the kernels stage."""
    t = torch.empty(count_table_bytes(N, K) // 4, dtype=torch.int32, device=device)
    _check(lib().pvq_build_count_table(N, K, _ptr(t), t.numel() * 4, _stream()), "pvq_build_count_table")
    return t


def count_table_view(table, N, K):
    """The first section of the blob: uint32 words [N][K+1][W] of N(n,k)."""
    W = code_words(N, K)
    return table[:N * (K + 1) * W].view(N, K + 1, W)


def build_scale_codebook(N, G, scale_bits, device="cuda"):
    """(edges [2^b - 1], levels [2^b]) float32 device tensors."""
    L = 1 << scale_bits
    edges = torch.empty(L - 1, dtype=torch.float32, device=device)
    levels = torch.empty(L, dtype=torch.float32, device=device)
    _check(lib().pvq_build_scale_codebook(N, G, scale_bits, _ptr(edges), _ptr(levels), _stream()),
           "pvq_build_scale_codebook")
    return edges, levels


# ---- hot path -------------------------------------------------------------------

def alloc_encoded(rows, G, W, scale_bits, device="cuda"):
    codes = torch.empty((rows, G, W), dtype=torch.int32, device=device)
    sidx = torch.empty((rows, scale_row_stride(G, scale_bits)), dtype=torch.uint8, device=device)
    rnorm = torch.empty(rows, dtype=torch.float32, device=device)
    return codes, sidx, rnorm


def encode(x, N, K, scale_bits, table, edges, out=None, amp_mode=None):
    """x [rows][cols] float32 / bfloat16 on the GPU -> (codes int32 [rows][G][W],
    scale_idx uint8 [rows][stride], row_norm float32 [rows]).  amp_mode (0 / 1) goes through
    pvq_encode_amp; scale_bits 16 takes no edges."""
    rows, cols = x.shape
    G = cols // N
    if out is None:
        out = alloc_encoded(rows, G, code_words(N, K), scale_bits, x.device)
    codes, sidx, rnorm = out
    if amp_mode is not None:
        _check(lib().pvq_encode_amp(_ptr(x), _dtype_code(x), rows, cols, x.stride(0), N, K, scale_bits, amp_mode,
                                    _ptr(table, torch.int32), _ptr(edges, torch.float32),
                                    _ptr(codes, torch.int32), _ptr(sidx, torch.uint8),
                                    _ptr(rnorm, torch.float32), _stream()), "pvq_encode_amp")
        return codes, sidx, rnorm
    _check(lib().pvq_encode(_ptr(x), _dtype_code(x), rows, cols, x.stride(0), N, K, scale_bits,
                            _ptr(table, torch.int32), _ptr(edges, torch.float32), _ptr(codes, torch.int32),
                            _ptr(sidx, torch.uint8), _ptr(rnorm, torch.float32), _stream()), "pvq_encode")
    return codes, sidx, rnorm


def decode(codes, sidx, rnorm, N, K, scale_bits, table, levels, out=None, status=None):
    """-> bfloat16 [rows][G*N].  `status`: optional int32 device tensor of one element."""
    rows, G, _ = codes.shape
    cols = G * N
    if out is None:
        out = torch.empty((rows, cols), dtype=torch.bfloat16, device=codes.device)
    _check(lib().pvq_decode(_ptr(codes, torch.int32), _ptr(sidx, torch.uint8), _ptr(rnorm, torch.float32),
                            rows, cols, N, K, scale_bits, _ptr(table, torch.int32),
                            _ptr(levels, torch.float32), _ptr(out, torch.bfloat16), out.stride(0),
                            _ptr(status, torch.int32), _stream()), "pvq_decode")
    return out


def decode_static_table(codes, sidx, rnorm, N, K, scale_bits, levels, out=None, status=None):
    """decode() for callers that must not allocate on the device: the count table is the
    one built into the library.  `out` has to be passed by such a caller; it is only
    created here when omitted."""
    rows, G, _ = codes.shape
    cols = G * N
    if out is None:
        out = torch.empty((rows, cols), dtype=torch.bfloat16, device=codes.device)
    _check(lib().pvq_decode_static_table(_ptr(codes, torch.int32), _ptr(sidx, torch.uint8),
                                         _ptr(rnorm, torch.float32), rows, cols, N, K, scale_bits,
                                         _ptr(levels, torch.float32), _ptr(out, torch.bfloat16),
                                         out.stride(0), _ptr(status, torch.int32), _stream()),
           "pvq_decode_static_table")
    return out


def roundtrip(x, N, K, scale_bits, table, edges, levels, out=None):
    """Fused encode -> decode: bfloat16 [rows][cols]."""
    rows, cols = x.shape
    if out is None:
        out = torch.empty((rows, cols), dtype=torch.bfloat16, device=x.device)
    _check(lib().pvq_roundtrip(_ptr(x), _dtype_code(x), rows, cols, x.stride(0), N, K, scale_bits,
                               _ptr(table, torch.int32), _ptr(edges, torch.float32),
                               _ptr(levels, torch.float32), _ptr(out, torch.bfloat16), out.stride(0),
                               _stream()), "pvq_roundtrip")
    return out


def rotate_encode(x, block, signs, N, K, scale_bits, table, edges, out=None):
    """encode() of the rows of x rotated on the fly by the random-sign Hadamard of size `block`
    (signs: float32 +-1, `block` of them)."""
    rows, cols = x.shape
    G = cols // N
    if out is None:
        out = alloc_encoded(rows, G, code_words(N, K), scale_bits, x.device)
    codes, sidx, rnorm = out
    _check(lib().pvq_rotate_encode(_ptr(x), _dtype_code(x), rows, cols, x.stride(0), block,
                                   _ptr(signs, torch.float32), N, K, scale_bits, _ptr(table, torch.int32),
                                   _ptr(edges, torch.float32), _ptr(codes, torch.int32),
                                   _ptr(sidx, torch.uint8), _ptr(rnorm, torch.float32), _stream()),
           "pvq_rotate_encode")
    return codes, sidx, rnorm


def rotate_roundtrip(x, block, signs, N, K, scale_bits, table, edges, levels, out=None):
    """roundtrip() of the rows of x rotated on the fly: bfloat16 [rows][cols] in the rotated basis."""
    rows, cols = x.shape
    if out is None:
        out = torch.empty((rows, cols), dtype=torch.bfloat16, device=x.device)
    _check(lib().pvq_rotate_roundtrip(_ptr(x), _dtype_code(x), rows, cols, x.stride(0), block,
                                      _ptr(signs, torch.float32), N, K, scale_bits,
                                      _ptr(table, torch.int32), _ptr(edges, torch.float32),
                                      _ptr(levels, torch.float32), _ptr(out, torch.bfloat16), out.stride(0),
                                      _stream()), "pvq_rotate_roundtrip")
    return out


def _descs(items):
    arr = (MatrixDesc * len(items))()
    for d, it in zip(arr, items):
        x, outp = it.get("x"), it.get("out")
        codes, sidx, rnorm = it["codes"], it["scale_idx"], it["row_norm"]
        rows, G, _ = codes.shape
        d.d_x = x.data_ptr() if x is not None else None
        d.d_out = outp.data_ptr() if outp is not None else None
        d.d_codes, d.d_scale_idx, d.d_row_norm = codes.data_ptr(), sidx.data_ptr(), rnorm.data_ptr()
        d.d_edges = it["edges"].data_ptr() if it.get("edges") is not None else None
        d.d_levels = it["levels"].data_ptr() if it.get("levels") is not None else None
        d.rows, d.cols = rows, it["cols"]
        d.ld = x.stride(0) if x is not None else it["cols"]
        d.ld_out = outp.stride(0) if outp is not None else it["cols"]
    return arr


def encode_batched(items, dtype, N, K, scale_bits, table):
    """items: dicts with x, codes, scale_idx, row_norm, edges, cols.  One launch."""
    arr = _descs(items)
    code = DTYPE_BF16 if dtype == torch.bfloat16 else DTYPE_F32
    _check(lib().pvq_encode_batched(arr, len(items), code, N, K, scale_bits, _ptr(table, torch.int32),
                                    _stream()), "pvq_encode_batched")


def decode_batched(items, N, K, scale_bits, table, status=None):
    """items: dicts with out, codes, scale_idx, row_norm, levels, cols.  One launch."""
    arr = _descs(items)
    _check(lib().pvq_decode_batched(arr, len(items), N, K, scale_bits, _ptr(table, torch.int32),
                                    _ptr(status, torch.int32), _stream()), "pvq_decode_batched")
