"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle
on the same seeded inputs.  Codes, amplitude indices, row norms and decoded bf16
values must match bit for bit."""
import numpy as np
import pytest
import torch

from oracle import beta_codebook as bc
from oracle import pvq_oracle as po
from paper_2410_16926_b200 import inputs, pvq

import blob_sections as bs

pytestmark = pytest.mark.gpu

DEV = "cuda"


def as_u32(t):
    return t.cpu().numpy().view(np.uint32)


def bf16_bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def to_device(x_np, kind):
    if kind == "bf16":
        return torch.from_numpy(x_np.view(np.int16)).to(DEV).view(torch.bfloat16)
    return torch.from_numpy(x_np).to(DEV)


class Codec:
    """Device tables for one (N, index_bits, G, scale_bits); the codebook is the oracle's,
    so that parity of the hot path does not hinge on two ways of computing quantiles."""

    def __init__(self, N, index_bits, G, b, K=None):
        self.N, self.G, self.b = N, G, b
        self.K = pvq.max_pulses(N, index_bits) if K is None else K
        self.W = pvq.code_words(N, self.K)
        self.table = pvq.build_count_table(N, self.K)
        self.edges_np = bc.edges_f32(N, G, b)
        self.levels_np = bc.levels_amp_f32(N, G, b)
        self.edges = torch.from_numpy(self.edges_np).to(DEV)
        self.levels = torch.from_numpy(self.levels_np).to(DEV)


GUARD = 64   # canary elements behind every output buffer


def guarded(shape, dtype, fill):
    """A tensor of `shape` whose storage is followed by GUARD canary elements; returns
    (tensor, check) where check() asserts that the canaries still hold `fill`."""
    n = int(np.prod(shape))
    flat = torch.full((n + GUARD,), fill, dtype=dtype, device=DEV)
    def check():
        assert bool((flat[n:] == fill).all()), "written past the end of an output buffer"
    return flat[:n].view(*shape), check


def check_encode(cd, x_np, kind, x_dev=None):
    x_dev = to_device(x_np, kind) if x_dev is None else x_dev
    rows = x_np.shape[0]
    codes, c1 = guarded((rows, cd.G, cd.W), torch.int32, 0x5A5A5A5A)
    sidx, c2 = guarded((rows, int(pvq.scale_row_stride(cd.G, cd.b))), torch.uint8, 0xA5)
    rnorm, c3 = guarded((rows,), torch.float32, 12345.0)
    pvq.encode(x_dev, cd.N, cd.K, cd.b, cd.table, cd.edges, out=(codes, sidx, rnorm))
    torch.cuda.synchronize()
    c1(), c2(), c3()
    o_codes, o_sidx, o_rnorm = po.encode(x_np, cd.N, cd.K, cd.b, cd.edges_np, W=cd.W)
    assert np.array_equal(rnorm.cpu().numpy().view(np.uint32), o_rnorm.view(np.uint32)), "row norms"
    assert np.array_equal(sidx.cpu().numpy(), o_sidx), "amplitude indices"
    bad = np.argwhere(as_u32(codes) != o_codes)
    assert bad.size == 0, "codes differ first at (row, group, word) %s" % (bad[0],)
    return (codes, sidx, rnorm), (o_codes, o_sidx, o_rnorm)


def check_decode(cd, enc_dev, enc_np):
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    rows, G, _ = enc_dev[0].shape
    out, c1 = guarded((rows, G * cd.N), torch.bfloat16, 7.0)
    pvq.decode(*enc_dev, cd.N, cd.K, cd.b, cd.table, cd.levels, status=status, out=out)
    torch.cuda.synchronize()
    c1()
    o_out, o_status = po.decode(*enc_np, cd.N, cd.K, cd.b, cd.levels_np)
    assert int(status.item()) == o_status
    bad = np.argwhere(bf16_bits(out) != o_out)
    assert bad.size == 0, "decoded values differ first at %s" % (bad[0],)
    return out


# ------------------------------------------------------------------ set-up kernels

@pytest.mark.parametrize("N,K", [(8, 6), (8, 40), (16, 18), (32, 22), (32, 50), (64, 96), (32, 1), (128, 187),
                                 (64, 405), (128, 386), (128, 782), (256, 369), (256, 760),
                                 (16, 1136), (32, 1858), (64, 3359), (128, 1576), (128, 6378), (32, 1024),
                                 (1, 1100), (2, 1500), (3, 2047), (8, 8191)])
def test_count_table_word_for_word(N, K):
    W = pvq.code_words(N, K)
    t = pvq.build_count_table(N, K)
    torch.cuda.synchronize()
    ref = po.count_table(N, K, W)[:N]          # rows n = 0..N-1
    assert np.array_equal(as_u32(pvq.count_table_view(t, N, K)), ref)


@pytest.mark.parametrize("N,K", [(8, 16), (16, 18), (32, 22), (32, 50), (32, 105), (64, 96), (64, 26), (128, 40),
                                 (64, 230), (128, 300), (256, 200), (16, 1136), (32, 1100)])
def test_table_blob_sections(N, K):
    """Every rearranged section of the table blob holds the numbers of the count table."""
    W = pvq.code_words(N, K)
    blob = as_u32(pvq.build_count_table(N, K))
    torch.cuda.synchronize()
    lay = bs.blob_layout(N, K, W)
    full = po.count_table(N, K, W + 1)                  # rows n = 0..N
    val = [[po.code_to_int(full[n, k]) for k in range(K + 1)] for n in range(N + 1)]
    srch = bs.section(val, N, K, W, lay["total"])
    want_bytes = lay["total"] if srch is None else srch["off"] + srch["total"]
    assert blob.size * 4 == want_bytes == pvq.count_table_bytes(N, K)
    mask = (1 << (32 * W)) - 1
    words = lambda v, nw: [(v >> (32 * w)) & 0xFFFFFFFF for w in range(nw)]
    bwn = lay["bound_words"]
    assert list(blob[lay["bound"] // 4: lay["bound"] // 4 + bwn]) == words(val[N][K], bwn)
    rowlen, top = lay["rowlen"], lay["top"]
    for name, sat_bits in (("walk_top", None), ("walk2", 62), ("walk1", 30)):
        off, nw = lay[name]
        if nw == 0:
            continue
        sec = blob[off // 4: off // 4 + N * rowlen * nw].reshape(N, rowlen, nw)
        for i in range(N):
            for col in range(K + 1):
                v = val[N - 1 - i][col]
                if sat_bits is not None and v >= (1 << sat_bits):
                    v = 1 << sat_bits
                assert list(sec[i, col]) == words(v, nw), (name, i, col)
    for name in ("enc_u", "enc_2v", "enc_v"):
        off = lay[name]
        sec = blob[off // 4: off // 4 + N * (K + 2) * top].reshape(N, K + 2, top)
        for i in range(N):
            V = [0]
            for col in range(K + 1):
                V.append(V[-1] + val[N - 1 - i][col])          # V[col + 1] = V(n, col), V[0] = V(n, -1)
            for c1 in range(K + 2):
                prev = V[c1 - 1] if c1 > 0 else 0
                want = {"enc_u": V[c1] + prev, "enc_2v": 2 * V[c1], "enc_v": V[c1]}[name] & mask
                assert list(sec[i, c1]) == words(want, top), (name, i, c1)
    if lay["walkd"] is not None:
        # the walk table as doubles, saturated at 2^53
        sec = blob[lay["walkd"] // 4: lay["walkd"] // 4 + N * rowlen * 2].view(np.float64).reshape(N, rowlen)
        for i in range(N):
            for col in range(K + 1):
                assert sec[i, col] == float(min(val[N - 1 - i][col], 1 << 53)), ("walkd", i, col)
        # U(n,k) = V(n,k) + V(n,k-1) with V(n,k) = sum_{j<=k} N(n,j) (App. C.2); U(-1, .) = 0
        def U(n, k):
            return 0 if n < 0 else 2 * sum(val[n][:k + 1]) - val[n][k]
        assert list(blob[lay["start"] // 4: lay["start"] // 4 + top]) == words(U(N - 1, K) & mask, top)
    if lay["cenc0"] is not None:
        for name, off in (("cenc0", lay["cenc0"]), ("cenc1", lay["cenc1"])):
            crow = lay["crow"]
            sec = blob[off // 4: off // 4 + N * crow * top].reshape(N, top, crow)      # rows of `top` word planes
            assert not sec[:, :, K + 1:].any()
            for i in range(N):
                n = N - 1 - i
                for k in range(K + 1):
                    sub = U(n, k) if name == "cenc0" else 2 * sum(val[n][:k + 1])
                    assert list(sec[i, :, k]) == words((U(n - 1, k) - sub) & mask, top), (name, i, k)
    if srch is not None:
        # the decoder's search section: header, row records, bucket tables, thresholds, increments
        sec = blob[srch["off"] // 4: (srch["off"] + srch["total"]) // 4]
        assert list(sec[:8]) == [bs.MAGIC, N, K, srch["total"]] + srch["counts"]
        for n in range(N):
            rec = sec[(srch["rec_off"] + 16 * n) // 4: (srch["rec_off"] + 16 * n) // 4 + 4]
            sh, nw, at, plane = srch["shifts"][n], srch["words"][n], srch["te_offs"][n], srch["plane"]
            want = [32 - sh, srch["e_off"] + at,
                    (srch["b_off"] + 4 * (srch["offs"][n] - (bs.KEY_OF_ONE >> sh))) & 0xFFFFFFFF, sh]
            assert list(rec) == want, ("record", n)
            b0 = srch["b_off"] // 4 + srch["offs"][n]
            assert list(sec[b0: b0 + srch["lens"][n]]) == srch["tables"][n], ("buckets", n)
            for name, vals in (("t_off", srch["T"]), ("e_off", srch["E"])):
                row = sec[(srch[name] + at) // 4: (srch[name] + at) // 4 + plane * nw].reshape(nw, plane)   # word planes
                for m in range(2 * K + 1):
                    assert list(row[:, m]) == words(vals[n][m], nw), (name, n, m)


@pytest.mark.parametrize("N,G,b", [(32, 16, 8), (32, 128, 4), (32, 448, 8), (64, 448, 6), (32, 128, 8),
                                   (8, 2, 3), (16, 5, 1)])
def test_scale_codebook_against_scipy(N, G, b):
    edges, levels = pvq.build_scale_codebook(N, G, b)
    torch.cuda.synchronize()
    e, l = edges.cpu().numpy(), levels.cpu().numpy()
    re_, rl = bc.edges_f32(N, G, b), bc.levels_amp_f32(N, G, b)
    # fp64 quantiles from two unrelated algorithms, each rounded once to fp32: at most one ulp apart
    assert np.all(np.abs(e.view(np.int32) - re_.view(np.int32)) <= 1)
    assert np.all(np.abs(l.view(np.int32) - rl.view(np.int32)) <= 1)
    assert np.mean(e.view(np.int32) == re_.view(np.int32)) > 0.98
    assert np.all(np.diff(e) > 0)


# ------------------------------------------------------------------------ hot path

SMALL = [
    # N, index_bits, rows, cols, scale_bits, dtype
    (8, 24, 7, 64, 3, "f32"),
    (8, 40, 5, 24, 5, "bf16"),       # G = 3
    (16, 40, 33, 208, 4, "bf16"),    # G = 13
    (32, 64, 70, 512, 8, "f32"),     # several tiles, ragged last tile
    (32, 96, 37, 4096, 4, "bf16"),   # G = 128
    (32, 96, 9, 14336, 8, "bf16"),   # G = 448: not a power of two
    (32, 128, 12, 1024, 6, "bf16"),  # 4-word codes
    (64, 192, 11, 3584, 6, "bf16"),  # N = 64, 6-word codes, G = 56
    (64, 64, 6, 640, 2, "f32"),      # few pulses per position
    (16, 48, 5, 14336, 4, "bf16"),   # G = 896: the paper's group size 16 on a 14336-column matrix (Sec. 4.1)
    (32, 96, 3, 28672, 8, "bf16"),   # G = 896 at group size 32: rows longer than a thread block
    (8, 24, 3, 32768, 4, "f32"),     # G = 4096: the longest row taken
    (32, 64, 5, 4800, 6, "f32"),     # G = 150: neither a power of two nor a multiple of 32
]


@pytest.mark.parametrize("N,bits,rows,cols,b,kind", SMALL)
def test_encode_decode_parity(N, bits, rows, cols, b, kind):
    rng = np.random.default_rng(N * 1000 + rows)
    x = (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
    x_np = inputs.f32_to_bf16_bits(x) if kind == "bf16" else x
    cd = Codec(N, bits, cols // N, b)
    enc_dev, enc_np = check_encode(cd, x_np, kind)
    check_decode(cd, enc_dev, enc_np)


def test_encode_status_word_stays_clear():
    # the encode-side calls report a staging time-out in the word of pvq_encode_status; on a
    # healthy run it stays zero and the results are those of a run without it
    rng = np.random.default_rng(77)
    x_np = inputs.f32_to_bf16_bits((rng.standard_normal((19, 2048)) * 0.02).astype(np.float32))
    cd = Codec(32, 96, 64, 4)
    word = torch.zeros(1, dtype=torch.int32, device=DEV)
    pvq.encode_status(word)
    try:
        check_encode(cd, x_np, "bf16")
        out = pvq.roundtrip(to_device(x_np, "bf16"), cd.N, cd.K, cd.b, cd.table, cd.edges, cd.levels)
        torch.cuda.synchronize()
    finally:
        pvq.encode_status(None)
    assert int(word.item()) == 0
    enc = po.encode(x_np, cd.N, cd.K, cd.b, cd.edges_np, W=cd.W)
    assert np.array_equal(bf16_bits(out), po.decode(*enc, cd.N, cd.K, cd.b, cd.levels_np)[0])


def test_heavy_tails_and_outliers():
    rng = np.random.default_rng(42)
    x = (rng.standard_t(2.0, size=(24, 1024)) * 0.05).astype(np.float32)
    x[3, 100] = 1e4
    x[5, :32] = 0.0
    x_np = inputs.f32_to_bf16_bits(x)
    cd = Codec(32, 96, 32, 8)
    enc_dev, enc_np = check_encode(cd, x_np, "bf16")
    check_decode(cd, enc_dev, enc_np)


def test_degenerate_inputs():
    N, rows, cols = 32, 12, 256
    x = np.zeros((rows, cols), dtype=np.float32)
    rng = np.random.default_rng(1)
    x[1] = rng.standard_normal(cols)              # ordinary row
    x[2, 40] = -3.0                               # one non-zero in the whole row
    x[3, :32] = 1.0                               # all-equal group: every residual ties
    x[3, 32:64] = -0.5
    x[4] = rng.standard_normal(cols)
    x[4, 64:96] = 0.0                             # zero group inside a non-zero row
    x[5] = -0.0                                   # negative zeros only
    x[6] = np.round(rng.standard_normal(cols) * 4) / 4      # many equal magnitudes
    x[7] = rng.standard_normal(cols) * 1e-30      # tiny values
    x[8] = rng.standard_normal(cols) * 1e15       # large but finite sums of squares
    x[9, ::2] = 1.0
    x[9, 1::2] = -1.0
    x[10, 5] = 1e-45                              # smallest subnormal: K / l1 overflows
    x[11] = rng.standard_normal(cols)
    x[11, 31] = 100.0                             # all pulses of a group in its last position
    cd = Codec(N, 64, cols // N, 8)
    for kind in ("f32", "bf16"):
        x_np = inputs.f32_to_bf16_bits(x) if kind == "bf16" else x
        enc_dev, enc_np = check_encode(cd, x_np, kind)
        check_decode(cd, enc_dev, enc_np)


@pytest.mark.parametrize("N,bits,b", [(32, 64, 8), (64, 192, 6), (128, 384, 16), (64, 256, 16)])
def test_non_finite_inputs_give_valid_codes(N, bits, b):
    """NaN, infinities and sums that overflow are outside the method (their result is left open), but
    every code written must be a valid one and the other rows must not notice."""
    rows, cols = 10, 8 * N
    rng = np.random.default_rng(N + b)
    x = (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
    x[1, 5] = np.nan
    x[3, N + 1] = np.inf
    x[3, 3 * N] = -np.inf
    x[5, :] = np.nan
    x[7, 2 * N: 3 * N] = 3e38                          # finite values, sums overflow
    x[8, 7] = -np.inf
    x[8, 9] = np.nan
    finite = np.array([0, 2, 4, 6, 9])
    K = pvq.max_pulses(N, bits)
    W = pvq.code_words(N, K)
    table = pvq.build_count_table(N, K)
    e_np = bc.edges_f32(N, cols // N, b) if b <= 8 else None
    l_np = bc.levels_amp_f32(N, cols // N, b) if b <= 8 else None
    edges = torch.from_numpy(e_np).to(DEV) if b <= 8 else None
    levels = torch.from_numpy(l_np).to(DEV) if b <= 8 else None
    codes, sidx, rnorm = pvq.encode(torch.from_numpy(x).to(DEV), N, K, b, table, edges)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out = pvq.decode(codes, sidx, rnorm, N, K, b, table, levels, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0                     # every code is below N(N,K)
    o_codes, o_sidx, o_rnorm = po.encode(np.ascontiguousarray(x[finite]), N, K, b, e_np, W=W)
    o_out, _ = po.decode(o_codes, o_sidx, o_rnorm, N, K, b, l_np)
    f = torch.from_numpy(finite).to(DEV)
    assert np.array_equal(as_u32(codes[f]), o_codes)
    assert np.array_equal(sidx[f].cpu().numpy(), o_sidx)
    assert np.array_equal(bf16_bits(out[f].contiguous()), o_out)


@pytest.mark.parametrize("N,bits,cols,ld,ldo", [(32, 96, 256, 320, 288), (128, 384, 1024, 1280, 1032),
                                               (64, 256, 512, 520, 640)])
def test_leading_dimensions(N, bits, cols, ld, ldo):
    rows = 10
    rng = np.random.default_rng(8)
    x = inputs.f32_to_bf16_bits((rng.standard_normal((rows, cols))).astype(np.float32))
    cd = Codec(N, bits, cols // N, 4)
    big = torch.zeros((rows, ld), dtype=torch.bfloat16, device=DEV)
    big[:, :cols] = to_device(x, "bf16")
    enc_dev, enc_np = check_encode(cd, x, "bf16", x_dev=big[:, :cols])
    out_big = torch.full((rows, ldo), 7.0, dtype=torch.bfloat16, device=DEV)
    pvq.decode(*enc_dev, cd.N, cd.K, cd.b, cd.table, cd.levels, out=out_big[:, :cols])
    torch.cuda.synchronize()
    o_out, _ = po.decode(*enc_np, cd.N, cd.K, cd.b, cd.levels_np)
    assert np.array_equal(bf16_bits(out_big[:, :cols].contiguous()), o_out)
    assert torch.all(out_big[:, cols:] == 7.0)       # nothing written past cols


@pytest.mark.parametrize("N,bits", [(32, 64), (128, 380), (64, 300)])
def test_invalid_codes_set_status_and_decode_to_zero(N, bits):
    cd = Codec(N, bits, 8, 8)
    W = cd.W
    rng = np.random.default_rng(5)
    x = rng.standard_normal((4, 8 * N)).astype(np.float32)
    enc_dev, enc_np = check_encode(cd, x, "f32")
    codes = enc_np[0].copy()
    codes[1, 3, :] = 0xFFFFFFFF                      # >= N(N,K)
    total = po.code_to_int(po.count_table(N, cd.K, W + 1)[N, cd.K])
    assert total < 1 << (32 * W)
    codes[2, 0, :] = po.int_to_code(total, W)         # the first invalid value
    codes[2, 1, :] = po.int_to_code(total - 1, W)     # the last valid one
    enc_np2 = (codes, enc_np[1], enc_np[2])
    enc_dev2 = (torch.from_numpy(codes.view(np.int32)).to(DEV), enc_dev[1], enc_dev[2])
    out = check_decode(cd, enc_dev2, enc_np2)
    assert torch.all(out[1, 3 * N:4 * N] == 0) and torch.all(out[2, :N] == 0)
    assert torch.any(out[2, N:2 * N] != 0)


def _random_codes(rng, total, shape, W):
    """Codes drawn uniformly from [0, total) with Python integers, as (..., W) uint32 words."""
    n = int(np.prod(shape))
    nbytes = (total.bit_length() + 7) // 8 + 8              # 64 spare bits: the modulo bias is below 2^-64
    raw = rng.integers(0, 256, size=(n, nbytes), dtype=np.uint8)
    out = np.empty((n, W), dtype=np.uint32)
    for j in range(n):
        out[j] = po.int_to_code(int.from_bytes(raw[j].tobytes(), "little") % total, W)
    return out.reshape(*shape, W)


@pytest.mark.parametrize("N,K", [(32, 22), (32, 50), (64, 96), (128, 187), (64, 199), (16, 27), (8, 40)])
def test_decode_of_codes_the_encoder_did_not_make(N, K):
    # Algorithm 3 on codes that come from no encoder: uniform over [0, N(N,K)), where the
    # remainder shrinks at a different pace than on encoded Gaussian data, and batches built so
    # that one thread of a warp keeps a wide remainder while the other 31 go narrow at once
    # (and the reverse), which is what decides when a warp may switch to narrower arithmetic.
    rows, G, b = 6, 64, 8
    cd = Codec(N, 0, G, b, K=K)
    W = cd.W
    total = po.code_to_int(po.count_table(N, K, W + 1)[N, K])
    rng = np.random.default_rng(1000 * N + K)
    codes = _random_codes(rng, total, (rows, G), W)
    big = po.int_to_code(total - 1, W)
    small = _random_codes(rng, min(total, 1 << 20), (rows, G), W)
    flat = codes.reshape(-1, W)
    sflat = small.reshape(-1, W)
    n = flat.shape[0]
    third = n // 3 // 32 * 32
    # second third: lane 0 of every warp holds N(N,K) - 1, the rest hold small codes
    flat[third:2 * third] = sflat[third:2 * third]
    flat[third:2 * third:32] = big
    # last third: lane 0 holds a small code, the rest hold large random ones (as drawn)
    flat[2 * third::32] = sflat[2 * third::32]
    flat[-1] = big
    flat[0] = 0
    sidx = rng.integers(0, 256, size=(rows, int(pvq.scale_row_stride(G, b))), dtype=np.uint8)
    rnorm = (rng.random(rows).astype(np.float32) + 0.5)
    enc_np = (codes, sidx, rnorm)
    enc_dev = (torch.from_numpy(codes.view(np.int32)).to(DEV), torch.from_numpy(sidx).to(DEV),
               torch.from_numpy(rnorm).to(DEV))
    check_decode(cd, enc_dev, enc_np)


@pytest.mark.parametrize("N,K", [(32, 50), (32, 22), (16, 27), (8, 40), (64, 31), (32, 105)])
def test_decode_of_codes_on_the_search_thresholds(N, K):
    """Codes whose running value sits on a threshold of the searching decoder, or next to one:
    points y = (a_0, ..., a_p, rest) where the rest is the first or the last point of its
    pyramid put the value of position p + 1 exactly on, or one beyond, a threshold, which the
    leading 24 bits cannot tell apart; also the neighbours of such codes."""
    from oracle import pvq_pyref as pr
    rows, G, b = 4, 64, 8
    cd = Codec(N, 0, G, b, K=K)
    W = cd.W
    count = pr.count_table(N, K)
    total = count[N][K]
    rng = np.random.default_rng(77 * N + K)
    want = rows * G
    ints = []
    while len(ints) < want:
        # a random prefix, then all remaining pulses on one late coordinate (first / last points of
        # the sub-pyramids behind the prefix), either sign
        p = int(rng.integers(0, N - 1))
        y = [0] * N
        left = K
        for i in range(p):
            if left == 0:
                break
            v = int(rng.integers(0, min(left, 4) + 1))
            y[i] = v if rng.integers(0, 2) else -v
            left -= v
        pos = int(rng.choice([p, N - 1]))
        y[pos] += left if rng.integers(0, 2) else -left
        if sum(abs(v) for v in y) != K:
            continue
        c = pr.enumerate_point(y, K)
        for d in (0, -1, 1):
            if 0 <= c + d < total:
                ints.append(c + d)
    codes = np.array([po.int_to_code(c, W) for c in ints[:want]], dtype=np.uint32).reshape(rows, G, W)
    if cd.W <= 4 and K <= 127:
        sec = bs.section(count, N, K, W, 0)
        if sec is not None:   # these inputs do reach the full compare
            ties = []
            for c in ints[:want]:
                bs.decode_with(sec, count, c, N, K, ties)
            assert len(ties) > want // 4
    sidx = rng.integers(0, 256, size=(rows, int(pvq.scale_row_stride(G, b))), dtype=np.uint8)
    rnorm = (rng.random(rows).astype(np.float32) + 0.5)
    enc_np = (codes, sidx, rnorm)
    enc_dev = (torch.from_numpy(codes.view(np.int32)).to(DEV), torch.from_numpy(sidx).to(DEV),
               torch.from_numpy(rnorm).to(DEV))
    check_decode(cd, enc_dev, enc_np)


@pytest.mark.parametrize("N,K", [(8, 1), (8, 2), (8, 3), (8, 17), (8, 64), (8, 100), (8, 127), (16, 1), (16, 5), (16, 33),
                                 (16, 64), (16, 90), (16, 127), (32, 1), (32, 2), (32, 7), (32, 31), (32, 32), (32, 63),
                                 (32, 64), (32, 77), (32, 104), (64, 1), (64, 2), (64, 9), (64, 20), (64, 31)])
def test_decode_across_pulse_counts(N, K):
    """Random codes, the first and the last code, and codes at the edges of the first coordinate's
    blocks, over pulse counts from one to the most that a byte per coordinate and four words per
    code allow: every table shape of the searching decoder (plane sizes, row widths, shifts)."""
    from oracle import pvq_pyref as pr
    rows, G, b = 3, 64, 8
    cd = Codec(N, 0, G, b, K=K)
    W = cd.W
    if W > 4:
        pytest.skip("more than four words: decoded by the walk, covered elsewhere")
    count = pr.count_table(N, K)
    total = count[N][K]
    rng = np.random.default_rng(5000 * N + K)
    codes = _random_codes(rng, total, (rows, G), W)
    flat = codes.reshape(-1, W)
    # block ends of position 0: N(N-1,K), then + 2 N(N-1,K-j) ... (Algorithm 3's subtractions), and their neighbours
    edge, special = count[N - 1][K], [0, total - 1]
    for j in range(1, K + 1):
        special += [edge - 1, edge, min(edge + 1, total - 1)]
        edge += 2 * count[N - 1][K - j]
    for i, c in enumerate(special[:flat.shape[0]]):
        flat[i] = po.int_to_code(max(0, min(c, total - 1)), W)
    sidx = rng.integers(0, 256, size=(rows, int(pvq.scale_row_stride(G, b))), dtype=np.uint8)
    rnorm = (rng.random(rows).astype(np.float32) + 0.5)
    enc_np = (codes, sidx, rnorm)
    enc_dev = (torch.from_numpy(codes.view(np.int32)).to(DEV), torch.from_numpy(sidx).to(DEV),
               torch.from_numpy(rnorm).to(DEV))
    check_decode(cd, enc_dev, enc_np)


def test_decode_refuses_a_table_built_for_other_parameters():
    """The searching decoder's look-ups follow what the table says, so it checks the header of
    its section first: with the table of another K nothing is decoded and the status says so."""
    N, G, b, rows = 32, 64, 8, 4
    cd = Codec(N, 0, G, b, K=50)
    assert pvq.code_words(N, 49) == cd.W
    assert pvq.count_table_bytes(N, 49) <= pvq.count_table_bytes(N, 50)
    rng = np.random.default_rng(3)
    codes = torch.from_numpy(rng.integers(0, 1 << 20, size=(rows, G, cd.W), dtype=np.int64).astype(np.int32)).to(DEV)
    sidx = torch.zeros((rows, int(pvq.scale_row_stride(G, b))), dtype=torch.uint8, device=DEV)
    rnorm = torch.ones(rows, dtype=torch.float32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out, check = guarded((rows, G * N), torch.bfloat16, 7.0)
    pvq.decode(codes, sidx, rnorm, N, 49, b, cd.table, cd.levels, status=status, out=out)   # cd.table is for K = 50
    torch.cuda.synchronize()
    check()
    assert int(status.item()) == pvq.STATUS_TABLE_MISMATCH
    assert bool((out == 7.0).all())


def test_fused_roundtrip_equals_encode_then_decode():
    for (N, bits, rows, cols, b, kind) in [(32, 64, 40, 4096, 8, "bf16"), (16, 40, 9, 208, 4, "f32"),
                                           (64, 192, 5, 3584, 6, "bf16")]:
        rng = np.random.default_rng(rows)
        x = rng.standard_normal((rows, cols)).astype(np.float32)
        x_np = inputs.f32_to_bf16_bits(x) if kind == "bf16" else x
        cd = Codec(N, bits, cols // N, b)
        out = pvq.roundtrip(to_device(x_np, kind), cd.N, cd.K, cd.b, cd.table, cd.edges, cd.levels)
        torch.cuda.synchronize()
        enc = po.encode(x_np, cd.N, cd.K, cd.b, cd.edges_np, W=cd.W)
        o_out, _ = po.decode(*enc, cd.N, cd.K, cd.b, cd.levels_np)
        assert np.array_equal(bf16_bits(out), o_out)


@pytest.mark.parametrize("N,bits,rows,cols,b,kind", [
    (128, 512, 6, 1024, 8, "bf16"),      # activations at group size 128, 4 bits of direction (Sec. 4.3)
    (128, 384, 9, 4096, 16, "bf16"),
    (64, 256, 5, 512, 6, "f32"),         # computed in 8 words
    (256, 768, 3, 1024, 16, "bf16"),     # computed in 32 words
    (128, 96, 4, 512, 4, "f32"),         # few pulses
])
def test_fused_roundtrip_global_table_kernels(N, bits, rows, cols, b, kind):
    rng = np.random.default_rng(rows + N)
    x = rng.standard_normal((rows, cols)).astype(np.float32)
    x[1, :N] = 0.0
    x_np = inputs.f32_to_bf16_bits(x) if kind == "bf16" else x
    K = pvq.max_pulses(N, bits)
    W = pvq.code_words(N, K)
    table = pvq.build_count_table(N, K)
    e_np = bc.edges_f32(N, cols // N, b) if b <= 8 else None
    l_np = bc.levels_amp_f32(N, cols // N, b) if b <= 8 else None
    edges = torch.from_numpy(e_np).to(DEV) if b <= 8 else None
    levels = torch.from_numpy(l_np).to(DEV) if b <= 8 else None
    out = pvq.roundtrip(to_device(x_np, kind), N, K, b, table, edges, levels)
    torch.cuda.synchronize()
    enc = po.encode(x_np, N, K, b, e_np, W=W)
    o_out, _ = po.decode(*enc, N, K, b, l_np)
    assert np.array_equal(bf16_bits(out), o_out)


@pytest.mark.parametrize("N,bits", [(32, 96), (128, 384), (64, 320)])
def test_batched_calls_match_single_calls(N, bits):
    """All matrices of a decoder layer in one launch, on the shared-memory kernels and (group size
    128; wide codes) on the global-table kernels, whose blocks then cover rows of different lengths."""
    wl = inputs.config3(scale_div=256)       # the seven matrices of a layer, 1/256 of the rows
    b = wl.scale_bits
    K = pvq.max_pulses(N, bits)
    W = pvq.code_words(N, K)
    table = pvq.build_count_table(N, K)
    items, refs = [], []
    books = {}
    for m in wl.matrices:
        G = m.cols // N
        if G not in books:
            books[G] = (bc.edges_f32(N, G, b), bc.levels_amp_f32(N, G, b))
        e_np, l_np = books[G]
        codes, sidx, rnorm = pvq.alloc_encoded(m.rows, G, W, b)
        items.append(dict(x=to_device(m.data, "bf16"), codes=codes, scale_idx=sidx, row_norm=rnorm,
                          edges=torch.from_numpy(e_np).to(DEV), levels=torch.from_numpy(l_np).to(DEV),
                          out=torch.empty((m.rows, m.cols), dtype=torch.bfloat16, device=DEV), cols=m.cols))
        enc = po.encode(m.data, N, K, b, e_np, W=W)
        refs.append((enc, po.decode(*enc, N, K, b, l_np)[0]))
    pvq.encode_batched(items, torch.bfloat16, N, K, b, table)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    pvq.decode_batched(items, N, K, b, table, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for it, (enc, out) in zip(items, refs):
        assert np.array_equal(as_u32(it["codes"]), enc[0])
        assert np.array_equal(it["scale_idx"].cpu().numpy(), enc[1])
        assert np.array_equal(it["row_norm"].cpu().numpy().view(np.uint32), enc[2].view(np.uint32))
        assert np.array_equal(bf16_bits(it["out"]), out)


def test_library_codebook_end_to_end():
    # With the library's own codebook the amplitude indices may differ from the oracle's only
    # where u sits within an ulp of an edge; the direction codes do not depend on it.
    N, G, b = 32, 128, 4
    wl = inputs.config2(rows=64)
    x_np = wl.matrices[0].data
    K = pvq.max_pulses(N, 96)
    table = pvq.build_count_table(N, K)
    edges, levels = pvq.build_scale_codebook(N, G, b)
    codes, sidx, rnorm = pvq.encode(to_device(x_np, "bf16"), N, K, b, table, edges)
    torch.cuda.synchronize()
    o_codes, o_sidx, o_rnorm = po.encode(x_np, N, K, b, bc.edges_f32(N, G, b))
    assert np.array_equal(as_u32(codes), o_codes)
    q = po.unpack_scale_idx(sidx.cpu().numpy(), G, b)
    oq = po.unpack_scale_idx(o_sidx, G, b)
    assert np.mean(q != oq) < 1e-3 and np.max(np.abs(q - oq)) <= 1
    # uniform bin occupancy on Gaussian rows (Sec. 3.4): every 4-bit bin near 1/16
    occ = np.bincount(q.ravel(), minlength=16) / q.size
    assert np.all(np.abs(occ - 1 / 16) < 0.02)


# ------------------------------------------------------------- rotation on the fly

@pytest.mark.parametrize("N,bits,rows,cols,block,b,kind", [
    (32, 64, 37, 4096, 4096, 8, "bf16"),     # a block spans 128 threads: shuffles and shared memory
    (32, 96, 9, 14336, 512, 8, "bf16"),      # 16 threads per block: shuffles only; G = 448
    (32, 64, 21, 512, 32, 8, "f32"),         # block = group: in-thread stages only
    (16, 40, 11, 192, 64, 4, "f32"),         # G = 12, three blocks per row
    (64, 192, 5, 3584, 512, 6, "bf16"),      # N = 64
    # the kernels with the tables in global memory
    (128, 512, 5, 4096, 4096, 8, "bf16"),    # activations at group size 128: a block spans 32 threads
    (128, 384, 3, 1024, 128, 8, "f32"),      # block = group
    (128, 256, 4, 2048, 512, 6, "bf16"),     # four threads per block
    (64, 256, 6, 1024, 256, 8, "f32"),       # wide codes at N = 64
    (256, 768, 2, 2048, 1024, 8, "bf16"),    # N = 256
    (128, 384, 2, 16384, 16384, 4, "bf16"),  # a block of 128 threads
])
def test_rotate_encode_and_roundtrip_parity(N, bits, rows, cols, block, b, kind):
    rng = np.random.default_rng(block + rows)
    x = rng.standard_normal((rows, cols)).astype(np.float32)
    x[:, 3] *= 20.0                                            # an outlier channel to spread
    x_np = inputs.f32_to_bf16_bits(x) if kind == "bf16" else x
    signs = (rng.integers(0, 2, size=block) * 2 - 1).astype(np.float32)
    cd = Codec(N, bits, cols // N, b)
    xr = po.rotate(x_np, block, signs)                         # oracle: rotate, then the usual path
    o_codes, o_sidx, o_rnorm = po.encode(xr, cd.N, cd.K, cd.b, cd.edges_np, W=cd.W)
    o_out, _ = po.decode(o_codes, o_sidx, o_rnorm, cd.N, cd.K, cd.b, cd.levels_np)
    x_dev = to_device(x_np, kind)
    s_dev = torch.from_numpy(signs).to(DEV)
    codes, sidx, rnorm = pvq.rotate_encode(x_dev, block, s_dev, cd.N, cd.K, cd.b, cd.table, cd.edges)
    torch.cuda.synchronize()
    assert np.array_equal(rnorm.cpu().numpy().view(np.uint32), o_rnorm.view(np.uint32)), "row norms"
    assert np.array_equal(sidx.cpu().numpy(), o_sidx), "amplitude indices"
    assert np.array_equal(as_u32(codes), o_codes), "codes"
    global_tables = cd.W > {8: 2, 16: 3, 32: 4, 64: 6}.get(N, 0)
    if cd.K <= 127 or global_tables:
        out = pvq.rotate_roundtrip(x_dev, block, s_dev, cd.N, cd.K, cd.b, cd.table, cd.edges, cd.levels)
        torch.cuda.synchronize()
        assert np.array_equal(bf16_bits(out), o_out), "fused round trip"


def test_rotate_rejects_bad_blocks():
    cd = Codec(32, 64, 8, 8)
    x = torch.zeros((4, 256), dtype=torch.float32, device=DEV)
    s = torch.ones(256, dtype=torch.float32, device=DEV)
    for block in (0, 16, 48, 512):          # zero, below N, not a power of two, not dividing cols
        with pytest.raises(pvq.PvqError):
            pvq.rotate_encode(x, block, s, cd.N, cd.K, cd.b, cd.table, cd.edges)


# ------------------------------------- 16-bit amplitudes and the least-squares amplitude

@pytest.mark.parametrize("N,bits,rows,cols,b,amp_mode,kind", [
    (32, 96, 19, 4096, 16, 0, "bf16"),
    (32, 96, 19, 4096, 16, 1, "bf16"),
    (32, 64, 33, 512, 8, 1, "f32"),
    (16, 40, 9, 208, 16, 1, "f32"),       # G = 13
    (64, 192, 5, 3584, 16, 0, "bf16"),
    (32, 96, 7, 14336, 4, 1, "bf16"),
])
def test_amplitude_variants_parity(N, bits, rows, cols, b, amp_mode, kind):
    rng = np.random.default_rng(rows * 7 + b + amp_mode)
    x = (rng.standard_t(4.0, size=(rows, cols)) * 0.03).astype(np.float32)
    x[0, :N] = 0.0                                             # a group without direction
    x_np = inputs.f32_to_bf16_bits(x) if kind == "bf16" else x
    G = cols // N
    K = pvq.max_pulses(N, bits)
    W = pvq.code_words(N, K)
    table = pvq.build_count_table(N, K)
    e_np = bc.edges_f32(N, G, b) if b <= 8 else None
    l_np = bc.levels_amp_f32(N, G, b) if b <= 8 else None
    edges = torch.from_numpy(e_np).to(DEV) if b <= 8 else None
    levels = torch.from_numpy(l_np).to(DEV) if b <= 8 else None
    o_codes, o_sidx, o_rnorm = po.encode(x_np, N, K, b, e_np, W=W, amp_mode=amp_mode)
    o_out, _ = po.decode(o_codes, o_sidx, o_rnorm, N, K, b, l_np)
    codes, sidx, rnorm = pvq.encode(to_device(x_np, kind), N, K, b, table, edges, amp_mode=amp_mode)
    torch.cuda.synchronize()
    assert np.array_equal(as_u32(codes), o_codes), "codes"
    assert np.array_equal(sidx.cpu().numpy(), o_sidx), "amplitudes"
    assert np.array_equal(rnorm.cpu().numpy().view(np.uint32), o_rnorm.view(np.uint32)), "row norms"
    out = pvq.decode(codes, sidx, rnorm, N, K, b, table, levels)
    torch.cuda.synchronize()
    assert np.array_equal(bf16_bits(out), o_out), "decoded"
    if amp_mode == 0 and K <= 127:                             # the fused kernel, 16-bit amplitudes included
        rt = pvq.roundtrip(to_device(x_np, kind), N, K, b, table, edges, levels)
        torch.cuda.synchronize()
        assert np.array_equal(bf16_bits(rt), o_out), "fused"


def test_qsnr_curve_on_a_gaussian_source_equals_the_oracles():
    # the quality experiment of Sec. 2.6 / Fig. 3 (PVQ curve) through the CUDA path
    rng = np.random.default_rng(0)
    x = rng.standard_normal((128, 1024)).astype(np.float32)
    xd = torch.from_numpy(x).to(DEV)
    curve = []
    for bpw in (2.0, 3.0, 4.0):
        N, bits = 32, int(bpw * 32)
        K = pvq.max_pulses(N, bits)
        table = pvq.build_count_table(N, K)
        enc = pvq.encode(xd, N, K, 16, table, None, amp_mode=1)
        out = pvq.decode(*enc, N, K, 16, table, None).float()
        torch.cuda.synchronize()
        q_gpu = 10 * torch.log10((xd.double() ** 2).sum() / ((xd.double() - out.double()) ** 2).sum()).item()
        c, s, r = po.encode(x, N, K, 16, W=(bits + 31) // 32, amp_mode=1)
        o, _ = po.decode(c, s, r, N, K, 16)
        xh = inputs.bf16_bits_to_f32(o).astype(np.float64)
        q_cpu = 10 * np.log10((x.astype(np.float64) ** 2).sum() / ((x - xh) ** 2).sum())
        assert abs(q_gpu - q_cpu) < 1e-9
        curve.append(q_gpu)
    assert curve[0] < curve[1] < curve[2] and 9.5 < curve[0] < 10.5


# -------------------------------------- large groups and wide codes (tables in global memory)

@pytest.mark.parametrize("N,bits,rows,cols,b,amp_mode,kind", [
    (128, 384, 9, 4096, 16, 0, "bf16"),      # the paper's 3 bits + 16-bit amplitudes at group size 128
    (128, 384, 5, 14336, 16, 1, "bf16"),     # G = 112, least-squares amplitudes
    (128, 256, 7, 1024, 8, 0, "f32"),        # 8-word codes, quantile amplitudes
    (128, 96, 6, 512, 4, 0, "f32"),          # few pulses: K below 128, byte slots
    # the rest of the paper's grid of group sizes and direction bits (Sec. 4.1) that fits 1023 pulses
    (16, 112, 6, 256, 4, 0, "f32"),          # 7 bits per weight at group size 16: 4 words
    (32, 160, 7, 512, 8, 0, "bf16"),         # 5 bits per weight: 5 words
    (32, 192, 3, 256, 16, 1, "bf16"),        # 6 bits per weight
    (64, 256, 5, 1024, 6, 1, "bf16"),        # 4 bits per weight: 8 words
    (64, 320, 4, 512, 16, 0, "f32"),         # 5 bits per weight: 10 words, computed in 16
    (128, 512, 5, 1024, 16, 0, "bf16"),      # 4 bits per weight: 16 words
    (128, 640, 3, 512, 16, 0, "f32"),        # 5 bits per weight: 20 words, computed in 32
    (256, 768, 3, 1024, 16, 0, "bf16"),      # group size 256 at 3 bits per weight: 24 words
    (256, 1024, 3, 512, 16, 1, "f32"),       # 4 bits per weight: 32 words
    (256, 192, 4, 512, 8, 0, "bf16"),        # group size 256 with a short code
    # more than 1023 pulses: the high-rate end of the grid
    (16, 128, 5, 256, 8, 0, "bf16"),         # 8 bits per weight at group size 16: K = 1136
    (32, 256, 4, 256, 16, 1, "f32"),         # 8 bits per weight at group size 32: K = 1858
    (64, 512, 3, 512, 16, 0, "bf16"),        # 8 bits per weight at group size 64: K = 3359, 16 words
    (128, 768, 3, 512, 16, 1, "f32"),        # 6 bits per weight at group size 128: K = 1576, 24 words
    (128, 1024, 3, 512, 16, 1, "bf16"),      # 8 bits per weight at group size 128: K = 6378, 32 words
])
def test_large_group_parity(N, bits, rows, cols, b, amp_mode, kind):
    rng = np.random.default_rng(bits + rows)
    x = (rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)
    x[1, :N] = 0.0
    x[2, N:2 * N] = np.round(x[2, N:2 * N] * 200) / 200            # many equal magnitudes: ties
    x_np = inputs.f32_to_bf16_bits(x) if kind == "bf16" else x
    G = cols // N
    K = pvq.max_pulses(N, bits)
    W = pvq.code_words(N, K)
    table = pvq.build_count_table(N, K)
    e_np = bc.edges_f32(N, G, b) if b <= 8 else None
    l_np = bc.levels_amp_f32(N, G, b) if b <= 8 else None
    edges = torch.from_numpy(e_np).to(DEV) if b <= 8 else None
    levels = torch.from_numpy(l_np).to(DEV) if b <= 8 else None
    o_codes, o_sidx, o_rnorm = po.encode(x_np, N, K, b, e_np, W=W, amp_mode=amp_mode)
    o_out, _ = po.decode(o_codes, o_sidx, o_rnorm, N, K, b, l_np)
    codes, sidx, rnorm = pvq.encode(to_device(x_np, kind), N, K, b, table, edges, amp_mode=amp_mode)
    torch.cuda.synchronize()
    assert np.array_equal(rnorm.cpu().numpy().view(np.uint32), o_rnorm.view(np.uint32)), "row norms"
    assert np.array_equal(sidx.cpu().numpy(), o_sidx), "amplitudes"
    bad = np.argwhere(as_u32(codes) != o_codes)
    assert bad.size == 0, "codes differ first at %s" % (bad[0],)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out = pvq.decode(codes, sidx, rnorm, N, K, b, table, levels, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(bf16_bits(out), o_out), "decoded"


# ------------------------------------------------------------ seeded random configurations

def _random_case(seed):
    rng = np.random.default_rng(9000 + seed)
    N = int(rng.choice([8, 16, 32, 64, 128, 256]))
    max_bits = {8: 64, 16: 128, 32: 256, 64: 512, 128: 1024, 256: 1024}[N]
    bits = int(rng.integers(max(N // 2, 8), max_bits + 1))
    G = int(rng.integers(2, 24))
    rows = int(rng.integers(1, 8))
    b = int(rng.choice([1, 2, 3, 4, 5, 6, 7, 8, 16]))
    kind = str(rng.choice(["f32", "bf16"]))
    amp_mode = int(rng.integers(0, 2))
    dist = str(rng.choice(["gauss", "student", "sparse"]))
    return N, bits, G, rows, b, kind, amp_mode, dist


@pytest.mark.parametrize("seed", range(40))
def test_random_configuration_parity(seed):
    N, bits, G, rows, b, kind, amp_mode, dist = _random_case(seed)
    K = pvq.max_pulses(N, bits)
    if K < 1:
        pytest.skip("no pulse fits %d bits at N = %d" % (bits, N))
    W = pvq.code_words(N, K)
    rng = np.random.default_rng(seed)
    cols = N * G
    if dist == "gauss":
        x = rng.standard_normal((rows, cols)) * 0.02
    elif dist == "student":
        x = rng.standard_t(3.0, size=(rows, cols))
    else:
        x = rng.standard_normal((rows, cols)) * (rng.random((rows, cols)) < 0.15)
    x = x.astype(np.float32)
    x_np = inputs.f32_to_bf16_bits(x) if kind == "bf16" else x
    table = pvq.build_count_table(N, K)
    e_np = bc.edges_f32(N, G, b) if b <= 8 else None
    l_np = bc.levels_amp_f32(N, G, b) if b <= 8 else None
    edges = torch.from_numpy(e_np).to(DEV) if b <= 8 else None
    levels = torch.from_numpy(l_np).to(DEV) if b <= 8 else None
    o_codes, o_sidx, o_rnorm = po.encode(x_np, N, K, b, e_np, W=W, amp_mode=amp_mode)
    o_out, o_st = po.decode(o_codes, o_sidx, o_rnorm, N, K, b, l_np)
    codes, sidx, rnorm = pvq.encode(to_device(x_np, kind), N, K, b, table, edges, amp_mode=amp_mode)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out = pvq.decode(codes, sidx, rnorm, N, K, b, table, levels, status=status)
    torch.cuda.synchronize()
    what = "N=%d bits=%d K=%d W=%d G=%d rows=%d b=%d %s amp_mode=%d %s" % (N, bits, K, W, G, rows, b, kind, amp_mode, dist)
    assert np.array_equal(rnorm.cpu().numpy().view(np.uint32), o_rnorm.view(np.uint32)), what
    assert np.array_equal(sidx.cpu().numpy(), o_sidx), what
    assert np.array_equal(as_u32(codes), o_codes), what
    assert int(status.item()) == o_st == 0, what
    assert np.array_equal(bf16_bits(out), o_out), what

