"""CPU-only checks of the C-ABI library: it loads, exports what include/pvq.h
declares, its host helpers agree with the oracle, and bad arguments are turned
into status codes before any CUDA work."""
import ctypes as C
import os
import re

import pytest

from oracle import pvq_oracle as po
from paper_2410_16926_b200 import pvq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "pvq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pvq_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = pvq.lib()
    names = declared_functions()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(pvq.EXPORTS) == names


def test_strerror():
    for s in range(0, 7):
        assert pvq.lib().pvq_strerror(s)
    assert b"OK" in pvq.lib().pvq_strerror(0)


@pytest.mark.parametrize("N,bits", [(32, 64), (32, 96), (64, 192), (16, 40), (8, 24), (128, 384), (64, 320), (128, 512), (256, 768), (32, 256), (128, 768)])
def test_pulse_selection_matches_oracle(N, bits):
    K = pvq.max_pulses(N, bits)
    assert K == po.max_pulses(N, bits)
    assert pvq.index_bits(N, K) == po.index_bits(N, K) <= bits
    assert pvq.index_bits(N, K + 1) > bits
    W = pvq.code_words(N, K)
    assert W == (bits + 31) // 32
    assert pvq.count_table_bytes(N, K) >= N * (K + 1) * W * 4      # the count table is the blob's first section


@pytest.mark.parametrize("N,K", [(8, 6), (8, 40), (16, 18), (16, 40), (32, 22), (32, 30), (32, 50), (32, 105),
                                 (32, 127), (64, 26), (64, 31), (64, 96), (128, 40), (32, 1), (16, 127)])
def test_blob_size_counts_the_search_section(N, K):
    """The host lays out the search section from exact thresholds: its size is the one a plain
    Python computation from the oracle's count table gives (shifts, bucket-table lengths)."""
    import blob_sections as bs
    from oracle import pvq_pyref as pr
    W = pvq.code_words(N, K)
    lay = bs.blob_layout(N, K, W)
    srch = bs.section(pr.count_table(N, K), N, K, W, lay["total"])
    want = lay["total"] if srch is None else srch["off"] + srch["total"]
    assert pvq.count_table_bytes(N, K) == want
    if (N, K) in ((32, 50), (32, 22), (16, 18), (64, 31)):
        assert srch is not None
    if (N, K) in ((64, 96), (128, 40), (32, 127)):
        assert srch is None


@pytest.mark.parametrize("N,K", [(4, 3), (4, 5), (4, 8), (8, 3)])
def test_search_recipe_is_algorithm_3_exhaustively(N, K):
    """Decoding by one threshold search per position (the tables of the blob's search section,
    here built in Python) gives the point of Algorithm 3 for every code of small pyramids."""
    import blob_sections as bs
    from oracle import pvq_pyref as pr
    count = pr.count_table(N, K)
    sec = bs.section(count, N, K, 1, 0)
    assert sec is not None
    for code in range(count[N][K]):
        y, ok = pr.deenumerate_code(code, N, K)
        assert ok and bs.decode_with(sec, count, code, N, K) == y


@pytest.mark.parametrize("N,K,W", [(32, 50, 3), (32, 22, 2), (16, 40, 2), (8, 60, 2), (64, 31, 4)])
def test_search_recipe_is_algorithm_3_on_random_codes(N, K, W):
    import random
    import blob_sections as bs
    from oracle import pvq_pyref as pr
    count = pr.count_table(N, K)
    sec = bs.section(count, N, K, W, 0)
    assert sec is not None
    rnd = random.Random(N * 1000 + K)
    total = count[N][K]
    for code in [0, 1, total - 1, total // 2] + [rnd.randrange(total) for _ in range(200)]:
        y, ok = pr.deenumerate_code(code, N, K)
        assert ok and bs.decode_with(sec, count, code, N, K) == y
    # the most lopsided points: all pulses on one coordinate, either sign
    for pos in (0, N // 2, N - 1):
        for sign in (1, -1):
            y = [0] * N
            y[pos] = sign * K
            assert bs.decode_with(sec, count, pr.enumerate_point(y, K), N, K) == y


def test_index_bits_small_cases():
    # N(2,7) = 28 -> 5 bits; N(1,k) = 2 -> 1 bit; N(n,0) = 1 -> 0 bits
    assert pvq.index_bits(2, 7) == 5
    assert pvq.index_bits(1, 9) == 1
    assert pvq.index_bits(5, 0) == 0
    for n in range(1, 12):
        for k in range(0, 12):
            assert pvq.index_bits(n, k) == po.index_bits(n, k)


def test_scale_row_stride():
    for G in (1, 2, 5, 16, 128, 448, 1000):
        for b in range(1, 9):
            assert pvq.scale_row_stride(G, b) == po.scale_row_stride(G, b)
    assert pvq.scale_row_stride(128, 4) == 64
    assert pvq.scale_row_stride(448, 6) == 336
    assert pvq.scale_row_stride(5, 3) == 4


def test_bad_arguments_are_rejected_without_a_gpu():
    L = pvq.lib()
    buf = (C.c_uint32 * 64)()
    p = C.cast(buf, C.c_void_p)
    INVALID, UNSUPPORTED, ALIGN, SMALL = 1, 2, 3, 4
    # table builder
    assert L.pvq_build_count_table(32, 22, None, 1 << 20, None) == INVALID
    assert L.pvq_build_count_table(0, 22, p, 1 << 20, None) == INVALID
    assert L.pvq_build_count_table(32, 22, p, 16, None) == SMALL
    assert L.pvq_build_count_table(32, 9000, p, 1 << 30, None) == UNSUPPORTED
    assert L.pvq_build_count_table(32, 22, C.c_void_p(p.value + 4), 1 << 20, None) == ALIGN
    # codebook
    assert L.pvq_build_scale_codebook(32, 1, 4, p, p, None) == INVALID
    assert L.pvq_build_scale_codebook(32, 16, 9, p, p, None) == INVALID
    assert L.pvq_build_scale_codebook(31, 16, 4, p, p, None) == INVALID
    assert L.pvq_build_scale_codebook(32, 16, 4, None, None, None) == INVALID
    # encode
    enc = lambda x=p, dt=1, rows=4, cols=64, ld=64, N=32, K=22, b=8, tab=p, e=p, c=p, s=p, r=p: \
        L.pvq_encode(x, dt, rows, cols, ld, N, K, b, tab, e, c, s, r, None)
    assert enc(x=None) == INVALID
    assert enc(cols=48) == INVALID          # not a multiple of N
    assert enc(N=24) == INVALID             # not a power of two
    assert enc(b=0) == INVALID
    assert enc(dt=7) == INVALID
    assert enc(ld=32) == INVALID            # ld < cols
    assert enc(cols=32, ld=32) == UNSUPPORTED   # one group per row: no quantile codebook
    assert enc(N=512, cols=1024, ld=1024) == UNSUPPORTED
    assert enc(ld=68) == ALIGN
    assert enc(x=C.c_void_p(p.value + 2)) == ALIGN
    assert enc(tab=None) == INVALID
    assert enc(e=None) == INVALID
    assert enc(K=0) == INVALID
    # decode
    dec = lambda c=p, s=p, r=p, rows=4, cols=64, N=32, K=22, b=8, tab=p, lev=p, out=p, ldo=64: \
        L.pvq_decode(c, s, r, rows, cols, N, K, b, tab, lev, out, ldo, None, None)
    assert dec(out=None) == INVALID
    assert dec(c=None) == INVALID
    assert dec(lev=None) == INVALID
    assert dec(ldo=60) == INVALID
    assert dec(ldo=68) == ALIGN
    assert dec(rows=0) == INVALID
    # batched
    assert L.pvq_encode_batched(None, 1, 1, 32, 22, 8, p, None) == INVALID
    d = (pvq.MatrixDesc * 1)()
    assert L.pvq_encode_batched(d, 0, 1, 32, 22, 8, p, None) == INVALID
    assert L.pvq_encode_batched(d, 33, 1, 32, 22, 8, p, None) == INVALID
    assert L.pvq_decode_batched(d, 1, 32, 22, 8, p, None, None) == INVALID   # empty descriptor


def _build_c_example(tmp_path):
    """The plain C consumer of the library (no Python, no torch), built with gcc."""
    import shutil
    import subprocess
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    pkg = os.path.join(root, "paper_2410_16926_b200")
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    if shutil.which("gcc") is None or not os.path.isdir(os.path.join(cuda, "include")):
        pytest.skip("needs gcc and the CUDA headers")
    exe = str(tmp_path / "roundtrip_c")
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(root, "include"),
                    "-I", os.path.join(cuda, "include"), os.path.join(pkg, "examples", "roundtrip.c"),
                    "-L", pkg, "-lpvq_b200", "-L", os.path.join(cuda, "lib64"), "-lcudart", "-lm", "-o", exe],
                   check=True)
    env = dict(os.environ, LD_LIBRARY_PATH=pkg + ":" + os.path.join(cuda, "lib64") + ":" +
               os.environ.get("LD_LIBRARY_PATH", ""))
    return exe, env


def test_c_example_builds_against_the_header(tmp_path):
    """include/pvq.h is plain C and the library links from C; without a GPU the program gets as
    far as the host helpers and stops at its first CUDA call."""
    import subprocess
    pvq.lib()
    exe, env = _build_c_example(tmp_path)
    r = subprocess.run([exe], env=env, capture_output=True, text=True, timeout=120)
    assert "N=32 K=50 W=3 table" in r.stdout
    assert r.returncode in (0, 3)          # 3: no CUDA device here


@pytest.mark.gpu
def test_c_example_round_trip_on_the_gpu(tmp_path):
    import subprocess
    pvq.lib()
    exe, env = _build_c_example(tmp_path)
    r = subprocess.run([exe], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "status 0, QSNR" in r.stdout

