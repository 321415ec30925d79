"""GPU parity at the full benchmark sizes, in the launch configuration bench.py times.

The kernels run on the whole workload (so that grids, tiles per block and table staging are
the benchmark's); the oracle then recomputes a seeded sample of rows one by one (every row
for the smallest workloads) and those rows must match bit for bit: direction codes,
amplitude indices, row norms and decoded bf16 values.
"""
import numpy as np
import pytest
import torch

from oracle import beta_codebook as bc
from oracle import pvq_oracle as po
from paper_2410_16926_b200 import inputs, pvq

pytestmark = pytest.mark.gpu

DEV = "cuda"


def dev_bf16(bits):
    return torch.from_numpy(bits.view(np.int16)).to(DEV).view(torch.bfloat16)


def bf16_bits(t):
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def sample_rows(rows, n, seed):
    if rows <= n:
        return np.arange(rows)
    rng = np.random.default_rng(seed)
    pick = rng.choice(rows, size=n - 2, replace=False)
    return np.unique(np.concatenate([pick, [0, rows - 1]]))       # first and last rows always


def workload_items(wl, K, W):
    N, b = wl.N, wl.scale_bits
    items, books = [], {}
    for m in wl.matrices:
        G = m.cols // N
        if G not in books and b <= 8:
            e_np, l_np = bc.edges_f32(N, G, b), bc.levels_amp_f32(N, G, b)
            books[G] = (e_np, l_np, torch.from_numpy(e_np).to(DEV), torch.from_numpy(l_np).to(DEV))
        elif G not in books:                # 16-bit amplitudes use no codebook
            books[G] = (None, None, None, None)
        e_np, l_np, e_d, l_d = books[G]
        codes, sidx, rnorm = pvq.alloc_encoded(m.rows, G, W, b)
        x = dev_bf16(m.data) if m.dtype == "bf16" else torch.from_numpy(m.data).to(DEV)
        items.append(dict(x=x, codes=codes, scale_idx=sidx, row_norm=rnorm, edges=e_d, levels=l_d, cols=m.cols,
                          out=torch.empty((m.rows, m.cols), dtype=torch.bfloat16, device=DEV),
                          e_np=e_np, l_np=l_np))
    return items


def check_rows(wl, items, K, W, nrows, what):
    """Oracle on sampled rows of every matrix against what the GPU wrote for those rows."""
    N, b = wl.N, wl.scale_bits
    for mi, (m, it) in enumerate(zip(wl.matrices, items)):
        rows = sample_rows(m.rows, nrows, seed=100 + mi)
        x = np.ascontiguousarray(m.data[rows])
        o_codes, o_sidx, o_rnorm = po.encode(x, N, K, b, it["e_np"], W=W)
        if "codes" in what:
            r = torch.from_numpy(rows).to(DEV)
            assert np.array_equal(it["codes"][r].cpu().numpy().view(np.uint32), o_codes), m.name
            assert np.array_equal(it["scale_idx"][r].cpu().numpy(), o_sidx), m.name
            assert np.array_equal(it["row_norm"][r].cpu().numpy().view(np.uint32), o_rnorm.view(np.uint32)), m.name
        if "out" in what:
            o_out, st = po.decode(o_codes, o_sidx, o_rnorm, N, K, b, it["l_np"])
            assert st == 0
            r = torch.from_numpy(rows).to(DEV)
            assert np.array_equal(bf16_bits(it["out"][r].contiguous()), o_out), m.name


def test_c2_q_proj_every_row():
    wl = inputs.config2()
    K = pvq.max_pulses(wl.N, wl.index_bits)
    W = pvq.code_words(wl.N, K)
    table = pvq.build_count_table(wl.N, K)
    items = workload_items(wl, K, W)
    pvq.encode_batched(items, torch.bfloat16, wl.N, K, wl.scale_bits, table)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    pvq.decode_batched(items, wl.N, K, wl.scale_bits, table, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    check_rows(wl, items, K, W, nrows=4096, what=("codes", "out"))


def test_c3_decoder_layer_batched_sampled_rows():
    wl = inputs.config3()
    K = pvq.max_pulses(wl.N, wl.index_bits)
    W = pvq.code_words(wl.N, K)
    table = pvq.build_count_table(wl.N, K)
    items = workload_items(wl, K, W)
    pvq.encode_batched(items, torch.bfloat16, wl.N, K, wl.scale_bits, table)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    pvq.decode_batched(items, wl.N, K, wl.scale_bits, table, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    check_rows(wl, items, K, W, nrows=96, what=("codes", "out"))


def test_c4_down_proj_70b_decode_sampled_rows():
    wl = inputs.config4()
    K = pvq.max_pulses(wl.N, wl.index_bits)
    W = pvq.code_words(wl.N, K)
    assert (K, W) == (96, 6)
    table = pvq.build_count_table(wl.N, K)
    items = workload_items(wl, K, W)
    pvq.encode_batched(items, torch.bfloat16, wl.N, K, wl.scale_bits, table)   # codes resident in HBM
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    pvq.decode_batched(items, wl.N, K, wl.scale_bits, table, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    check_rows(wl, items, K, W, nrows=48, what=("codes", "out"))


def test_c5_activations_fused_sampled_rows():
    wl = inputs.config5()
    K = pvq.max_pulses(wl.N, wl.index_bits)
    W = pvq.code_words(wl.N, K)
    table = pvq.build_count_table(wl.N, K)
    items = workload_items(wl, K, W)
    it = items[0]
    pvq.roundtrip(it["x"], wl.N, K, wl.scale_bits, table, it["edges"], it["levels"], out=it["out"])
    torch.cuda.synchronize()
    check_rows(wl, items, K, W, nrows=512, what=("out",))


def test_c1_fp32_every_row():
    wl = inputs.config1()
    K = pvq.max_pulses(wl.N, wl.index_bits)
    W = pvq.code_words(wl.N, K)
    table = pvq.build_count_table(wl.N, K)
    items = workload_items(wl, K, W)
    pvq.encode_batched(items, torch.float32, wl.N, K, wl.scale_bits, table)
    pvq.decode_batched(items, wl.N, K, wl.scale_bits, table)
    torch.cuda.synchronize()
    check_rows(wl, items, K, W, nrows=512, what=("codes", "out"))


def test_c10_activations_group_128_fused_sampled_rows():
    wl = inputs.config10()
    K = pvq.max_pulses(wl.N, wl.index_bits)
    W = pvq.code_words(wl.N, K)
    assert (K, W) == (386, 16)
    table = pvq.build_count_table(wl.N, K)
    items = workload_items(wl, K, W)
    it = items[0]
    pvq.roundtrip(it["x"], wl.N, K, wl.scale_bits, table, it["edges"], it["levels"], out=it["out"])
    torch.cuda.synchronize()
    check_rows(wl, items, K, W, nrows=96, what=("out",))


def test_c10r_activations_group_128_rotated_on_the_fly_sampled_rows():
    wl = inputs.config10_unrotated()
    K = pvq.max_pulses(wl.N, wl.index_bits)
    W = pvq.code_words(wl.N, K)
    table = pvq.build_count_table(wl.N, K)
    items = workload_items(wl, K, W)
    it = items[0]
    signs = torch.from_numpy(wl.signs).to(DEV)
    pvq.rotate_roundtrip(it["x"], wl.rot_block, signs, wl.N, K, wl.scale_bits, table, it["edges"], it["levels"],
                         out=it["out"])
    torch.cuda.synchronize()
    m = wl.matrices[0]
    rows = sample_rows(m.rows, 64, seed=77)
    xr = po.rotate(np.ascontiguousarray(m.data[rows]), wl.rot_block, wl.signs)
    enc = po.encode(xr, wl.N, K, wl.scale_bits, it["e_np"], W=W)
    o_out, st = po.decode(*enc, wl.N, K, wl.scale_bits, it["l_np"])
    r = torch.from_numpy(rows).to(DEV)
    assert st == 0 and np.array_equal(bf16_bits(it["out"][r].contiguous()), o_out)


def test_c9_group_16_sampled_rows():
    wl = inputs.config9()
    K = pvq.max_pulses(wl.N, wl.index_bits)
    W = pvq.code_words(wl.N, K)
    assert (K, W) == (27, 2)
    table = pvq.build_count_table(wl.N, K)
    items = workload_items(wl, K, W)
    pvq.encode_batched(items, torch.bfloat16, wl.N, K, wl.scale_bits, table)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    pvq.decode_batched(items, wl.N, K, wl.scale_bits, table, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    check_rows(wl, items, K, W, nrows=128, what=("codes", "out"))


def test_c5r_activations_rotated_on_the_fly_sampled_rows():
    wl = inputs.config5_unrotated()
    K = pvq.max_pulses(wl.N, wl.index_bits)
    W = pvq.code_words(wl.N, K)
    table = pvq.build_count_table(wl.N, K)
    items = workload_items(wl, K, W)
    it = items[0]
    signs = torch.from_numpy(wl.signs).to(DEV)
    pvq.rotate_roundtrip(it["x"], wl.rot_block, signs, wl.N, K, wl.scale_bits, table, it["edges"], it["levels"],
                         out=it["out"])
    torch.cuda.synchronize()
    m = wl.matrices[0]
    rows = sample_rows(m.rows, 256, seed=55)
    xr = po.rotate(np.ascontiguousarray(m.data[rows]), wl.rot_block, wl.signs)
    enc = po.encode(xr, wl.N, K, wl.scale_bits, it["e_np"], W=W)
    o_out, st = po.decode(*enc, wl.N, K, wl.scale_bits, it["l_np"])
    r = torch.from_numpy(rows).to(DEV)
    assert st == 0 and np.array_equal(bf16_bits(it["out"][r].contiguous()), o_out)


@pytest.mark.parametrize("config,expect", [(inputs.config6, (187, 12)), (inputs.config7, (199, 8)),
                                           (inputs.config8, (369, 24))])
def test_global_table_kernels_sampled_rows(config, expect):
    """Group sizes and code widths of Sec. 4.1 that run with the tables in global memory."""
    wl = config()
    K = pvq.max_pulses(wl.N, wl.index_bits)
    W = pvq.code_words(wl.N, K)
    assert (K, W) == expect
    table = pvq.build_count_table(wl.N, K)
    m = wl.matrices[0]
    G = m.cols // wl.N
    x = dev_bf16(m.data)
    codes, sidx, rnorm = pvq.encode(x, wl.N, K, 16, table, None)
    out = pvq.decode(codes, sidx, rnorm, wl.N, K, 16, table, None)
    torch.cuda.synchronize()
    rows = sample_rows(m.rows, 128, seed=66)
    o_codes, o_sidx, o_rnorm = po.encode(np.ascontiguousarray(m.data[rows]), wl.N, K, 16, W=W)
    o_out, st = po.decode(o_codes, o_sidx, o_rnorm, wl.N, K, 16)
    r = torch.from_numpy(rows).to(DEV)
    assert st == 0
    assert np.array_equal(codes[r].cpu().numpy().view(np.uint32), o_codes)
    assert np.array_equal(sidx[r].cpu().numpy(), o_sidx)
    assert np.array_equal(bf16_bits(out[r].contiguous()), o_out)
