"""The decode entry point for callers that cannot allocate device memory.

pvq_decode_static_table keeps the count table in an array that is part of the
library instead of a buffer from the caller (an engine plug-in or a frozen
real-time loop has no cudaMalloc to call).  It must give exactly what
pvq_decode gives, call after call, including when the (N, K) it is asked for
changes and the shared array is refilled.  This file sorts last so that a run
that stops at the first failure has been through every other test first.
"""
import numpy as np
import pytest
import torch

from oracle import beta_codebook as bc
from oracle import pvq_oracle as po
from paper_2410_16926_b200 import pvq

pytestmark = pytest.mark.gpu

DEV = "cuda"


def _encoded(N, bits, rows, cols, b, seed):
    rng = np.random.default_rng(seed)
    x = torch.from_numpy((rng.standard_normal((rows, cols)) * 0.02).astype(np.float32)).to(DEV)
    G = cols // N
    K = pvq.max_pulses(N, bits)
    table = pvq.build_count_table(N, K)
    edges = torch.from_numpy(bc.edges_f32(N, G, b)).to(DEV)
    levels = torch.from_numpy(bc.levels_amp_f32(N, G, b)).to(DEV)
    enc = pvq.encode(x, N, K, b, table, edges)
    return K, table, levels, enc


def _oracle_bits(enc, N, K, b, G):
    """Algorithm 3 + Sec. 3.4 by the CPU oracle on the same codes: bf16 bit patterns."""
    codes, sidx, rnorm = (t.cpu().numpy() for t in enc)
    out, status = po.decode(codes.view(np.uint32), sidx, rnorm, N, K, b, bc.levels_amp_f32(N, G, b))
    assert status == 0
    return torch.from_numpy(out.view(np.int16)).to(DEV)


def _same_bits(a, b):
    return torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_static_table_decode_equals_decode_on_consecutive_calls():
    # two calls in a row with the same (N, K): the second reuses the table the first built
    K, table, levels, enc = _encoded(32, 96, 37, 4096, 4, seed=11)
    ref = pvq.decode(*enc, 32, K, 4, table, levels)
    out1 = torch.empty_like(ref)
    out2 = torch.full_like(ref, 3.0)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    pvq.decode_static_table(*enc, 32, K, 4, levels, out=out1, status=st)
    pvq.decode_static_table(*enc, 32, K, 4, levels, out=out2, status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert _same_bits(out1, ref) and _same_bits(out2, ref)
    assert torch.equal(out1.view(torch.int16), _oracle_bits(enc, 32, K, 4, 4096 // 32))

    # a different (N, K) refills the shared array; going back refills it again
    K2, table2, levels2, enc2 = _encoded(32, 64, 19, 512, 8, seed=12)
    ref2 = pvq.decode(*enc2, 32, K2, 8, table2, levels2)
    out3 = pvq.decode_static_table(*enc2, 32, K2, 8, levels2, out=torch.empty_like(ref2))
    out4 = pvq.decode_static_table(*enc, 32, K, 4, levels, out=torch.empty_like(ref))
    torch.cuda.synchronize()
    assert _same_bits(out3, ref2) and _same_bits(out4, ref)
    assert torch.equal(out3.view(torch.int16), _oracle_bits(enc2, 32, K2, 8, 512 // 32))


def test_static_table_same_parameters_on_two_streams():
    # The first call fills the shared array on its own stream; a second call with the same
    # (N, K) on another stream, with no dependency of the caller's making, must still read the
    # finished table: the library orders it behind the fill.
    K, table, levels, enc = _encoded(32, 96, 23, 2048, 4, seed=21)
    K0, _, levels0, enc0 = _encoded(16, 40, 5, 256, 4, seed=22)
    ref = pvq.decode(*enc, 32, K, 4, table, levels)
    pvq.decode_static_table(*enc0, 16, K0, 4, levels0)      # leave another (N, K) in the array
    torch.cuda.synchronize()
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    out1, out2 = torch.empty_like(ref), torch.empty_like(ref)
    with torch.cuda.stream(s1):
        pvq.decode_static_table(*enc, 32, K, 4, levels, out=out1)
    with torch.cuda.stream(s2):
        pvq.decode_static_table(*enc, 32, K, 4, levels, out=out2)
    torch.cuda.synchronize()
    assert _same_bits(out1, ref) and _same_bits(out2, ref)


def test_static_table_calls_leave_device_memory_alone():
    # once set-up is over (first call made, output preallocated) repeated calls neither take
    # nor give back device memory: the driver's free-byte count and torch's allocator agree
    K, table, levels, enc = _encoded(32, 96, 8, 1024, 4, seed=31)
    out = torch.empty((8, 1024), dtype=torch.bfloat16, device=DEV)
    pvq.decode_static_table(*enc, 32, K, 4, levels, out=out)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0 = torch.cuda.memory_allocated()
    for _ in range(5):
        pvq.decode_static_table(*enc, 32, K, 4, levels, out=out)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0 and torch.cuda.memory_allocated() == alloc0


def test_static_table_rejects_what_does_not_fit():
    # N = 128 at 384-bit codes needs a table far beyond the built-in array
    K = pvq.max_pulses(128, 384)
    assert pvq.count_table_bytes(128, K) > 1024 * 1024
    dummy = torch.zeros(64, dtype=torch.int32, device=DEV)
    rc = pvq.lib().pvq_decode_static_table(dummy.data_ptr(), dummy.data_ptr(), dummy.data_ptr(), 1, 256, 128,
                                           K, 4, dummy.data_ptr(), dummy.data_ptr(), 256, None, None)
    assert rc == 4      # PVQ_ERR_TABLE_TOO_SMALL, before any GPU work
