"""Seeded synthetic inputs for the PVQ codec: the five benchmark workloads.

This module only makes numbers to feed the codec (random draws, Hadamard
rotations, rounding to the storage type).  It contains none of the codec's
arithmetic and imports neither the CUDA binding nor the CPU oracle, so both
can be fed the same bytes.

The matrices stand in for rotated LLM weights and activations: Gaussian or
heavy-tailed entries, multiplied along the input dimension by a random-sign
Walsh-Hadamard matrix (Sec. 2.3 "Hadamard coherence processing", Sec. 3.3
Step 1), stored as bf16 (fp32 for the smallest case).
"""
from dataclasses import dataclass
from typing import List

import numpy as np


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest, ties to even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def hadamard_rows(x: np.ndarray, block: int, signs: np.ndarray) -> np.ndarray:
    """x <- (x * signs) H_block / sqrt(block), independently on every contiguous
    `block` columns of every row.  H is the Sylvester-Walsh-Hadamard matrix;
    `signs` (+-1, length block) is shared by all blocks and rows."""
    rows, cols = x.shape
    assert cols % block == 0 and block & (block - 1) == 0
    y = (x.reshape(rows, cols // block, block) * signs.astype(np.float32)).astype(np.float32)
    h = 1
    while h < block:
        y = y.reshape(rows, cols // block, block // (2 * h), 2, h)
        a = y[:, :, :, 0, :] + y[:, :, :, 1, :]
        b = y[:, :, :, 0, :] - y[:, :, :, 1, :]
        y = np.stack([a, b], axis=3)
        h *= 2
    y = y.reshape(rows, cols) * np.float32(1.0 / np.sqrt(block))
    return y.astype(np.float32)


def _rng(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(seed))


def _signs(rng: np.random.Generator, n: int) -> np.ndarray:
    return (rng.integers(0, 2, size=n).astype(np.float32) * 2.0 - 1.0).astype(np.float32)


@dataclass
class Matrix:
    """One input matrix: `data` is float32, or uint16 holding bf16 bit patterns."""
    name: str
    data: np.ndarray
    dtype: str  # "f32" or "bf16"

    @property
    def rows(self):
        return self.data.shape[0]

    @property
    def cols(self):
        return self.data.shape[1]


@dataclass
class Workload:
    """A benchmark configuration: matrices plus the codec parameters."""
    name: str
    N: int           # group size
    index_bits: int  # bits of one group's direction code
    scale_bits: int  # bits of one group's amplitude index
    mode: str        # "encode+decode", "decode", "roundtrip", "rotate_roundtrip"
    matrices: List[Matrix]
    rot_block: int = 0          # "rotate_roundtrip": size of the Hadamard blocks applied on the fly
    signs: np.ndarray = None    # ... and their +-1 signs (float32, rot_block of them)

    @property
    def weights(self) -> int:
        return sum(m.rows * m.cols for m in self.matrices)


def gaussian_f32(rows, cols, sigma, seed) -> np.ndarray:
    return (_rng(seed).standard_normal((rows, cols), dtype=np.float32) * np.float32(sigma)).astype(np.float32)


def config1(rows=512, cols=512) -> Workload:
    """fp32, iid N(0, 0.02^2), seed 0, no rotation; N=32, 64-bit codes, 8-bit amplitudes."""
    x = gaussian_f32(rows, cols, 0.02, 0)
    return Workload("c1_fp32_512", 32, 64, 8, "encode+decode", [Matrix("w", x, "f32")])


def config2(rows=4096, cols=4096) -> Workload:
    """bf16 q_proj shape, N(0, 0.02^2) then a cols-point random-sign Hadamard on the
    input dimension; N=32, 96-bit codes, 4-bit amplitudes."""
    rng = _rng(2)
    x = (rng.standard_normal((rows, cols), dtype=np.float32) * np.float32(0.02)).astype(np.float32)
    x = hadamard_rows(x, cols, _signs(rng, cols))
    return Workload("c2_bf16_q_proj", 32, 96, 4, "encode+decode",
                    [Matrix("q_proj", f32_to_bf16_bits(x), "bf16")])


LLAMA3_8B_LAYER = [("q_proj", 4096, 4096), ("k_proj", 1024, 4096), ("v_proj", 1024, 4096),
                   ("o_proj", 4096, 4096), ("gate_proj", 14336, 4096), ("up_proj", 14336, 4096),
                   ("down_proj", 4096, 14336)]


def config3(scale_div: int = 1) -> Workload:
    """One Llama-3-8B decoder layer in bf16: Student-t(5) * 0.02 entries, 512-point
    random-sign Hadamard blocks along the input dimension; N=32, 96-bit codes, 8-bit
    amplitudes.  scale_div > 1 divides every row count (test-sized variant)."""
    mats = []
    for i, (name, rows, cols) in enumerate(LLAMA3_8B_LAYER):
        rng = _rng(300 + i)
        r = max(rows // scale_div, 1)
        x = (rng.standard_t(5.0, size=(r, cols)).astype(np.float32) * np.float32(0.02)).astype(np.float32)
        x = hadamard_rows(x, 512, _signs(rng, 512))
        mats.append(Matrix(name, f32_to_bf16_bits(x), "bf16"))
    return Workload("c3_llama3_8b_layer", 32, 96, 8, "encode+decode", mats)


def config4(rows=8192, cols=28672) -> Workload:
    """Llama-3-70B down_proj shape in bf16, N(0, 0.015^2), 512-point Hadamard blocks;
    N=64, 192-bit codes, 6-bit amplitudes; decode throughput on pre-encoded codes."""
    rng = _rng(4)
    x = (rng.standard_normal((rows, cols), dtype=np.float32) * np.float32(0.015)).astype(np.float32)
    x = hadamard_rows(x, 512, _signs(rng, 512))
    return Workload("c4_bf16_down_proj_70b", 64, 192, 6, "decode",
                    [Matrix("down_proj", f32_to_bf16_bits(x), "bf16")])


def config5(tokens=16384, hidden=4096) -> Workload:
    """Activations in bf16: rows iid N(0,1), 0.1 % of the channels scaled by 20, then a
    hidden-point random-sign Hadamard per token; N=32, 64-bit codes, 8-bit amplitudes;
    fused encode -> decode."""
    rng = _rng(5)
    x = rng.standard_normal((tokens, hidden), dtype=np.float32)
    n_out = max(int(round(hidden * 0.001)), 1)
    ch = rng.choice(hidden, size=n_out, replace=False)
    x[:, ch] *= np.float32(20.0)
    x = hadamard_rows(x, hidden, _signs(rng, hidden))
    return Workload("c5_bf16_activations", 32, 64, 8, "roundtrip",
                    [Matrix("act", f32_to_bf16_bits(x), "bf16")])


def config5_unrotated(tokens=16384, hidden=4096) -> Workload:
    """config5's activations before their rotation (same seed, same draws): rows iid N(0,1)
    with 0.1 % of the channels scaled by 20, in bf16, plus the signs of the hidden-point
    random-sign Hadamard that the codec applies on the fly; N=32, 64-bit codes, 8-bit
    amplitudes; rotate -> encode -> decode in one kernel."""
    rng = _rng(5)
    x = rng.standard_normal((tokens, hidden), dtype=np.float32)
    n_out = max(int(round(hidden * 0.001)), 1)
    ch = rng.choice(hidden, size=n_out, replace=False)
    x[:, ch] *= np.float32(20.0)
    signs = _signs(rng, hidden)
    return Workload("c5r_bf16_activations_rotated_on_the_fly", 32, 64, 8, "rotate_roundtrip",
                    [Matrix("act", f32_to_bf16_bits(x), "bf16")], rot_block=hidden, signs=signs)


def config6(rows=4096, cols=4096) -> Workload:
    """The paper's weight-only setting of Sec. 4.1 on config2's matrix: group size 128, 3 bits per
    weight of direction (384-bit codes, K = 187) and 16-bit amplitudes, 3.125 bits per weight."""
    wl = config2(rows, cols)
    return Workload("c6_bf16_q_proj_group128", 128, 384, 16, "encode+decode", wl.matrices)


def config7(rows=4096, cols=4096) -> Workload:
    """Sec. 4.1's grid at a higher rate on config2's matrix: group size 64, 4 bits per weight of
    direction (256-bit codes, K = 199) and 16-bit amplitudes."""
    wl = config2(rows, cols)
    return Workload("c7_bf16_q_proj_group64_4bit", 64, 256, 16, "encode+decode", wl.matrices)


def config8(rows=4096, cols=4096) -> Workload:
    """Sec. 4.1's largest group size on config2's matrix: group size 256, 3 bits per weight of
    direction (768-bit codes, K = 369) and 16-bit amplitudes."""
    wl = config2(rows, cols)
    return Workload("c8_bf16_q_proj_group256", 256, 768, 16, "encode+decode", wl.matrices)


def config9(rows=4096, cols=4096) -> Workload:
    """The setting of the paper's headline result (abstract; weight-only tables of Sec. 4: 3 bits of
    direction and 4-bit amplitudes at group size 16, 3.25 bits per weight) on config2's matrix:
    48-bit codes, K = 27."""
    wl = config2(rows, cols)
    return Workload("c9_bf16_q_proj_group16", 16, 48, 4, "encode+decode", wl.matrices)


def config10(tokens=16384, hidden=4096) -> Workload:
    """config5's activations at the setting of the paper's weight-and-activation results (Sec. 4.3:
    4.125 bits per activation at group size 128): 4 bits of direction per value (512-bit codes,
    K = 386) and 16-bit amplitudes; fused encode -> decode."""
    wl = config5(tokens, hidden)
    return Workload("c10_bf16_activations_group128", 128, 512, 16, "roundtrip", wl.matrices)


def config10_unrotated(tokens=16384, hidden=4096) -> Workload:
    """config10 from the activations before their rotation (config5_unrotated's input and signs):
    rotate -> encode -> decode in one kernel at group size 128."""
    wl = config5_unrotated(tokens, hidden)
    return Workload("c10r_bf16_activations_group128_rotated_on_the_fly", 128, 512, 16, "rotate_roundtrip",
                    wl.matrices, rot_block=wl.rot_block, signs=wl.signs)
