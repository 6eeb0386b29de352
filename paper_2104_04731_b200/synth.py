"""Seeded synthetic tensors for tests and benchmarks.

Holds no convolution arithmetic: only a counter-based byte generator and the table of benchmark
shapes.  Both the CPU oracle's tests and the GPU path's tests draw their inputs from here, so
the two sides see identical bytes without sharing any other code.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


def mix64(z: np.ndarray) -> np.ndarray:
    """SplitMix64 output function (Steele, Lea, Flood 2014) applied element-wise to uint64."""
    z = z.astype(np.uint64, copy=True)
    with np.errstate(over="ignore"):
        z = (z + np.uint64(0x9E3779B97F4A7C15)) & _M64
        z = ((z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
        z = ((z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
        z = z ^ (z >> np.uint64(31))
    return z


def int8_uniform(shape, seed: int) -> np.ndarray:
    """int8 tensor, i.i.d. uniform over all 256 codes; element i (C order) = low byte of mix64(seed * 2^32 + i)."""
    n = int(np.prod(shape)) if len(shape) else 1
    with np.errstate(over="ignore"):
        ctr = np.arange(n, dtype=np.uint64) + (np.uint64(seed) << np.uint64(32))
    return (mix64(ctr) & np.uint64(0xFF)).astype(np.uint8).view(np.int8).reshape(shape)


@dataclass(frozen=True)
class ConvShape:
    name: str
    N: int
    C: int
    H: int
    W: int
    K: int
    R: int
    S: int
    stride: int
    pad: int
    dilation: int
    shift: int
    out_mode: int  # bit0: int32 accumulators, bit1: requantised int8

    @property
    def P(self):
        return (self.H + 2 * self.pad - self.dilation * (self.R - 1) - 1) // self.stride + 1

    @property
    def Q(self):
        return (self.W + 2 * self.pad - self.dilation * (self.S - 1) - 1) // self.stride + 1

    @property
    def macs(self):
        return self.N * self.K * self.P * self.Q * self.C * self.R * self.S

    @property
    def algorithmic_bytes(self):
        """int8 input once + int8 weights once + the requested outputs."""
        out_elems = self.N * self.K * self.P * self.Q
        per = (4 if self.out_mode & 1 else 0) + (1 if self.out_mode & 2 else 0)
        return self.N * self.C * self.H * self.W + self.K * self.C * self.R * self.S + out_elems * per

    def tensors(self, instance: int = 0):
        """(x NCHW int8, w KCRS int8) for this shape; `instance` selects an independent draw."""
        idx = CONFIGS.index(self) + 1 if self in CONFIGS else 99
        x = int8_uniform((self.N, self.C, self.H, self.W), 1000 + idx + 100 * instance)
        w = int8_uniform((self.K, self.C, self.R, self.S), 2000 + idx + 100 * instance)
        return x, w


# The five benchmark shapes: stand-ins for the paper's DeepBench inference layers (dense 3x3,
# low-channel 7x7 stride 2, single-channel wide speech kernel, large-batch compute-bound 3x3).
CONFIGS = [
    ConvShape("cfg1_c16_14x14_k16_3x3", 1, 16, 14, 14, 16, 3, 3, 1, 1, 1, 8, 3),
    ConvShape("cfg2_c64_56x56_k64_3x3", 1, 64, 56, 56, 64, 3, 3, 1, 1, 1, 0, 1),
    ConvShape("cfg3_c3_224x224_k64_7x7s2", 4, 3, 224, 224, 64, 7, 7, 2, 3, 1, 0, 1),
    ConvShape("cfg4_c1_96x480_k32_9x21s2", 2, 1, 96, 480, 32, 9, 21, 2, 0, 1, 0, 1),
    ConvShape("cfg5_n32_c256_14x14_k512_3x3s2", 32, 256, 14, 14, 512, 3, 3, 2, 1, 1, 10, 2),
]

# Extra shapes for the candidate report: the shape classes of the paper's dilated rows (Table 3:
# dilation 2 and 4) and of its batch-1 rows on the 8x8x8 intrinsic (Table 5: data (1, C, H, W),
# weights (K, C, R, S), pad, stride), int32 output.
REPORT_EXTRA = [
    ConvShape("dil2_c16_64x64_k32_3x3", 1, 16, 64, 64, 32, 3, 3, 1, 2, 2, 0, 1),
    ConvShape("dil4_c3_96x96_k16_3x3", 1, 3, 96, 96, 16, 3, 3, 1, 4, 4, 0, 1),
    ConvShape("t5_c32_16x16_k64_3x3", 1, 32, 16, 16, 64, 3, 3, 1, 1, 1, 0, 1),
    ConvShape("t5_c72_56x56_k96_1x1", 1, 72, 56, 56, 96, 1, 1, 1, 0, 1, 0, 1),
    ConvShape("t5_c8_224x224_k24_3x3s2", 1, 8, 224, 224, 24, 3, 3, 2, 1, 1, 0, 1),
]
