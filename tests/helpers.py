"""Small numpy helpers shared by the tests (no method arithmetic beyond textbook formulas)."""
import numpy as np

from paper_2607_28150_b200.workloads import bf16_bits_to_f32, f32_to_bf16_bits


def rand_bf16(rng, shape, scale=1.0):
    return f32_to_bf16_bits((scale * rng.standard_normal(shape)).astype(np.float32))


def widen(bits):
    return bf16_bits_to_f32(bits).astype(np.float64)


def cu_of(lengths):
    return np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
