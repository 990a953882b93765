"""Inputs that sit on rounding boundaries of the 4-bit formats, for both the oracle's pins and the GPU parity tests.

Every block of 32 holds one largest value 6 * s (so that the block scale is a chosen number s) and values m * s with m
on the E2M1 grid and on its midpoints (0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5): a quotient x / s that is an exact tie.
s is a power of two, an E4M3 value, or the midpoint of two neighbouring E4M3 values (a tie of the scale itself).
All values are exactly representable in bf16.
"""
import numpy as np
import torch

MULT = np.array([0.25, 0.5, 0.75, 1.0, 1.25, 1.5, 1.75, 2.0, 2.5, 3.0, 3.5, 4.0, 5.0, 6.0])


def e4m3_values():
    return torch.arange(0x7F, dtype=torch.uint8).view(torch.float8_e4m3fn).double().numpy()      # codes 0x00 .. 0x7E


def make_tie_matrix(R, K, seed):
    """[R, K] bf16 tensor; K a multiple of 32"""
    rng = np.random.default_rng(seed)
    e4 = e4m3_values()
    X = np.zeros((R, K))
    for r in range(R):
        row_exp = int(rng.integers(-6, 5))
        for b in range(K // 32):
            kind = rng.integers(0, 4)
            c = int(rng.integers(0x20, 0x50))
            if kind == 0:
                s = 2.0 ** int(rng.integers(-3, 3))
            elif kind == 1:
                s = e4[c]
            elif kind == 2:
                s = 0.5 * (e4[c] + e4[c + 1])                # the block maximum is a tie between two scale codes
            else:
                s = e4[c] * 2.0 ** -int(rng.integers(4, 12))  # a block far below the others
            vals = rng.choice(MULT, size=32) * rng.choice([-1.0, 1.0], size=32)
            vals[int(rng.integers(0, 32))] = 6.0 * rng.choice([-1.0, 1.0])
            X[r, 32 * b:32 * b + 32] = vals * s * 2.0 ** row_exp
    t = torch.from_numpy(X).to(torch.bfloat16)
    assert np.array_equal(t.double().numpy(), X), "tie values must be exact in bf16"
    return t
