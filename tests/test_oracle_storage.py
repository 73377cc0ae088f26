"""CPU pins of the storage oracle (oracle/storage.py): the bfloat16 rounding is checked against values fixed
by the format's definition and against an independent library conversion, not against itself."""
import numpy as np
import pytest
import torch

from oracle import storage


def test_hand_values_of_the_format():
    # 8 significant bits: in [1, 2) the spacing is 2^-7; halves go to the even neighbour
    cases = {
        1.0: 1.0,
        1.0 + 2.0 ** -7: 1.0 + 2.0 ** -7,                    # representable
        1.0 + 2.0 ** -8: 1.0,                                # tie between 1 and 1+2^-7: 1 has the even last bit
        1.0 + 3 * 2.0 ** -8: 1.0 + 2.0 ** -6,                # tie between 1+2^-7 (odd) and 1+2^-6 (even)
        1.0 + 2.0 ** -8 + 2.0 ** -30: 1.0 + 2.0 ** -7,       # just above the tie
        1.0 + 2.0 ** -8 - 2.0 ** -30: 1.0,                   # just below the tie
        2.0 - 2.0 ** -9: 2.0,                                # rounds up into the next binade
        255.0: 255.0, 256.0: 256.0, 257.0: 256.0, 259.0: 260.0, 258.0: 258.0,   # integers: spacing 2 above 256
        0.1: 0.10009765625,                                  # 0x3DCD
        -0.1: -0.10009765625,
        3.0e38: 226 * 2.0 ** 120,                            # top binade [2^127, 2^128): spacing 2^120, 3e38 / 2^120 = 225.7
        3.4e38: np.inf,                                      # beyond the largest finite value (3.3895e38)
        2.0 ** -133: 2.0 ** -133,                            # smallest subnormal
        0.4 * 2.0 ** -133: 0.0,                              # below half of it
        0.0: 0.0,
    }
    for x, want in cases.items():
        got = float(storage.round_to_bf16(np.array([x]))[0])
        assert got == want, (x, got, want)


def test_matches_the_library_conversion_of_float32_values():
    # float32 inputs are exact in float64, so both sides round once
    rng = np.random.default_rng(5)
    a = np.concatenate([rng.standard_normal(200000), rng.standard_normal(1000) * 1e-30,
                        rng.standard_normal(1000) * 1e30, rng.standard_normal(1000) * 1e-39]).astype(np.float32)
    lib = torch.from_numpy(a).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(storage.round_to_bf16(a.astype(np.float64)), lib)


def test_every_bf16_value_is_a_fixed_point_and_halfway_points_go_to_even():
    bits = np.arange(0, 0x7F80, dtype=np.int32)              # all non-negative finite bfloat16 patterns
    vals = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    assert np.array_equal(storage.round_to_bf16(vals), vals)
    assert np.array_equal(storage.round_to_bf16(-vals), -vals)
    mid = 0.5 * (vals[:-1] + vals[1:])                       # exact in float64
    want = np.where(bits[:-1] % 2 == 0, vals[:-1], vals[1:])
    assert np.array_equal(storage.round_to_bf16(mid), want)


def test_error_bound_and_monotonicity():
    rng = np.random.default_rng(6)
    a = np.sort(rng.standard_normal(100000) * np.exp(rng.uniform(-20, 20, 100000)))
    r = storage.round_to_bf16(a)
    assert np.all(np.abs(r - a) <= 0.5 * storage.bf16_spacing(a))
    assert np.all(np.abs(r - a) <= 2.0 ** -8 * np.abs(a))     # half a unit in the last place, relative to |a| >= 2^lead
    assert np.all(np.diff(r) >= 0)


def test_spacing():
    assert storage.bf16_spacing(np.array([1.0, 1.99, 2.0, 0.5, 300.0, 0.0])).tolist() == \
        [2.0 ** -7, 2.0 ** -7, 2.0 ** -6, 2.0 ** -8, 2.0, 2.0 ** -133]
