"""Pins of the oracle's round-to-nearest quantisation (App. "Integrate with Quantization")."""
import numpy as np

from oracle import xkv_oracle as O


def _bf16_matrix(n, m, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    return O.bf16_round((rng.standard_normal((n, m)) * scale).astype(np.float32))


def test_values_on_the_grid_are_reproduced_exactly():
    # a group whose values are zero + code * scale with bf16 zero and scale: quantisation must return those codes
    rng = np.random.default_rng(1)
    for bits in (3, 4):
        scale, zero = np.float32(0.0625), np.float32(-1.5)                # both exact in bf16; products exact
        codes = rng.integers(0, 1 << bits, size=(5, 64)).astype(np.uint8)
        codes[:, 0], codes[:, 1] = 0, (1 << bits) - 1                       # the group spans the whole range
        codes[:, 32], codes[:, 33] = 0, (1 << bits) - 1
        X = codes.astype(np.float32) * scale + zero
        c, s, z = O.rtn_quantize(X, bits)
        assert np.array_equal(c, codes) and np.all(s == scale) and np.all(z == zero)
        assert np.array_equal(O.rtn_dequantize(c, s, z), X)


def test_round_trip_error_is_half_a_step_plus_the_rounding_of_the_parameters():
    X = _bf16_matrix(64, 256, 2)
    for bits in (3, 4, 8):
        c, s, z = O.rtn_quantize(X, bits)
        assert c.max() <= (1 << bits) - 1
        Xh = O.rtn_dequantize(c, s, z)
        step = np.repeat(s, O.RTN_GROUP, axis=1)
        # half a step from rounding the code; the bf16 rounding of scale (2^-9 relative, times up to 2^b - 1 steps),
        # of the offset and of the result (2^-9 of the magnitude each) on top
        bound = 0.5 * step + ((1 << bits) - 1) * step * 2.0 ** -8 + 2.0 ** -7 * np.abs(X).max()
        assert np.all(np.abs(Xh - X) <= bound)
        # more bits, smaller error
    e4 = np.abs(O.rtn_dequantize(*O.rtn_quantize(X, 4)) - X).mean()
    e3 = np.abs(O.rtn_dequantize(*O.rtn_quantize(X, 3)) - X).mean()
    assert e4 < 0.6 * e3


def test_constant_group_and_extremes():
    X = np.full((2, 32), 0.75, dtype=np.float32)
    c, s, z = O.rtn_quantize(X, 4)
    assert np.all(c == 0) and np.all(s == 0) and np.all(z == 0.75)
    assert np.array_equal(O.rtn_dequantize(c, s, z), X)
    # the minimum of a group maps to code 0 and the maximum to the top code (up to the bf16 rounding of the offset)
    X = _bf16_matrix(16, 64, 3)
    c, s, z = O.rtn_quantize(X, 4)
    Xg, cg = X.reshape(16, 2, 32), c.reshape(16, 2, 32)
    assert np.all(np.take_along_axis(cg, Xg.argmin(axis=2)[..., None], axis=2) <= 1)
    assert np.all(np.take_along_axis(cg, Xg.argmax(axis=2)[..., None], axis=2) >= 14)


def test_codes_by_scalar_brute_force():
    # the vectorised routine against a scalar restatement with explicit fp32 steps
    X = _bf16_matrix(3, 64, 4, scale=3.0)
    c, s, z = O.rtn_quantize(X, 4)
    for i in range(3):
        for g in range(2):
            grp = X[i, 32 * g:32 * g + 32]
            lo, hi = np.float32(grp.min()), np.float32(grp.max())
            zero = O.bf16_round(np.array([lo]))[0]
            scale = O.bf16_round(np.array([(hi - lo) / np.float32(15)], dtype=np.float32))[0]
            assert s[i, g] == scale and z[i, g] == zero
            for j, x in enumerate(grp):
                q = np.float32(np.float32(x - zero) / scale)
                code = int(min(15, max(0, np.rint(q))))
                assert c[i, 32 * g + j] == code


def test_stored_bits_and_printed_ratios():
    assert O.quantized_bits_per_scalar(4) == 5.0 and O.quantized_bits_per_scalar(3) == 4.0
    assert abs(O.quantized_compression_ratio(8.03, 4) - 25.70) < 0.0075      # the paper's xKV-4bit row
    assert abs(O.quantized_compression_ratio(8.03, 3) - 32.12) < 0.0075      # the paper's xKV-3bit row


def test_single_step_bf16_rounding_matches_the_two_step_routine_where_both_are_exact():
    # on float32 inputs whose low 16 bits hold no sticky information beyond bit 15 the two roundings agree;
    # on a constructed double-rounding case they differ and the single-step routine is the correct one
    x = _bf16_matrix(8, 8, 5).astype(np.float64) * (1.0 + 2.0 ** -10)          # not bf16 values any more
    assert np.array_equal(O.bf16_round_exact(x), O.bf16_round(x.astype(np.float32)))
    tricky = 1.0 + 2.0 ** -8 + 2.0 ** -40          # just above the tie between 1 and 1 + 2^-7: must round up
    assert O.bf16_round_exact(np.array([tricky]))[0] == np.float32(1.0 + 2.0 ** -7)
    assert O.bf16_round(np.array([tricky], dtype=np.float32))[0] == np.float32(1.0)   # float32 first lands on the tie
