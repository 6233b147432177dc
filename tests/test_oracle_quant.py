"""Pins for the oracle's quantiser / dequantiser (Eq. 9-12)."""
import os

import numpy as np
import pytest

from oracle import xsv_oracle as orc
from paper_2602_21780_b200 import synth


def _rows(path):
    for line in open(path):
        line = line.strip()
        if line and not line.startswith("#"):
            yield [f.strip() for f in line.split(";")]


def test_hand_worked_examples(golden_dir):
    n = 0
    for bits, xs, s, z, codes, deq in _rows(os.path.join(golden_dir, "quantizer_worked.txt")):
        x = np.array([float(v) for v in xs.split()], np.float32)
        c, s_o, z_o = orc.quantize_groups(x[None, :], int(bits))
        assert float(s_o[0]) == float(s)
        assert float(z_o[0]) == float(z)
        assert c[0].tolist() == [int(v) for v in codes.split()]
        d = orc.dequantize(c, s_o[:, None], z_o[:, None])
        assert d[0].tolist() == [float(v) for v in deq.split()]
        n += 1
    assert n >= 11


@pytest.mark.parametrize("bits", [2, 4, 8])
@pytest.mark.parametrize("offset", [0.0, 3.0, -40.0])
def test_error_bound_min_max_and_range(bits, offset):
    rng = np.random.default_rng(bits * 7 + int(abs(offset)))
    x = (rng.standard_normal((4000, 64)) * rng.uniform(0.01, 20, (4000, 1)) + offset).astype(np.float32)
    c, s, z = orc.quantize_groups(x, bits)
    n = (1 << bits) - 1
    assert c.min() >= 0 and c.max() <= n
    # group minimum -> code 0 exactly; group maximum -> n or n-1 (fp32 rounding of s)
    amin, amax = x.argmin(axis=1), x.argmax(axis=1)
    r = np.arange(x.shape[0])
    assert np.all(c[r, amin] == 0)
    assert np.all(c[r, amax] >= n - 1)
    # |x - DQ(Q(x))| <= s/2 (float64 evaluation on the stored float32 s), plus the
    # float32 roundings of x - offset, of the quotient and of code * s + offset, each
    # at most 2^-24 |x|, which matters only for groups far from zero.
    d = orc.dequantize(c, s[:, None], z[:, None]).astype(np.float64)
    x64 = x.astype(np.float64)
    err = np.abs(d - x64)
    assert np.all(err <= 0.5 * s[:, None].astype(np.float64) * (1 + 2.0 ** -12) + 2.0 ** -22 * np.abs(x64))
    # monotone: larger x never gets a smaller code
    order = np.argsort(x, axis=1)
    cs = np.take_along_axis(c.astype(np.int64), order, axis=1)
    assert np.all(np.diff(cs, axis=1) >= 0)


def test_scale_and_offset_formulas_fp32():
    # s and the offset are the formulas evaluated in float32 (independent re-evaluation
    # with Python floats rounded to float32 at each operation), and so are the codes.
    rng = np.random.default_rng(3)
    for bits in (2, 4, 8):
        n = (1 << bits) - 1
        for _ in range(200):
            x = rng.standard_normal(64).astype(np.float32) * np.float32(rng.uniform(0.1, 5))
            c, s, z = orc.quantize_groups(x[None], bits)
            mn, mx = np.float32(x.min()), np.float32(x.max())
            s_ref = np.float32(np.float32(mx - mn) / np.float32(n))
            assert float(s[0]) == float(s_ref) and float(z[0]) == float(mn)
            for i in (0, 17, 63):
                q = np.rint(np.float32(np.float32(x[i] - mn) / s_ref))
                assert int(c[0, i]) == int(min(max(q, 0), n))


def test_extremes_are_reproduced_and_requantisation_is_idempotent():
    # the property that keeps repeated quantisation of the cache stable: a group's minimum dequantises to itself
    # exactly and its maximum to within the float32 rounding of n * s; quantising the dequantised group again
    # changes neither the codes nor (beyond that rounding) the parameters
    rng = np.random.default_rng(11)
    for bits in (2, 4, 8):
        n = (1 << bits) - 1
        x = (rng.standard_normal((500, 64)) * rng.uniform(0.01, 30, (500, 1)) + rng.uniform(-50, 50, (500, 1))).astype(np.float32)
        c, s, z = orc.quantize_groups(x, bits)
        d = orc.dequantize(c, s[:, None], z[:, None])
        r = np.arange(500)
        assert np.array_equal(d[r, x.argmin(axis=1)], x.min(axis=1))
        assert np.all(np.abs(d.max(axis=1).astype(np.float64) - x.max(axis=1)) <= 2.0 ** -22 * np.abs(x).max(axis=1))
        c2, s2, z2 = orc.quantize_groups(d, bits)
        assert np.array_equal(c2, c) and np.array_equal(z2, z)
        assert np.all(np.abs(s2.astype(np.float64) - s) <= 2.0 ** -21 * s)


def test_constant_and_tiny_groups_are_exact():
    for v in (0.0, 1.5, -2.25, 6e-39, -65504.0):
        x = np.full((1, 64), v, np.float32)
        for bits in (2, 4, 8):
            c, s, z = orc.quantize_groups(x, bits)
            assert np.all(c == 0)
            d = orc.dequantize(c, s[:, None], z[:, None])
            assert np.all(d == np.float32(v))


def test_two_element_groups_exhaustive_fp16_b2():
    # every finite fp16 value paired with a fixed partner: the smaller maps to
    # code 0, the larger to n (or n-1), and both dequantise within s/2.
    allv = np.arange(65536, dtype=np.uint16).view(np.float16).astype(np.float32)
    allv = allv[np.isfinite(allv)]
    for partner in (0.0, 1.0, -3.5, 1000.0):
        x = np.stack([allv, np.full_like(allv, partner)], axis=1)
        c, s, z = orc.quantize_groups(x, 2)
        lo = x.argmin(axis=1)
        r = np.arange(x.shape[0])
        distinct = x[:, 0] != x[:, 1]
        assert np.all(c[r, lo] == 0)
        assert np.all(c[r, 1 - lo][distinct] >= 2)
        d = orc.dequantize(c, s[:, None], z[:, None]).astype(np.float64)
        assert np.all(np.abs(d - x) <= 0.5 * s[:, None].astype(np.float64) * (1 + 2.0 ** -12))


def test_granularity_direction_matches_table1():
    # Table 1's direction on outlier-channel keys: per-channel groups (along tokens)
    # give several times lower MSE than per-token groups (along channels); for
    # values without outliers the two are close.
    from paper_2602_21780_b200 import synth
    st = synth.Stream(H=4, d=64, F=512, dtype="bf16")
    _, K, V = st.frame(0)

    def mse(x, axis_tokens, bits):
        H, T, d = x.shape
        if axis_tokens:       # per-channel: groups of 64 tokens
            g = x.reshape(H, T // 64, 64, d).transpose(0, 1, 3, 2)
        else:                 # per-token: groups of 64 channels
            g = x.reshape(H, T, 1, d)
        c, s, z = orc.quantize_groups(g, bits)
        dq = orc.dequantize(c, s[..., None], z[..., None])
        return float(np.mean((dq.astype(np.float64) - g) ** 2))

    for bits, factor in ((4, 3.0), (2, 1.0)):
        # (at 2 bits the outlier channels' own error dominates both schemes on this
        # synthetic data, so only the direction is asserted there)
        assert mse(K, False, bits) > factor * mse(K, True, bits)
        rv = mse(V, False, bits) / mse(V, True, bits)
        assert 0.5 < rv < 2.0


# --------------------------------------------------------------------------
# quantization_mse (Eq. 11 granularities, the quantity of Table 1)
# --------------------------------------------------------------------------
def test_mse_is_zero_for_values_on_the_grid():
    rng = np.random.default_rng(3)
    for bits in (2, 4, 8):
        n = (1 << bits) - 1
        # per token: every token's 64 channels lie on a grid with step 2^-3 that contains both ends
        c = rng.integers(0, n + 1, size=(2, 70, 64))
        c[..., 0], c[..., 1] = 0, n
        z = rng.integers(-5, 6, size=(2, 70, 1))
        x = ((c - z) * 0.125).astype(np.float32)
        assert orc.quantization_mse(x, bits, "token") == 0.0
        # per channel: the same construction along the token axis, groups of 64 tokens (the second group is partial)
        c = rng.integers(0, n + 1, size=(2, 70, 64))
        c[:, 0, :], c[:, 1, :], c[:, 64, :], c[:, 65, :] = 0, n, 0, n
        x = ((c - 3) * 0.25).astype(np.float32)
        assert orc.quantization_mse(x, bits, "channel") == 0.0


def test_mse_hand_worked_example():
    # 2 bits (n = 3).  Token 0: [0, 1, 3] -> s = 1, offset 0, exact.  Token 1: [0, 0.4, 3] -> s = 1, 0.4 rounds to 0.
    x = np.array([[[0.0, 1.0, 3.0], [0.0, 0.4, 3.0]]], dtype=np.float32)
    want = float(np.float64(np.float32(0.4)) ** 2) / 6.0
    assert orc.quantization_mse(x, 2, "token") == pytest.approx(want, rel=1e-12)
    # per channel over the (partial) group of the two tokens: channel 1 is [1, 0.4] -> s = 0.2, offset 0.4,
    # codes 3 and 0, dequantised 3 * 0.2 + 0.4 = 1.0 (up to float32 rounding) and 0.4; channels 0 and 2 are constant
    got = orc.quantization_mse(x, 2, "channel")
    assert got < 1e-14


def test_mse_per_channel_is_per_token_of_the_transpose():
    rng = np.random.default_rng(4)
    x = rng.normal(size=(3, 64, 64)).astype(np.float32)
    for bits in (2, 4):
        a, b = orc.quantization_mse(x, bits, "channel"), orc.quantization_mse(x.transpose(0, 2, 1).copy(), bits, "token")
        assert a == pytest.approx(b, rel=1e-12)      # same groups, same errors; only the order of the float64 sum differs


def test_mse_of_uniform_data_is_step_squared_over_twelve():
    rng = np.random.default_rng(5)
    x = rng.uniform(-1.0, 1.0, size=(4, 256, 64)).astype(np.float32)
    for bits in (4, 8):
        n = (1 << bits) - 1
        step = 2.0 / n                       # groups of 64 uniform samples span almost the whole interval
        got = orc.quantization_mse(x, bits, "token")
        assert 0.8 * step * step / 12 < got < 1.05 * step * step / 12


def test_mse_direction_of_table_1_on_outlier_channels():
    # keys with a few channels of ten-fold magnitude (Fig. 4): per-channel groups keep the outliers apart, per-token
    # groups stretch every token's range over them; values without outliers show no such gap
    st = synth.Stream(H=4, d=64, F=256, dtype="bf16", layer=2)
    _, K, V = st.frame(0)
    for bits, gap in ((2, 1.0), (4, 0.3), (8, 0.3)):
        k_ch, k_tok = orc.quantization_mse(K, bits, "channel"), orc.quantization_mse(K, bits, "token")
        v_ch, v_tok = orc.quantization_mse(V, bits, "channel"), orc.quantization_mse(V, bits, "token")
        assert k_ch < gap * k_tok      # at 2 bits the outlier channels' own error dominates both schemes
        assert 0.9 < v_ch / v_tok < 1.1
