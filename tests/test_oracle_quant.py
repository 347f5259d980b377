"""Pins for oracle.quant (Eq. 1-3): hand-worked values, round-trip bound, grid points, ties, saturation."""
import os

import numpy as np
import pytest

from oracle import quant
from oracle.quant import QParams

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "quantizer_eq1.txt")


def _golden_rows():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                a, b = line.split()
                rows.append((float(a), int(b)))
    return rows


def test_hand_worked_example_eq1_eq3():
    # b = 4, l = -1.5, u = 6 -> s = 0.5, z = 3 (worked in the fixture's header)
    X = np.array([-1.5, 6.0, 0.1], dtype=np.float32)
    qp = quant.qparams_minmax(X, bits=4)
    assert qp.scale == 0.5 and qp.zero_point == 3 and (qp.qmin, qp.qmax) == (0, 15)
    xs = np.array([r[0] for r in _golden_rows()])
    want = np.array([r[1] for r in _golden_rows()])
    np.testing.assert_array_equal(quant.quantize(xs, qp), want)


def test_eq2_eq3_8bit_range_ends():
    X = np.array([-1.0, 3.0, 0.5, 2.0], dtype=np.float32)
    qp = quant.qparams_minmax(X)
    assert qp.scale == pytest.approx(4.0 / 255.0, rel=1e-7)
    assert qp.zero_point == 64                    # round(63.75)
    q = quant.quantize(X, qp)
    assert q[0] == 0 and q[1] == 255              # l -> 0, u -> 2^b - 1


@pytest.mark.parametrize("mode", ["sym", "minmax"])
def test_round_trip_bound_inside_clip_range(mode):
    rng = np.random.default_rng(7)
    X = (rng.standard_normal(20000) * 3).astype(np.float32)
    qp = quant.qparams_symmetric(float(np.abs(X).max())) if mode == "sym" else quant.qparams_minmax(X)
    lo, hi = qp.scale * (qp.qmin - qp.zero_point), qp.scale * (qp.qmax - qp.zero_point)
    inside = (X >= lo) & (X <= hi)
    assert inside.mean() > 0.99
    err = np.abs(X.astype(np.float64) - quant.dequantize(quant.quantize(X, qp), qp))
    # s/2 plus float32 slack of the single product x * (1/s)
    assert err[inside].max() <= qp.scale / 2 * (1 + 1e-5)
    # and the bound is attained to within 2 % somewhere (a truncating quantizer would give ~s)
    assert err[inside].max() >= 0.49 * qp.scale


def test_grid_points_map_to_their_index():
    for qp in (QParams(0.037, 0, -127, 127), QParams(0.11, 17, 0, 255)):
        k = np.arange(qp.qmin - qp.zero_point, qp.qmax - qp.zero_point + 1)
        x = (np.float32(qp.scale) * k.astype(np.float32)).astype(np.float32)
        np.testing.assert_array_equal(quant.quantize(x, qp), k + qp.zero_point)


def test_ties_go_to_even():
    qp = QParams(0.25, 5, 0, 255)        # power-of-two scale: x/s exact
    x = np.array([0.5, 1.5, 2.5, 3.5, -0.5, -1.5, -2.5]) * 0.25
    np.testing.assert_array_equal(quant.quantize(x, qp), np.array([0, 2, 2, 4, 0, -2, -2]) + 5)


def test_saturation_both_ends():
    qp = QParams(0.1, 0, -127, 127)
    with np.errstate(over="ignore"):
        q = quant.quantize(np.array([-1e9, -12.75, 12.75, 1e9, np.float32(3e38)]), qp)
    np.testing.assert_array_equal(q, [-127, -127, 127, 127, 127])
    qp = QParams(0.1, 10, 0, 255)
    np.testing.assert_array_equal(quant.quantize(np.array([-5.0, 50.0]), qp), [0, 255])


def test_rounding_decision_is_taken_in_float32():
    # find float32 (x, s) whose float32 product x*(1/s) is an exact tie k+0.5 while the float64
    # product of the same operands falls on the side that rounds AWAY from the even neighbour
    rng = np.random.default_rng(99)
    cases = []
    for _ in range(20000):
        s = np.float32(rng.uniform(0.01, 0.2))
        inv = np.float32(1.0) / s
        k = int(rng.integers(-100, 100))
        x = np.float32((k + 0.5) * float(s))
        p32 = np.float32(x * inv)
        p64 = np.float64(x) * np.float64(inv)
        if p32 == np.float32(k + 0.5) and p64 != k + 0.5:
            even = k if k % 2 == 0 else k + 1
            if int(np.rint(p64)) != even:
                cases.append((x, s, even))
        if len(cases) >= 5:
            break
    assert len(cases) >= 5
    for x, s, even in cases:
        assert quant.quantize(np.array([x]), QParams(float(s), 0, -127, 127))[0] == even


def test_degenerate_range_takes_unit_scale():
    assert quant.qparams_symmetric(0.0).scale == 1.0
    assert quant.qparams_minmax(np.full(5, 2.0, dtype=np.float32)).scale == 1.0


def test_per_token_quantizer_and_linear():
    """Per-row scales: each row is the tensor-wise quantizer applied to that row alone, and the per-token linear
    is the float product it approximates to within the quantization steps."""
    from oracle import linear
    rng = np.random.default_rng(21)
    X = (rng.standard_normal((6, 48)) * np.array([0.1, 1, 10, 100, 1e-3, 0])[:, None]).astype(np.float32)
    q, s = quant.quantize_per_token(X)
    for m in range(6):
        qp = quant.qparams_symmetric(float(np.abs(X[m]).max()))
        np.testing.assert_array_equal(q[m], quant.quantize(X[m], qp))
        assert s[m] == np.float32(qp.scale)
        if m < 5:
            assert np.abs(q[m]).max() == 127 and np.abs(X[m] - s[m] * q[m]).max() <= s[m] / 2 * (1 + 1e-5)
    assert s[5] == 1.0 and not q[5].any()
    # scaling a row by a power of two changes its scale only
    X2 = X.copy()
    X2[2] *= 4
    q2, s2 = quant.quantize_per_token(X2)
    np.testing.assert_array_equal(q2, q)
    assert s2[2] == 4 * s[2]
    # linear: exact on values that sit on both grids
    W = rng.integers(-127, 128, size=(5, 48)).astype(np.int32)
    ws = np.full(5, 0.5, dtype=np.float32)
    Xg = (q[:5] * s[:5, None]).astype(np.float32)         # activations exactly on their grids
    qg, sg = quant.quantize_per_token(Xg)
    y = linear.w8a8_linear_per_token(qg, sg, W, ws, None)
    want = (Xg.astype(np.float64)) @ (W.astype(np.float64) * 0.5).T
    np.testing.assert_allclose(y, want, rtol=1e-6, atol=1e-9)
    # and equals the tensor-wise linear when all rows share a scale
    qp = quant.QParams(0.25, 0, -127, 127)
    qa = rng.integers(-127, 128, size=(4, 48)).astype(np.int32)
    np.testing.assert_array_equal(linear.w8a8_linear_per_token(qa, np.full(4, 0.25, dtype=np.float32), W, ws, None),
                                  linear.w8a8_linear(qa, qp, W, ws, W.sum(axis=1), None))


@pytest.mark.parametrize("bits", [4, 6, 2])
def test_weight_per_channel_low_bit(bits):
    """b-bit weights (bits = 4: the W4A8 setting of Table 2): the grid has 2^bits - 1 levels around zero."""
    rng = np.random.default_rng(5)
    W = (rng.standard_normal((7, 64)) * 0.02).astype(np.float32)
    top = (1 << (bits - 1)) - 1
    q, s, cs = quant.quantize_weight_per_channel(W, bits)
    assert q.min() == -top or q.max() == top
    assert np.abs(q).max() == top and set(np.unique(q)) <= set(range(-top, top + 1))
    for n in range(7):
        assert s[n] == np.float32(np.abs(W[n]).max()) / np.float32(top)
        assert np.abs(W[n] - s[n] * q[n]).max() <= s[n] / 2 * (1 + 1e-5)      # inside the range: half a step
        assert cs[n] == int(q[n].sum())
    # a value already on the grid is reproduced exactly; brute force against the definition of Eq. 1
    Wg = (np.arange(-top, top + 1, dtype=np.float32) * np.float32(0.25)).reshape(1, -1)
    qg, sg, _ = quant.quantize_weight_per_channel(Wg, bits)
    np.testing.assert_array_equal(qg[0], np.arange(-top, top + 1))
    for n in range(2):
        for k in range(64):
            want = int(np.clip(np.rint(np.float32(W[n, k]) * (np.float32(1.0) / s[n])), -top, top))
            assert q[n, k] == want


def test_weight_per_channel():
    rng = np.random.default_rng(3)
    W = (rng.standard_normal((9, 40)) * 0.02).astype(np.float32)
    W[4] = 0
    q, s, cs = quant.quantize_weight_per_channel(W)
    assert q.shape == W.shape and s.dtype == np.float32
    for n in range(9):
        if n == 4:
            assert s[n] == 1.0 and not q[n].any()
            continue
        j = np.argmax(np.abs(W[n]))
        assert abs(q[n, j]) == 127 and np.sign(q[n, j]) == np.sign(W[n, j])
        assert np.abs(q[n]).max() == 127
        assert s[n] == np.float32(np.abs(W[n]).max()) / np.float32(127)
        assert np.abs(W[n] - s[n] * q[n]).max() <= s[n] / 2 * (1 + 1e-5)
        assert cs[n] == int(q[n].sum())
    # channel-wise: scaling one row changes only that row's scale, never its codes
    W2 = W.copy()
    W2[2] *= 4
    q2, s2, _ = quant.quantize_weight_per_channel(W2)
    np.testing.assert_array_equal(q2, q)
    assert s2[2] == pytest.approx(4 * s[2]) and s2[3] == s[3]


def test_int4_pack_hand_worked_bytes_and_round_trip():
    rows = []
    with open(os.path.join(os.path.dirname(__file__), "golden", "int4_pack.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                a, b, h = line.split()
                rows.append((int(a), int(b), int(h, 16)))
    codes = np.array([[r[0], r[1]] for r in rows], dtype=np.int32)
    np.testing.assert_array_equal(quant.pack_int4(codes)[:, 0], np.array([r[2] for r in rows], dtype=np.uint8))
    # every byte value decodes to two codes in [-8, 7] and encodes back to itself (the map is a bijection)
    allb = np.arange(256, dtype=np.uint8).reshape(16, 16)
    un = quant.unpack_int4(allb)
    assert un.shape == (16, 32) and un.min() == -8 and un.max() == 7
    np.testing.assert_array_equal(quant.pack_int4(un), allb)
    # definition by bit arithmetic, element by element
    for byte in (0x00, 0x7F, 0x80, 0xE3, 0x9C):
        lo, hi = byte & 0xF, byte >> 4
        want = [lo - 16 if lo & 8 else lo, hi - 16 if hi & 8 else hi]
        assert quant.unpack_int4(np.array([[byte]], dtype=np.uint8))[0].tolist() == want
    # order inside a row: code 2j low nibble, code 2j+1 high nibble
    q = np.array([[1, 2, 3, 4, -1, -2]], dtype=np.int32)
    assert quant.pack_int4(q)[0].tolist() == [0x21, 0x43, 0xEF]
    np.testing.assert_array_equal(quant.unpack_int4(quant.pack_int4(q)), q)
    with pytest.raises(ValueError):
        quant.pack_int4(np.array([[8, 0]]))
    with pytest.raises(ValueError):
        quant.pack_int4(np.array([[1, 2, 3]]))


def test_int4_weights_survive_packing():
    rng = np.random.default_rng(5)
    W = (rng.standard_normal((12, 64)) * 0.02).astype(np.float32)
    q, s, cs = quant.quantize_weight_per_channel(W, bits=4)
    assert q.min() >= -7 and q.max() <= 7
    back = quant.unpack_int4(quant.pack_int4(q))
    np.testing.assert_array_equal(back, q)
    np.testing.assert_array_equal(back.sum(axis=1), cs)
