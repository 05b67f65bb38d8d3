"""Pins of the oracle's embedding codec (Supplement, "Data Compression for Historical Embedding Storage": the encoded
polyline scheme, one row = one delta-coded sequence).

What fixes it from outside the oracle:
  * the worked examples printed in the published description of the encoded polyline algorithm (a single value, and a
    three-point path whose latitude / longitude deltas are the integer sequence encoded here);
  * the quantiser against exact rational arithmetic (fractions.Fraction), round half away from zero;
  * hand-worked one-byte codes, the reconstruction error bound 0.5 * 10^-p, round trips, and rejection of malformed rows.
"""
from fractions import Fraction

import numpy as np
import pytest

from oracle import sat_ref as orc


def test_published_single_value():
    # the published example: -179.9832104 at five decimals -> the integer -17998321 -> "`~oia@".
    # fp32 cannot hold that value to five decimals, so the integer is produced here as a delta at zero decimals:
    # row (1, -17998320) -> e = 1, -17998321 (both entries are exact in fp32).
    data, off = orc.codec_encode(np.array([[1.0, -17998320.0]], dtype=np.float32), 0)
    assert bytes(data) == b"A`~oia@" and list(off) == [0, 7]


def test_published_three_point_path():
    # points (38.5, -120.2), (40.7, -120.95), (43.252, -126.453): the encoder's integer sequence is
    # lat0, lng0, dlat1, dlng1, dlat2, dlng2 = 3850000, -12020000, 220000, -75000, 255200, -550300 (x 1e-5).
    # One row whose consecutive differences are exactly these integers reproduces the published string.
    deltas = np.array([3850000, -12020000, 220000, -75000, 255200, -550300], dtype=np.int64)
    q = np.cumsum(deltas)
    x = (q.astype(np.float64) / 1e5).astype(np.float32)[None, :]
    # fp32 keeps |x * 1e5 - q| < 0.5 for these magnitudes, so the quantiser returns q
    assert np.all(np.abs(x.astype(np.float64)[0] * 1e5 - q) < 0.5)
    data, off = orc.codec_encode(x, 5)
    assert bytes(data) == b"_p~iF~ps|U_ulLnnqC_mqNvxq`@"
    back = orc.codec_decode(data, off, 6, 5)
    assert np.array_equal(back, (q.astype(np.float64) / 1e5).astype(np.float32)[None, :])


def test_hand_worked_codes():
    # q = 0 -> v = 0 -> '?';  q = 1 -> v = 2 -> 'A';  q = -1 -> v = ~(-2) = 1 -> '@';  q = 15 -> v = 30 -> ']';
    # q = 16 -> v = 32 -> groups (0 | 0x20, 1) -> '_', '@'
    for value, want in ((0.0, b"?"), (1.0, b"A"), (-1.0, b"@"), (15.0, b"]"), (16.0, b"_@")):
        data, _ = orc.codec_encode(np.array([[value]], dtype=np.float32), 0)
        assert bytes(data) == want, value
    # deltas inside a row: [3, 3, 1] -> e = 3, 0, -2 -> v = 6, 0, 3 -> 'E', '?', 'B'
    data, off = orc.codec_encode(np.array([[3.0, 3.0, 1.0]], dtype=np.float32), 0)
    assert bytes(data) == b"E?B" and list(off) == [0, 3]


def _quantise_exact(x: np.ndarray, p: int) -> np.ndarray:
    out = np.zeros(x.shape, dtype=object)
    for idx, v in np.ndenumerate(x):
        t = Fraction(float(v)) * (10 ** p)
        n = int(abs(t) + Fraction(1, 2))            # floor(|t| + 1/2): half away from zero
        out[idx] = n if t >= 0 else -n
    return out


@pytest.mark.parametrize("p", [0, 2, 5, 7])
def test_quantiser_against_exact_rationals(p):
    rng = np.random.default_rng(p)
    x = np.concatenate([rng.normal(size=(6, 9)), rng.normal(size=(6, 9)) * 37.0]).astype(np.float32)
    # ties and near-ties at the rounding boundary, zeros, negative zero
    x[0, :4] = np.array([0.5, -0.5, 1.5, -2.5], dtype=np.float32) / np.float32(10 ** p)
    x[1, :3] = [0.0, -0.0, 1e-30]
    data, off = orc.codec_encode(x, p)
    back = orc.codec_decode(data, off, x.shape[1], p)
    q = _quantise_exact(x, p)
    want = np.array([[np.float32(float(Fraction(int(q[i, j]), 10 ** p))) for j in range(x.shape[1])] for i in range(x.shape[0])],
                    dtype=np.float32)
    assert np.array_equal(back, want)
    assert np.all(np.abs(back.astype(np.float64) - x.astype(np.float64)) <= 0.5 * 10.0 ** -p + 2e-7 * np.abs(x) + 1e-12)


def test_round_trip_is_idempotent_and_sizes_add_up():
    rng = np.random.default_rng(3)
    x = (rng.normal(size=(40, 33)) * 3).astype(np.float32)
    x[5] = 0.0                                    # an all-zero row: one byte per value
    data, off = orc.codec_encode(x, 3)
    assert off[0] == 0 and off[-1] == data.shape[0] and np.all(np.diff(off) >= x.shape[1])
    assert off[6] - off[5] == x.shape[1] and bytes(data[off[5]:off[6]]) == b"?" * x.shape[1]
    assert data.min() >= 63 and data.max() <= 126  # printable ASCII, as the scheme promises
    once = orc.codec_decode(data, off, x.shape[1], 3)
    data2, off2 = orc.codec_encode(once, 3)
    assert np.array_equal(data, data2) and np.array_equal(off, off2)
    # ReLU outputs at three decimals compress well below 4 bytes per value
    h = np.maximum(rng.normal(size=(64, 256)), 0).astype(np.float32)
    hd, ho = orc.codec_encode(h, 2)
    assert ho[-1] < 0.6 * h.size * 4


def test_malformed_rows_are_rejected():
    data, off = orc.codec_encode(np.array([[1.0, 2.0, 3.0]], dtype=np.float32), 1)
    with pytest.raises(ValueError):
        orc.codec_decode(data, off, 4, 1)          # one value too many asked for
    with pytest.raises(ValueError):
        orc.codec_decode(data, off, 2, 1)          # bytes left over
    bad = data.copy()
    bad[-1] = ord("_")                             # continuation bit on the last byte: the value never ends
    with pytest.raises(ValueError):
        orc.codec_decode(bad, off, 3, 1)
