"""Pins for the oracle's MXINT quantiser (Section 2.2, Section 4.1)."""
import os

import numpy as np
import pytest

from oracle import mxint

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "mxint_blocks.txt")


def _golden_blocks():
    out = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            bits, vals, e, mant = [p.strip() for p in line.split(";")]
            out.append((int(bits), [float(x) for x in vals.split()], int(e), [int(x) for x in mant.split()]))
    return out


@pytest.mark.parametrize("bits,vals,e,mant", _golden_blocks())
def test_hand_worked_blocks(bits, vals, e, mant):
    v = np.zeros(16, np.float32)
    v[: len(vals)] = np.array(vals, dtype=np.float32)
    m, ex = mxint.quantize(v, bits, axis=0)
    assert ex.shape == (1,) and int(ex[0]) == e
    assert m[: len(mant)].tolist() == mant
    assert not m[len(mant):].any()
    # dequantised value is mantissa * 2^(e-(bits-2))
    dq = mxint.dequantize(m, ex, bits, axis=0)
    assert np.array_equal(dq[: len(mant)], np.array(mant) * 2.0 ** (e - (bits - 2)))


def test_hand_worked_dot_product():
    # The MXINT inner product is an integer dot plus an exponent addition (Section 2.2):
    # m_x = [32,-16,24,96] (e_x = 1), m_w = [3,-2,6,0] (e_w = -5): 272 * 2^(1-6) * 2^(-5-2) = 272 * 2^-12
    x = np.zeros(16, np.float32); x[:4] = [1, -0.5, 0.75, 3]
    w = np.zeros(16, np.float32); w[:4] = [0.02, -0.013, 0.05, 0.0039]
    xm, xe = mxint.quantize(x, 8, 0)
    wm, we = mxint.quantize(w, 4, 0)
    idot = int(np.dot(xm.astype(np.int64), wm.astype(np.int64)))
    assert idot == 272
    val = idot * 2.0 ** (int(xe[0]) - 6 + int(we[0]) - 2)
    assert val == 0.06640625
    assert float(mxint.dequantize(xm, xe, 8, 0) @ mxint.dequantize(wm, we, 4, 0)) == val


def _rand_blocks(seed, n=400, scale_spread=12):
    g = np.random.default_rng(seed)
    v = g.standard_normal((n, 16)) * np.exp2(g.integers(-scale_spread, scale_spread, size=(n, 1)))
    return v.astype(np.float32)


@pytest.mark.parametrize("bits", [2, 4, 6, 8])
def test_invariants(bits):
    v = _rand_blocks(bits)
    m, e = mxint.quantize(v, bits, axis=1)
    qmax = 2 ** (bits - 1) - 1
    assert m.min() >= -qmax and m.max() <= qmax
    dq = mxint.dequantize(m, e, bits, axis=1)
    # idempotence: q(dq(q(v))) == q(v) unless the block maximum was clipped at a binade edge
    m2, e2 = mxint.quantize(dq, bits, axis=1)
    assert np.array_equal(mxint.dequantize(m2, e2, bits, axis=1), dq)
    # odd symmetry
    mn, en = mxint.quantize(-v, bits, axis=1)
    assert np.array_equal(mn, -m) and np.array_equal(en, e)
    # scaling by a power of two moves only the exponent
    for j in (-5, 3):
        mj, ej = mxint.quantize(v * np.float32(2.0 ** j), bits, axis=1)
        assert np.array_equal(mj, m) and np.array_equal(ej, e + j)
    # the exponent is the fp32 exponent field of the block maximum
    amax = np.abs(v).max(axis=1)
    field = ((amax.view(np.uint32) >> 23) & 0xFF).astype(np.int64) - 127
    assert np.array_equal(e[:, 0], field)
    # error bound: half a step, one step where the value was clipped
    step = np.exp2(e.astype(np.float64) - (bits - 2))
    err = np.abs(v.astype(np.float64) - dq)
    clipped = np.abs(np.rint(v / step)) > qmax
    assert np.all(err[~clipped] <= 0.5 * step.repeat(16, axis=1)[~clipped])
    assert np.all(err[clipped] <= step.repeat(16, axis=1)[clipped])
    # block maximum lands in [2^(bits-2), 2^(bits-1)) steps before rounding
    top = amax / step[:, 0]
    assert np.all(top >= 2 ** (bits - 2)) and np.all(top < 2 ** (bits - 1))


def test_block_orientation():
    # blocks run along the chosen axis only: [1,16] for X, [16,1] for W (Section 4.1)
    g = np.random.default_rng(5)
    v = g.standard_normal((32, 48)).astype(np.float32)
    m0, e0 = mxint.quantize(v, 8, axis=0)
    assert m0.shape == (32, 48) and e0.shape == (2, 48)
    m1, e1 = mxint.quantize(v, 8, axis=1)
    assert e1.shape == (32, 3)
    mt, et = mxint.quantize(v.T.copy(), 8, axis=1)
    assert np.array_equal(mt.T, m0) and np.array_equal(et.T, e0)
    # a block's result depends on that block only
    v2 = v.copy(); v2[16:, :] *= 100
    m2, e2 = mxint.quantize(v2, 8, axis=0)
    assert np.array_equal(m2[:16], m0[:16]) and np.array_equal(e2[0], e0[0])
    assert not np.array_equal(e2[1], e0[1])


def test_window_and_specials():
    v = np.zeros((4, 16), np.float32)
    v[0, 0] = 2.0 ** -70          # below the window -> e = exp_min, mantissa rounds to 0
    v[1, 0] = 2.0 ** 80           # above the window -> e = exp_max, saturates
    v[2, 0] = np.inf; v[2, 1] = -np.inf; v[2, 2] = 1.0
    v[3, 0] = np.nan; v[3, 1] = 0.75
    m, e = mxint.quantize(v, 8, axis=1)
    assert e[:, 0].tolist() == [mxint.EXP_MIN, mxint.EXP_MAX, mxint.EXP_MAX, -1]
    assert m[0, 0] == 0 and m[1, 0] == 127
    assert m[2, :3].tolist() == [127, -127, 0]
    assert m[3, 0] == 0 and m[3, 1] == 96
    assert mxint.exponent_bytes(e)[:, 0].tolist() == [71, 182, 182, 126]


def test_four_bit_exponent_window():
    # A 4-bit shared exponent holds 16 values (Section 4.1: weights and low-rank matrices); with the window [-12, 3]:
    # a block max of 0.05 (e = -5) is inside and quantises as in the wide window; 2^-20 is below it and takes
    # e = -12, step 2^-14 (4-bit), so 2^-13 = 2 steps -> 2 and 2^-20 -> 0; 100 (e = 6) is above it and takes e = 3,
    # step 2: 100 / 2 = 50 -> clamped to 7, 5 -> 2.5 steps -> 2 (half to even), 7 -> 3.5 steps -> 4.
    v = np.zeros((3, 16), np.float32)
    v[0, :4] = [0.02, -0.013, 0.05, 0.0039]
    v[1, :2] = [2.0 ** -13, 2.0 ** -20]
    v[2, :3] = [100.0, 5.0, 7.0]
    m, e = mxint.quantize(v, 4, axis=1, exp_min=-12, exp_max=3)
    assert e[:, 0].tolist() == [-5, -12, 3]
    assert m[0, :4].tolist() == [3, -2, 6, 0]
    assert m[1, :2].tolist() == [2, 0]
    assert m[2, :3].tolist() == [7, 2, 4]
    assert mxint.exponent_bytes(e)[:, 0].tolist() == [122, 115, 130]


def test_padding_is_neutral():
    g = np.random.default_rng(9)
    b = g.standard_normal((8, 5)).astype(np.float32)
    bp = mxint.pad_axis(b, axis=0)
    assert bp.shape == (16, 5) and not bp[8:].any()
    m, e = mxint.quantize(bp, 8, axis=0)
    amax = np.abs(b).max(axis=0)
    assert np.array_equal(e[0], np.floor(np.log2(amax)).astype(np.int64))
    assert not m[8:].any()


def test_round_bf16_hand_cases_and_library_agreement():
    # bfloat16 keeps 8 significant bits: the spacing in [1, 2) is 2^-7
    cases = [(1.0 + 2.0 ** -8, 1.0),                       # exact tie, lower neighbour has the even mantissa
             (1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -6),       # exact tie, upper neighbour is even
             (1.0 + 2.0 ** -8 + 2.0 ** -20, 1.0 + 2.0 ** -7),
             (-0.3, -0.30078125), (3.14159, 3.140625), (255.5, 256.0), (0.0, 0.0), (1e-3, 0.00099945068359375)]
    for v, want in cases:
        assert mxint.round_bf16(np.array([v]))[0] == want, v
    # a correctly rounded value is within half a spacing, and the result is a fixed point
    g = np.random.default_rng(5)
    x = g.standard_normal(4000) * np.exp2(g.integers(-20, 20, 4000))
    r = mxint.round_bf16(x)
    assert np.all(np.abs(r - x) <= mxint.bf16_half_ulp(x))
    assert np.array_equal(mxint.round_bf16(r), r)
    # against a library's conversion (fp32 inputs, so that both start from the same number)
    torch = pytest.importorskip("torch")
    x32 = x.astype(np.float32)
    lib = torch.from_numpy(x32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(mxint.round_bf16(x32), lib)
