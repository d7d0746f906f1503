"""Pins for the CPU oracle: values the paper prints, closed forms, brute force.

Every check here compares the oracle with something other than itself: the
worked examples of Sec. 3.2 / 3.3 (fixtures under tests/golden/), exhaustive
search in exact rational arithmetic, a textbook FP4 E2M1 rounding routine, and
invariants that hold for any input.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2501_01144_b200 import inputs

FB = oracle.formatbook()


# ----------------------------------------------------------------------------
# Formatbook: printed rows and the structure Sec. 3.1 states
# ----------------------------------------------------------------------------
def test_dialect4_and_5_match_printed_values(golden_dialect4):
    g = golden_dialect4
    assert list(FB[4]) == sorted(g["dialect4_values_desc"])
    big, small = (int(2 * v) for v in g["pair_differing_real"])
    assert big in FB[4] and small not in FB[4]
    assert small in FB[5] and big not in FB[5]
    assert sorted(set(FB[4]) - {big}) == sorted(set(FB[5]) - {small})
    assert FB[4][7] == FB[5][7] == int(2 * g["pair_shared_max_real"][0])


def test_formatbook_equals_the_stated_reading():
    # typo guard, not a paper value: the table as this build's reading of Sec. 3.1 states it, row by row
    from conftest import read_golden
    g = read_golden("formatbook_reading.txt")
    for d in range(16):
        assert list(FB[d]) == g[f"dialect{d}"], f"dialect {d}"


def test_formatbook_structure():
    maxima = []
    for p in range(8):
        even, odd = FB[2 * p], FB[2 * p + 1]
        for row in (even, odd):
            assert list(row) == sorted(set(row)) and len(set(row)) == 8     # ascending, distinct
            assert row[0] == 0 and row[7] <= 15                             # 0 .. 7.5 in 0.5 steps
        assert even[7] == odd[7]                                            # shared maximum
        diff = [j for j in range(8) if even[j] != odd[j]]
        assert diff == [6] and even[6] > odd[6]                             # one large value differs
        maxima.append(int(even[7]))
    assert maxima == list(range(15, 7, -1))                                 # 7.5 ... 4.0, all maxima
    fp4_six = [0, 1, 2, 3, 4, 6]                                            # E2M1: 0 .5 1 1.5 2 3
    assert sum(list(FB[d][:6]) == fp4_six for d in range(16)) >= 14         # "most" stay FP4's
    assert list(FB[7]) == [0, 1, 2, 3, 4, 6, 8, 12]                         # FP4 E2M1 itself


def test_effective_bits_closed_form():
    for line in open(os.path.join(os.path.dirname(__file__), "golden", "effective_bits.txt")):
        if line.startswith("#") or not line.strip():
            continue
        bs, bd, mx = line.split()
        bs = int(bs)
        # 4-bit element + (5-bit exponent + 4-bit dialect id) per block, printed with two decimals
        assert abs((4 + 9 / bs) - float(bd)) <= 0.005 + 1e-9
        assert abs((4 + 5 / bs) - float(mx)) <= 0.005 + 1e-9
    # canonical storage here: 16 code bytes + 1 id byte + 1 scale byte per block of 32
    codes, ids, scales = oracle.quantize(np.ones((3, 64), np.float32))
    assert codes.nbytes == 3 * 64 // 2 and ids.nbytes == scales.nbytes == 3 * 2


# ----------------------------------------------------------------------------
# Beneficial ranges (Sec. 3.2, stage 2)
# ----------------------------------------------------------------------------
def test_beneficial_range_dialect4_printed(golden_dialect4):
    g = golden_dialect4
    lo, hi = oracle.beneficial_range(4)
    assert (Fraction(lo, 4), Fraction(hi, 4)) == tuple(Fraction(v) for v in g["dialect4_range_real"])
    assert lo <= g["dialect4_range_top_code"][0] < hi
    assert not (lo <= g["dialect4_range_excluded_code"][0] < hi)
    prefix = g["dialect4_range_prefix4"][0]
    inside = [k for k in range(32) if lo <= k < hi]
    assert all(k in inside for k in range(32) if k >> 1 == prefix)


def test_beneficial_ranges_follow_midpoint_rule():
    for p in range(8):
        even, odd = [Fraction(int(v), 2) for v in FB[2 * p]], [Fraction(int(v), 2) for v in FB[2 * p + 1]]
        mid_pair = (even[6] + odd[6]) / 2
        assert oracle.beneficial_range(2 * p) == (int(4 * mid_pair), int(4 * (even[6] + even[7]) / 2))
        assert oracle.beneficial_range(2 * p + 1) == (int(4 * (odd[6] + odd[5]) / 2), int(4 * mid_pair))
        # inside its range a dialect's differing value is strictly nearer than any value of its partner
        for d, mine, other in ((2 * p, even, odd), (2 * p + 1, odd, even)):
            lo, hi = oracle.beneficial_range(d)
            for k in range(lo, hi):
                x = Fraction(k, 4) + Fraction(1, 8)   # a point strictly inside the code's cell
                assert abs(x - mine[6]) < min(abs(x - v) for v in other)


# ----------------------------------------------------------------------------
# Element rounding (Sec. 3.3)
# ----------------------------------------------------------------------------
def test_printed_rounding_example(golden_dialect4):
    g = golden_dialect4
    idx = oracle.round_code(4, g["example_code"][0])
    assert idx == g["example_index"][0]
    assert FB[4][idx] == g["example_value_half_units"][0]


def test_value10_boolean_form(golden_dialect4):
    g = golden_dialect4
    for k in range(32):
        bits = [(k >> i) & 1 for i in range(5)]
        printed = bool(bits[4] and not bits[3] and not (bits[2] and bits[1] and bits[0]))
        in_interval = g["value10_code_lo"][0] <= k <= g["value10_code_hi"][0]
        assert printed == in_interval
        assert (FB[4][oracle.round_code(4, k)] == 10) == printed


def _nearest_exhaustive(values, x):
    """Nearest of `values` to the real x; of two equally near the larger."""
    best = None
    for v in values:
        if best is None or abs(x - v) < abs(x - best) or (abs(x - v) == abs(x - best) and v > best):
            best = v
    return best


def test_rounding_equals_exhaustive_nearest_on_reals():
    rng = np.random.default_rng(11)
    for d in range(16):
        values = [Fraction(int(v), 2) for v in FB[d]]
        xs = [Fraction(n, 4) for n in range(32)]                                   # every boundary and tie
        xs += [Fraction(int(n), 1 << 20) for n in rng.integers(0, 8 << 20, 400)]   # untruncated reals
        for x in xs:
            q5 = int(x * 4)                                                         # truncation to 2 fraction bits
            got = Fraction(int(FB[d][oracle.round_code(d, q5)]), 2)
            assert got == _nearest_exhaustive(values, x), (d, x)


def _e2m1_round(x):
    """Textbook FP4 E2M1 (1-2-1) round-to-nearest of a magnitude, ties to the larger magnitude, saturating."""
    if x >= 6:
        return Fraction(6)
    if x < 1:                       # subnormal binade: spacing 0.5
        step = Fraction(1, 2)
    else:
        step = Fraction(2) ** (int(math.floor(math.log2(float(x)))) - 1)   # one mantissa bit per binade
    return min(Fraction(math.floor(x / step + Fraction(1, 2))) * step, Fraction(6))


def test_dialect7_is_fp4_e2m1():
    rng = np.random.default_rng(12)
    xs = [Fraction(n, 4) for n in range(32)] + [Fraction(int(n), 1 << 16) for n in rng.integers(0, 8 << 16, 500)]
    for x in xs:
        got = Fraction(int(FB[7][oracle.round_code(7, int(x * 4))]), 2)
        assert got == _e2m1_round(x), x


# ----------------------------------------------------------------------------
# Whole-block brute force in exact rational arithmetic
# ----------------------------------------------------------------------------
def _exact_block_two_stage(xs):
    """Two-stage rule restated with rationals and the paper's real-valued wording."""
    mags = [abs(Fraction(float(v))) for v in xs]
    amax = max(mags)
    if amax == 0:
        e = -127
    else:
        e = -200
        while Fraction(2) ** (e + 1) <= amax:    # floor(log2 amax) by search
            e += 1
        e = max(e - 2, -127)
    scaled = [m / Fraction(2) ** e for m in mags]
    trunc = [Fraction(math.floor(s * 4), 4) for s in scaled]          # two fraction bits kept
    bmax = min(Fraction(math.floor(max(trunc) * 2 + Fraction(1, 2)), 2), Fraction(15, 2))   # round to 0.5
    pair = next((p for p in range(8) if Fraction(int(FB[2 * p][7]), 2) == bmax), 7)
    ev = [Fraction(int(v), 2) for v in FB[2 * pair]]
    od = [Fraction(int(v), 2) for v in FB[2 * pair + 1]]
    mid = (ev[6] + od[6]) / 2
    cnt_e = sum(mid <= t < (ev[6] + ev[7]) / 2 for t in trunc)
    cnt_o = sum((od[6] + od[5]) / 2 <= t < mid for t in trunc)
    d = 2 * pair if cnt_e >= cnt_o else 2 * pair + 1
    vals = [Fraction(int(v), 2) for v in FB[d]]
    idx = [vals.index(_nearest_exhaustive(vals, s)) for s in scaled]   # nearest on the UNtruncated value
    return e, d, idx


def _unpack(codes_row):
    out = []
    for byte in codes_row:
        out += [int(byte) & 15, int(byte) >> 4]
    return out


@pytest.mark.parametrize("seed", range(4))
def test_two_stage_blocks_against_rational_brute_force(seed):
    rng = np.random.default_rng(100 + seed)
    rows = []
    for _ in range(24):
        kind = rng.integers(0, 5)
        b = rng.standard_normal(32)
        if kind == 1:
            b[rng.integers(0, 32)] *= 50.0                          # one outlier
        elif kind == 2:
            b = rng.uniform(0.55, 0.99, 32) * rng.choice([-1, 1], 32)   # many values near the maximum
        elif kind == 3:
            b = np.round(b * 4) / 4                                  # exact ties on the grid
        elif kind == 4:
            b *= 2.0 ** rng.integers(-40, 40)
        rows.append(b)
    x = np.array(rows, np.float32)
    codes, ids, scales = oracle.quantize(x)
    for r in range(x.shape[0]):
        e, d, idx = _exact_block_two_stage(x[r])
        assert int(scales[r, 0]) - 127 == e
        assert int(ids[r, 0]) == d
        nib = _unpack(codes[r])
        assert [n & 7 for n in nib] == idx
        assert [n >> 3 for n in nib] == [int(np.signbit(v)) for v in x[r]]


def test_stage1_rounds_block_max_to_half_grid():
    # scaled block maxima chosen around the rounding boundaries of Sec. 3.2 stage 1
    cases = {6.70: 13, 6.74: 13, 6.75: 14, 7.24: 14, 7.25: 15, 7.99: 15, 4.0: 8, 4.24: 8, 4.25: 9}
    for smax, want_max in cases.items():
        b = np.full(32, 0.1, np.float32)
        b[5] = smax                   # 4 <= smax < 8: shared exponent 0
        _, ids, scales = oracle.quantize(b[None, :])
        assert int(scales[0, 0]) == 127
        assert int(FB[ids[0, 0]][7]) == want_max, smax


def test_stage2_counts_decide_within_pair():
    base = np.full(32, 0.1, np.float32)
    base[0] = 6.5                     # pair (4, 5)
    a = base.copy(); a[1:4] = 5.0; a[4:6] = 4.0       # three in [4.5,5.75), two in [3.5,4.5)
    b = base.copy(); b[1:3] = 5.0; b[3:6] = 4.0       # two versus three
    c = base.copy(); c[1:3] = 5.0; c[3:5] = 4.0       # equal counts -> even
    d = base.copy()                                    # nothing in either range -> even
    ids = oracle.quantize(np.stack([a, b, c, d]))[1][:, 0]
    assert list(ids) == [4, 5, 4, 4]


def _exact_mse_errors(xs, e):
    mags = [abs(Fraction(float(v))) / Fraction(2) ** e for v in xs]
    errs = []
    for d in range(16):
        vals = [Fraction(int(v), 2) for v in FB[d]]
        errs.append(sum((m - _nearest_exhaustive(vals, m)) ** 2 for m in mags))
    return errs


def test_mse_selection_against_exhaustive_rational_errors():
    rng = np.random.default_rng(7)
    x = rng.standard_normal((48, 32)).astype(np.float32)
    x[::3, 4] *= 30.0
    x[1::3] = np.abs(x[1::3]) ** 0.3 * np.sign(x[1::3])
    codes, ids, scales = oracle.quantize(x, oracle.SELECT_MSE)
    c2, i2, s2 = oracle.quantize(x, oracle.SELECT_TWO_STAGE)
    assert (scales == s2).all()                       # the exponent does not depend on the rule
    for r in range(x.shape[0]):
        errs = _exact_mse_errors(x[r], int(scales[r, 0]) - 127)
        best = min(errs)
        winners = [d for d in range(16) if errs[d] == best]
        assert int(ids[r, 0]) == winners[0], (r, winners)          # lowest id among exact minima
        # codes are the nearest values under that dialect
        vals = [Fraction(int(v), 2) for v in FB[ids[r, 0]]]
        mags = [abs(Fraction(float(v))) / Fraction(2) ** (int(scales[r, 0]) - 127) for v in x[r]]
        assert [n & 7 for n in _unpack(codes[r])] == [vals.index(_nearest_exhaustive(vals, m)) for m in mags]
        # and the max-based rule never beats it
        assert errs[int(i2[r, 0])] >= best


# ----------------------------------------------------------------------------
# Invariants on realistic data
# ----------------------------------------------------------------------------
def test_invariants_on_tiny_case():
    X, W = inputs.tiny_case()
    for x, rule in ((X, oracle.SELECT_TWO_STAGE), (W, oracle.SELECT_MSE)):
        codes, ids, scales = oracle.quantize(x, rule)
        dq = oracle.dequantize(codes, ids, scales)
        xb = x.reshape(x.shape[0], -1, 32).astype(np.float64)
        e = scales.astype(np.int64) - 127
        scaled_max = np.abs(xb).max(-1) / np.exp2(e)
        assert ((scaled_max >= 4) & (scaled_max < 8)).all()                    # Sec. 3.1: range [0, 8)
        grid = np.abs(dq.reshape(xb.shape)) / np.exp2(e)[..., None] * 2        # half-units
        assert (grid == np.round(grid)).all() and grid.max() <= 15
        for r in range(x.shape[0]):
            for b in range(ids.shape[1]):
                allowed = set(int(v) for v in FB[ids[r, b]])
                assert set(int(v) for v in grid[r, b]) <= allowed             # on the chosen dialect's grid
        assert (np.signbit(dq) == np.signbit(x)).all()
        # error at most half the local gap, or the clip distance above the dialect maximum
        err = np.abs(np.abs(dq) - np.abs(x.astype(np.float64))).reshape(xb.shape) / np.exp2(e)[..., None]
        for r in range(x.shape[0]):
            for b in range(ids.shape[1]):
                vals = FB[ids[r, b]].astype(np.float64) / 2
                s = np.abs(xb[r, b]) / 2.0 ** e[r, b]
                j = np.clip(np.searchsorted(vals, s, side="right") - 1, 0, 6)
                bound = np.where(s > vals[7], s - vals[7], (vals[j + 1] - vals[j]) / 2)
                assert (err[r, b] <= bound + 1e-12).all()


def test_zero_block_sign_passthrough_and_clamp():
    x = np.zeros((3, 32), np.float32)
    x[0, 3] = -0.0
    x[1] = 1e-44                         # fp32 subnormals: exponent clamps at -127
    x[1, 0] = -3e-45
    x[2] = 2.0 ** -125                   # floor(log2) - 2 == -127 exactly, no clamp needed
    codes, ids, scales = oracle.quantize(x)
    assert int(scales[0, 0]) == 0 and int(ids[0, 0]) == 14
    nib = _unpack(codes[0])
    assert nib[3] == 8 and sum(nib) == 8
    assert int(scales[1, 0]) == 0 and int(ids[1, 0]) >= 14        # scaled maximum < 4 -> last pair
    assert int(scales[2, 0]) == 0 and int(FB[ids[2, 0]][7]) == 8
    dq = oracle.dequantize(codes, ids, scales)
    assert np.signbit(dq[0, 3]) and dq[0, 3] == 0
    assert np.signbit(dq[1, 0])
    assert abs(dq[2, 0] - 2.0 ** -125) == 0


def test_nonfinite_rejected():
    x = np.ones((1, 32), np.float32)
    x[0, 9] = np.inf
    with pytest.raises(FloatingPointError):
        oracle.quantize(x)


def test_16bit_inputs_read_exactly():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((4, 64)).astype(np.float32)
    xb = inputs.to_bf16_bits(x)
    a = oracle.quantize(xb, dtype=oracle.BF16)
    b = oracle.quantize(inputs.bf16_bits_to_f32(xb))
    assert all((u == v).all() for u, v in zip(a, b))
    xh = (x * 1e-3).astype(np.float16)
    xh[0, :8] = np.float16(6e-8) * np.arange(8)       # fp16 subnormals
    a = oracle.quantize(xh.view(np.uint16), dtype=oracle.F16)
    b = oracle.quantize(xh.astype(np.float32))
    assert all((u == v).all() for u, v in zip(a, b))


# ----------------------------------------------------------------------------
# GEMM reference (Sec. 3.3 block MAC)
# ----------------------------------------------------------------------------
def test_gemm_against_rational_brute_force_and_block_mac():
    rng = np.random.default_rng(3)
    A = rng.standard_normal((3, 64)).astype(np.float32)
    A[:, 5] *= 40
    B = (0.02 * rng.standard_normal((5, 64))).astype(np.float32)
    qa, qb = oracle.quantize(A), oracle.quantize(B, oracle.SELECT_MSE)
    da, db = oracle.dequantize(*qa), oracle.dequantize(*qb)
    Y, T = oracle.gemm(da, db)
    for m in range(3):
        for n in range(5):
            exact = sum(Fraction(float(u)) * Fraction(float(v)) for u, v in zip(da[m], db[n]))
            exact_abs = sum(abs(Fraction(float(u)) * Fraction(float(v))) for u, v in zip(da[m], db[n]))
            assert abs(Fraction(float(Y[m, n])) - exact) <= exact_abs * Fraction(1, 10 ** 13)
            assert abs(Fraction(float(T[m, n])) - exact_abs) <= exact_abs * Fraction(1, 10 ** 13)
    # integer in-block sums, one rescale by 2^(eA+eB-2) per block: same result up to fp64 rounding
    Yb = oracle.gemm_blockmac(qa, qb)
    assert np.abs(Yb - Y).max() <= 1e-13 * T.max()
    # a transposed operand would be caught: result is not symmetric in general
    assert Y.shape == (3, 5)


def test_alternative_formatbook_in_the_oracle():
    """bdo_set_formatbook: the selection and rounding follow whatever table is loaded (checked against the
    plain definitions on that table), malformed tables are refused, None restores the default."""
    default = oracle.formatbook()
    alt = default.copy()
    alt[0, 6], alt[1, 6] = 13, 11                       # other slot-6 values for pair 0
    alt[6] = [0, 1, 2, 3, 5, 7, 10, 12]                 # another common set for pair 3
    alt[7] = [0, 1, 2, 3, 5, 7, 8, 12]
    try:
        oracle.set_formatbook(alt)
        assert (oracle.formatbook() == alt).all()
        # beneficial ranges from the definition (Sec. 3.2): even [ (dE+dO)/2, (dE+max)/2 ), odd [ (v5+dO)/2, (dE+dO)/2 )
        for p in (0, 3):
            ev, od = [int(v) for v in alt[2 * p]], [int(v) for v in alt[2 * p + 1]]
            assert oracle.beneficial_range(2 * p) == (ev[6] + od[6], ev[6] + ev[7])
            assert oracle.beneficial_range(2 * p + 1) == (od[5] + od[6], ev[6] + od[6])
        # rounding = nearest value of the loaded table, ties toward the larger magnitude
        for d in (0, 1, 6, 7):
            vals = [Fraction(int(v), 2) for v in alt[d]]
            for q5 in range(32):
                x = Fraction(q5, 4)
                best = min(range(8), key=lambda j: (abs(vals[j] - x), -vals[j]))
                assert oracle.round_code(d, q5) == best, (d, q5)
        # a block whose maximum rounds to 6.0 lands in pair 3 and is quantised with the new values
        x = np.zeros((1, 32), np.float32)
        x[0, :4] = [6.0, 5.1, 3.4, -2.6]                # e = 0; 5.1 -> 5.0 exists only in the even member
        codes, ids, scales = oracle.quantize(x)
        assert int(ids[0, 0]) in (6, 7) and int(scales[0, 0]) == 127
        deq = oracle.dequantize(codes, ids, scales)[0, :4]
        allowed = set(float(v) / 2 for v in alt[int(ids[0, 0])])
        assert all(abs(float(v)) in allowed for v in deq)
        bad = alt.copy()
        bad[6, 7] = 11
        with pytest.raises(ValueError):
            oracle.set_formatbook(bad)
        assert (oracle.formatbook() == alt).all()
    finally:
        oracle.set_formatbook(None)
    assert (oracle.formatbook() == default).all()


def test_power_of_two_scaling_moves_only_the_exponent():
    """Scaling a block by 2^k is exact in binary floating point, so codes and dialect must not change and the
    stored exponent moves by k (Sec. 3.2: the shared exponent absorbs the block's magnitude); flipping every
    sign flips every sign bit and nothing else; permuting the elements of a block permutes its codes."""
    rng = np.random.default_rng(31)
    x = (rng.standard_t(4, (6, 96)) * np.exp2(rng.integers(-3, 4, (6, 1)))).astype(np.float32)
    codes, ids, scales = oracle.quantize(x)
    for k in (-9, -1, 3, 17):
        c2, i2, s2 = oracle.quantize(np.ldexp(x, k).astype(np.float32))
        assert np.array_equal(c2, codes) and np.array_equal(i2, ids)
        assert np.array_equal(s2.astype(int), scales.astype(int) + k)
    cn, in_, sn = oracle.quantize(-x)
    assert np.array_equal(in_, ids) and np.array_equal(sn, scales)
    assert np.array_equal(cn ^ 0x88, codes)                       # bit 3 of each nibble is the sign
    perm = rng.permutation(32)
    xp = x.reshape(6, 3, 32)[:, :, perm].reshape(6, 96)
    cp, ip, sp = oracle.quantize(xp)
    assert np.array_equal(ip, ids) and np.array_equal(sp, scales)
    nib = lambda c: np.stack([c & 15, c >> 4], -1).reshape(6, 3, 32)
    assert np.array_equal(nib(cp), nib(codes)[:, :, perm])
    for select in (oracle.SELECT_MSE,):
        a = oracle.quantize(x, select)
        b = oracle.quantize(np.ldexp(x, 5).astype(np.float32), select)
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_error_bound_and_idempotence():
    """Within a block the dequantised value lies within half a grid step of the input, where the step between the
    chosen dialect's neighbouring values is at most 2.5 units above the common values (Sec. 3.1: granularity 0.5
    below, one differing large value above), and never exceeds the rounded block maximum; quantising the
    dequantised values again reproduces codes, dialect and exponent (the grid points are fixed points)."""
    rng = np.random.default_rng(32)
    x = (rng.standard_normal((40, 64)) * np.exp2(rng.integers(-8, 8, (40, 1)))).astype(np.float32)
    x[:, 5] *= 13
    FB = oracle.formatbook()
    for select in (oracle.SELECT_TWO_STAGE, oracle.SELECT_MSE):
        codes, ids, scales = oracle.quantize(x, select)
        deq = oracle.dequantize(codes, ids, scales)
        for r in range(x.shape[0]):
            for b in range(2):
                seg = slice(32 * b, 32 * b + 32)
                e = int(scales[r, b]) - 127
                vals = FB[ids[r, b]].astype(np.float64) / 2
                gaps = np.diff(vals)
                scaled_in = np.abs(x[r, seg].astype(np.float64)) / 2.0 ** e
                scaled_out = np.abs(deq[r, seg]) / 2.0 ** e
                assert np.all(np.isin(scaled_out, vals))
                # the truncated 5-bit magnitude is what gets rounded: up to 0.25 lost, then half the local gap,
                # and values beyond the dialect's maximum saturate at it
                inside = scaled_in <= vals[-1]
                assert np.all(np.abs(scaled_out - scaled_in)[inside] <= 0.25 + gaps.max() / 2 + 1e-12)
                assert np.all(scaled_out[~inside] == vals[-1])
                assert np.all(scaled_in < 8.0)
        c2, i2, s2 = oracle.quantize(deq.astype(np.float32), oracle.SELECT_TWO_STAGE)
        if select == oracle.SELECT_TWO_STAGE:
            assert np.array_equal(s2, scales)
            assert np.array_equal(oracle.dequantize(c2, i2, s2), deq)


# ----------------------------------------------------------------------------
# Block sizes 16 and 64 (the block-size study of Sec. 4.2, Table 3): the same steps over a block of another length
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("block", [16, 64])
def test_other_block_sizes_against_rational_brute_force(block):
    rng = np.random.default_rng(300 + block)
    x = rng.standard_normal((12, 4 * block)).astype(np.float32)
    x[::3, 5] *= 60.0                                            # an outlier in the first block of some rows
    x[1::4] = np.round(x[1::4] * 4) / 4                          # exact ties on the grid
    x[2] *= 2.0 ** -30
    codes, ids, scales = oracle.quantize(x, block=block)
    assert ids.shape == scales.shape == (12, 4)
    for r in range(x.shape[0]):
        nib = _unpack(codes[r])
        for b in range(4):
            seg = x[r, b * block:(b + 1) * block]
            e, d, idx = _exact_block_two_stage(seg)              # the restatement takes any block length
            assert int(scales[r, b]) - 127 == e
            assert int(ids[r, b]) == d
            assert [n & 7 for n in nib[b * block:(b + 1) * block]] == idx
            assert [n >> 3 for n in nib[b * block:(b + 1) * block]] == [int(np.signbit(v)) for v in seg]


@pytest.mark.parametrize("block", [16, 64])
def test_other_block_sizes_mse_rule_and_product(block):
    rng = np.random.default_rng(310 + block)
    x = rng.standard_normal((6, 2 * block)).astype(np.float32)
    x[:, 3] *= 25.0
    codes, ids, scales = oracle.quantize(x, oracle.SELECT_MSE, block=block)
    for r in range(x.shape[0]):
        for b in range(2):
            errs = _exact_mse_errors(x[r, b * block:(b + 1) * block], int(scales[r, b]) - 127)
            assert int(ids[r, b]) == errs.index(min(errs))       # lowest id among exact minima
    # dequantised values sit on the block's grid, and the block MAC with one rescale per block equals the fp64 product
    w = (0.02 * rng.standard_normal((5, 2 * block))).astype(np.float32)
    qa, qb = oracle.quantize(x, block=block), oracle.quantize(w, block=block)
    da, db = oracle.dequantize(*qa), oracle.dequantize(*qb)
    for r in range(x.shape[0]):
        for b in range(2):
            grid = {float(v) * 0.5 * 2.0 ** (int(qa[2][r, b]) - 127) for v in FB[qa[1][r, b]]}
            assert set(np.abs(da[r, b * block:(b + 1) * block]).tolist()) <= grid
    Y, T = oracle.gemm(da, db)
    assert np.abs(oracle.gemm_blockmac(qa, qb) - Y).max() <= 1e-13 * T.max()


def test_smaller_blocks_never_share_an_exponent_across_their_border():
    # two halves of a 32-element row six binades apart: block 16 gives each half its own exponent, block 32 one
    x = np.concatenate([np.full(16, 5.0), np.full(16, 5.0 / 64)]).astype(np.float32)[None, :]
    s16 = oracle.quantize(x, block=16)[2]
    s32 = oracle.quantize(x, block=32)[2]
    assert s16.tolist() == [[127, 121]] and s32.tolist() == [[127]]
    assert np.array_equal(oracle.dequantize(*oracle.quantize(x, block=16)), x.astype(np.float64))   # both halves exact
    assert np.abs(oracle.dequantize(*oracle.quantize(x, block=32))[0, 16:]).max() == 0.0            # the small half is lost
