"""Pins for the CPU oracle: every check here is something the paper's equations or plain
mathematics fix, evaluated by a route that does not go through the oracle's own code
(hand-worked closed forms, exact rational arithmetic, numpy int64 products, brute-force
Python loops, numpy's own FP16 conversion)."""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- FP16

def test_half_to_float_matches_numpy_exhaustively():
    bits = np.arange(65536, dtype=np.uint16)
    ref = bits.view(np.float16).astype(np.float32)
    got = np.array([oracle.half_to_float(int(b)) for b in bits], dtype=np.float32)
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), ref[~nan].view(np.uint32))


def test_half_round_trip_is_identity_for_all_patterns():
    for b in range(65536):
        e, m = (b >> 10) & 31, b & 1023
        if e == 31 and m:  # NaN payloads are not preserved
            continue
        assert oracle.float_to_half_bits(oracle.half_to_float(b)) == b


def test_double_to_half_ties_between_adjacent_halves():
    # midpoint of two adjacent finite halves rounds to the one with an even last bit
    for b in list(range(0, 0x7BFF, 37)) + [0, 1, 0x3FF, 0x400, 0x7BFE]:
        lo = float(np.uint16(b).view(np.float16))
        hi = float(np.uint16(b + 1).view(np.float16))
        mid = (lo + hi) / 2  # exact in binary64
        want = b if b % 2 == 0 else b + 1
        assert oracle.double_to_half_bits(mid) == want
        assert oracle.double_to_half_bits(-mid) == (want | 0x8000)
        assert oracle.double_to_half_bits(np.nextafter(mid, np.inf)) == b + 1
        assert oracle.double_to_half_bits(np.nextafter(mid, -np.inf)) == b


def test_double_to_half_overflow_and_random_against_numpy():
    assert oracle.double_to_half_bits(65504.0) == 0x7BFF
    assert oracle.double_to_half_bits(65519.99) == 0x7BFF
    assert oracle.double_to_half_bits(65520.0) == 0x7C00  # tie goes to even = infinity
    assert oracle.double_to_half_bits(-1e9) == 0xFC00
    assert oracle.double_to_half_bits(0.0) == 0 and oracle.double_to_half_bits(-0.0) == 0x8000
    rng = np.random.default_rng(1)
    vals = np.concatenate([rng.standard_normal(4000) * 10.0 ** rng.integers(-9, 5, 4000),
                           rng.uniform(-2 ** -14, 2 ** -14, 2000)])
    with np.errstate(over="ignore"):
        ref = vals.astype(np.float16).view(np.uint16)
    got = np.array([oracle.double_to_half_bits(v) for v in vals], dtype=np.uint16)
    assert np.array_equal(got, ref)


# ------------------------------------------------------------------------ quantizers

def _golden_rows(bits):
    rows = []
    with open(os.path.join(GOLDEN, "quantizer_closed_form.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            n, x, c = line.split()
            if int(n) == bits:
                rows.append((float(x), int(c)))
    return rows


@pytest.mark.parametrize("e", [0, -3, 4])
def test_quantize_act_closed_form_power_of_two_scale(e):
    rows = _golden_rows(8)
    x = np.array([[v for v, _ in rows]], dtype=np.float64) * 2.0 ** e
    x16 = x.astype(np.float16)
    assert np.array_equal(x16.astype(np.float64), x)  # the fixture is FP16-exact
    q, s = oracle.quantize_act(x16)
    assert s[0] == np.float32(2.0 ** e)
    assert q[0].tolist() == [c for _, c in rows]


@pytest.mark.parametrize("e", [0, -5, 2])
def test_pack_w8_and_w4_closed_form_power_of_two_scale(e):
    rows = _golden_rows(8)
    w = (np.array([[v for v, _ in rows]]) * 2.0 ** e).astype(np.float16)
    wq, s = oracle.pack_w8(w)
    assert s[0] == np.float32(2.0 ** e) and wq[0].tolist() == [c for _, c in rows]
    rows4 = _golden_rows(4)
    vals = [v for v, _ in rows4]
    group = 32
    vals = vals + [0.0] * (group - len(vals))
    # second group: all zeros -> scale 0, codes 0
    w4 = (np.array([vals + [0.0] * group]) * 2.0 ** e).astype(np.float16)
    codes, sg = oracle.pack_w4(w4, group=group)
    assert sg.dtype == np.float16 and sg.shape == (1, 2)
    assert float(sg[0, 0]) == 2.0 ** e and float(sg[0, 1]) == 0.0
    assert codes[0, :len(rows4)].tolist() == [c for _, c in rows4]
    assert not codes[0, group:].any()


def _exact_code(x: float, a: float, bits: int) -> tuple[int, bool]:
    """Eq. 2 in exact rational arithmetic: clamp(rne((2^n-1) x / (2 a))); also says if it was a tie."""
    t = Fraction(x) * (2 ** bits - 1) / (2 * Fraction(a))
    fl = t.numerator // t.denominator
    frac = t - fl
    tie = frac == Fraction(1, 2)
    if frac > Fraction(1, 2) or (tie and fl % 2 == 1):
        r = fl + 1
    else:
        r = fl
    lo, hi = -(2 ** (bits - 1)), 2 ** (bits - 1) - 1
    return max(lo, min(hi, r)), tie


def test_quantize_act_agrees_with_exact_rational_rule_away_from_ties():
    rng = np.random.default_rng(7)
    x = (rng.standard_normal((24, 160)) * 10.0 ** rng.integers(-3, 3, (24, 1))).astype(np.float16)
    x[:, 5] *= 50
    # plant exact ties: x = a * (2j+1)/255 is rarely FP16-exact, so use x = -a (t = -127.5) and a/3-like values
    x[3, 7] = -np.abs(x[3]).max()
    q, s = oracle.quantize_act(x)
    n_tie = 0
    for m in range(x.shape[0]):
        a = float(np.abs(x[m]).max())
        assert s[m] == np.float32(a) / np.float32(127.5)
        for k in range(x.shape[1]):
            want, tie = _exact_code(float(x[m, k]), a, 8)
            if tie:
                n_tie += 1
                assert abs(int(q[m, k]) - want) <= 1
            else:
                assert int(q[m, k]) == want, (m, k, float(x[m, k]), a)
    assert n_tie >= 1


def test_pack_w8_agrees_with_exact_rational_rule_away_from_ties():
    rng = np.random.default_rng(8)
    w = (rng.standard_normal((12, 96)) * 0.02).astype(np.float16)
    wq, s = oracle.pack_w8(w)
    for n in range(w.shape[0]):
        a = float(np.abs(w[n]).max())
        for k in range(w.shape[1]):
            want, tie = _exact_code(float(w[n, k]), a, 8)
            # dividing by the binary32-rounded scale can move a value across a rounding
            # boundary only when it sits within 2^-22 (relative) of that boundary
            t = Fraction(float(w[n, k])) * 255 / (2 * Fraction(a))
            near = abs((t - Fraction(1, 2)) - round(t - Fraction(1, 2))) < Fraction(1, 2 ** 14)
            if not (tie or near):
                assert int(wq[n, k]) == want


def test_quantizer_invariants():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((32, 256)).astype(np.float16)
    x[:, [3, 77, 130, 200]] *= 50
    x[5] = 0  # all-zero row
    x[6, 10] = 0
    q, s = oracle.quantize_act(x)
    xf = x.astype(np.float64)
    # quantize -> dequantize error bound |x - q s| <= s/2 (small slack for the binary32 scale)
    err = np.abs(xf - q.astype(np.float64) * s[:, None].astype(np.float64))
    assert (err <= s[:, None] * (0.5 + 2.0 ** -14)).all()
    assert s[5] == 0 and not q[5].any()
    assert q[6, 10] == 0
    nz = [m for m in range(32) if m != 5]
    assert (np.abs(q[nz].astype(np.int32)).max(axis=1) >= 127).all()  # the range is used
    assert q.min() >= -128 and q.max() <= 127
    # codes are monotone in x within a row
    for m in nz[:8]:
        order = np.argsort(xf[m], kind="stable")
        assert (np.diff(q[m][order].astype(np.int32)) >= 0).all()
    # scaling a row by a power of two scales s and leaves the codes unchanged
    q2, s2 = oracle.quantize_act((xf * 0.25).astype(np.float16))
    assert np.array_equal(q2, q) and np.array_equal(s2, s * np.float32(0.25))
    # symmetric: negating the input negates the codes except where the clamp acts
    qn, sn = oracle.quantize_act((-xf).astype(np.float16))
    assert np.array_equal(sn, s)
    inner = (np.abs(q.astype(np.int32)) < 127) & (np.abs(qn.astype(np.int32)) < 127)
    assert np.array_equal(qn[inner], -q[inner])
    # the row maximum maps to +127 (clamped from 127.5 -> 128) and its negative to -128
    m = 0
    k = int(np.argmax(np.abs(xf[m])))
    assert int(q[m, k]) == (127 if xf[m, k] > 0 else -128)
    assert int(qn[m, k]) == (-128 if xf[m, k] > 0 else 127)


def test_pack_w4_invariants_and_stored_scale():
    rng = np.random.default_rng(4)
    w = (rng.standard_normal((16, 512)) * 0.02).astype(np.float16)
    w[2, 128:256] = 0
    codes, sg = oracle.pack_w4(w, 128)
    assert codes.min() >= -8 and codes.max() <= 7
    assert sg.shape == (16, 4) and float(sg[2, 1]) == 0.0 and not codes[2, 128:256].any()
    wf = w.astype(np.float64).reshape(16, 4, 128)
    a = np.abs(wf).max(axis=2)
    want_s = (a.astype(np.float32) / np.float32(7.5)).astype(np.float16)
    assert np.array_equal(sg, want_s)
    sf = sg.astype(np.float64)[:, :, None]
    err = np.abs(wf - codes.reshape(16, 4, 128) * sf)
    # codes are chosen against the stored FP16 scale: half a step everywhere, except the
    # element clamped from +8 to +7, whose error is a - 7 s with a <= 7.5 s (1 + 2^-11)
    assert (err <= sf * (0.5 + 7.5 * 2.0 ** -11 + 1e-6)).all()
    # exact rational rule against the stored scale, away from ties
    for n in range(3):
        for k in range(512):
            s = float(sg[n, k // 128])
            if s == 0:
                continue
            t = Fraction(float(w[n, k])) / Fraction(s)
            dist = abs((t - Fraction(1, 2)) - round(t - Fraction(1, 2)))
            if dist > Fraction(1, 2 ** 16):
                assert int(codes[n, k]) == max(-8, min(7, round(t)))


def test_nibble_pack_round_trips_all_byte_values():
    allb = np.arange(256, dtype=np.uint8).reshape(2, 128)
    codes = oracle.nibble_unpack(allb)
    assert codes.min() == -8 and codes.max() == 7
    # byte j holds k = 2j in its low nibble and k = 2j+1 in its high nibble, two's complement
    for j, b in enumerate(allb[0][:40]):
        lo, hi = int(b) & 15, int(b) >> 4
        assert codes[0, 2 * j] == (lo - 16 if lo >= 8 else lo)
        assert codes[0, 2 * j + 1] == (hi - 16 if hi >= 8 else hi)
    assert np.array_equal(oracle.nibble_pack(codes), allb)


# ----------------------------------------------------------------------------- GEMMs

def _ones(n):
    return np.ones((n,), np.float32)


def test_gemm_w8a8_brute_force_tiny_with_extremes():
    rng = np.random.default_rng(11)
    M, N, K = 5, 7, 9
    q = rng.integers(-128, 128, (M, K)).astype(np.int8)
    wq = rng.integers(-128, 128, (N, K)).astype(np.int8)
    q[0, :] = -128
    wq[0, :] = -128
    q[1, :] = 127
    wq[1, :] = -128
    acc, _ = oracle.gemm_w8a8(q, _ones(M), wq, _ones(N), want_y=False)
    for m in range(M):
        for n in range(N):
            want = sum(int(q[m, k]) * int(wq[n, k]) for k in range(K))
            assert int(acc[m, n]) == want
    assert int(acc[0, 0]) == K * 16384 and int(acc[1, 0]) == -K * 127 * 128


def test_gemm_w8a8_matches_numpy_int64_product_and_is_not_transposed():
    rng = np.random.default_rng(12)
    M, N, K = 33, 40, 300
    q = rng.integers(-128, 128, (M, K)).astype(np.int8)
    wq = rng.integers(-128, 128, (N, K)).astype(np.int8)
    acc, _ = oracle.gemm_w8a8(q, _ones(M), wq, _ones(N), want_y=False)
    assert np.array_equal(acc.astype(np.int64), q.astype(np.int64) @ wq.astype(np.int64).T)


def test_gemm_w8a8_identity_and_one_hot_weights():
    rng = np.random.default_rng(13)
    K = 64
    x = rng.standard_normal((8, K)).astype(np.float16)
    q, s_tok = oracle.quantize_act(x)
    eye = (np.eye(K) * 0.75).astype(np.float16)
    wq, s_ch = oracle.pack_w8(eye)           # +a -> 127.5 -> 128 -> clamped to 127
    assert np.array_equal(wq, (np.eye(K) * 127).astype(np.int8))
    acc, _ = oracle.gemm_w8a8(q, s_tok, wq, s_ch, want_y=False)
    assert np.array_equal(acc, 127 * q.astype(np.int32))
    wqn, _ = oracle.pack_w8((-eye).astype(np.float16))  # -a -> -127.5 -> -128 (tie to even)
    assert np.array_equal(wqn, (np.eye(K) * -128).astype(np.int8))
    accn, _ = oracle.gemm_w8a8(q, s_tok, wqn, s_ch, want_y=False)
    assert np.array_equal(accn, -128 * q.astype(np.int32))
    onehot = np.zeros((3, K), np.int8)
    onehot[0, 5], onehot[1, 63], onehot[2, 0] = 9, -128, 1
    acc1, _ = oracle.gemm_w8a8(q, s_tok, onehot, _ones(3), want_y=False)
    assert np.array_equal(acc1[:, 0], 9 * q[:, 5].astype(np.int32))
    assert np.array_equal(acc1[:, 1], -128 * q[:, 63].astype(np.int32))
    assert np.array_equal(acc1[:, 2], q[:, 0].astype(np.int32))


def test_int32_no_overflow_bound():
    # K * 128 * 128 < 2^31  <=>  K < 131072; the largest K of the workloads is 11008
    K = 11008
    q = np.full((1, K), -128, np.int8)
    w = np.full((1, K), -128, np.int8)
    acc, _ = oracle.gemm_w8a8(q, _ones(1), w, _ones(1), want_y=False)
    assert int(acc[0, 0]) == K * 16384 < 2 ** 31
    assert K * 127 * 127 < 2 ** 31
    K = 131072
    q = np.full((1, K), -128, np.int8)
    w = np.full((1, K), -128, np.int8)
    with pytest.raises(OverflowError):
        oracle.gemm_w8a8(q, _ones(1), w, _ones(1))
    w[0, 0] = 127  # one step inside the range again
    acc, _ = oracle.gemm_w8a8(q, _ones(1), w, _ones(1), want_y=False)
    assert int(acc[0, 0]) == (K - 1) * 16384 - 128 * 127


def test_dequant_power_of_two_scales_is_exact():
    rng = np.random.default_rng(14)
    M, N, K = 6, 10, 16
    q = rng.integers(-20, 21, (M, K)).astype(np.int8)
    wq = rng.integers(-20, 21, (N, K)).astype(np.int8)
    s_tok = (2.0 ** rng.integers(-6, 1, M)).astype(np.float32)
    s_ch = (2.0 ** rng.integers(-6, 1, N)).astype(np.float32)
    acc, y = oracle.gemm_w8a8(q, s_tok, wq, s_ch)
    # |acc| <= 6400 needs 13 bits > FP16's 11, so compare with numpy's own double -> half rounding
    want = (acc.astype(np.float64) * s_tok[:, None].astype(np.float64) * s_ch[None, :].astype(np.float64))
    assert np.array_equal(y.view(np.uint16), want.astype(np.float16).view(np.uint16))
    small = np.abs(acc) <= 2048
    assert small.any() and np.array_equal(y[small].astype(np.float64), want[small])  # exact there
    # zero scale gives an exact +0
    s_tok[0] = 0
    _, y0 = oracle.gemm_w8a8(q, s_tok, wq, s_ch)
    assert (y0[0].view(np.uint16) & 0x7FFF == 0).all()


def test_gemm_w4a8_group_accumulators_and_reduction_to_w8a8():
    rng = np.random.default_rng(15)
    M, N, K, G = 9, 12, 512, 4
    q = rng.integers(-128, 128, (M, K)).astype(np.int8)
    codes = rng.integers(-8, 8, (N, K)).astype(np.int8)
    codes[3, 128:256] = 0  # an all-zero group contributes exactly 0
    s_tok = (2.0 ** rng.integers(-4, 1, M)).astype(np.float32)
    sg_equal = np.full((N, G), 0.125, np.float16)
    acc_g, y = oracle.gemm_w4a8(q, s_tok, codes, sg_equal, 128)
    q64, c64 = q.astype(np.int64), codes.astype(np.int64)
    for g in range(G):
        sl = slice(128 * g, 128 * (g + 1))
        assert np.array_equal(acc_g[:, :, g].astype(np.int64), q64[:, sl] @ c64[:, sl].T)
    assert not acc_g[:, 3, 1].any()
    full = q64 @ c64.T
    assert np.array_equal(acc_g.astype(np.int64).sum(axis=2), full)
    # with all group scales equal to one power of two it reduces to the per-channel formula
    _, y8 = oracle.gemm_w8a8(q, s_tok, codes, np.full((N,), 0.125, np.float32))
    assert np.array_equal(y.view(np.uint16), y8.view(np.uint16))
    # distinct group scales: compare with the definition written out in numpy binary64
    sg = (rng.uniform(0.5, 2.0, (N, G)) * 2.0 ** -8).astype(np.float16)
    acc_g2, y2 = oracle.gemm_w4a8(q, s_tok, codes, sg, 128)
    R = (acc_g2.astype(np.float64) * sg.astype(np.float64)[None]).sum(axis=2)
    want = (R * s_tok[:, None].astype(np.float64)).astype(np.float16)
    diff = np.abs(y2.astype(np.float64) - want.astype(np.float64))
    assert (diff <= 2.0 ** -10 * np.abs(want.astype(np.float64))).all()  # summation order only
    # extremes: -128 x -8 over one group
    qe = np.full((1, 128), -128, np.int8)
    ce = np.full((1, 128), -8, np.int8)
    ae, _ = oracle.gemm_w4a8(qe, _ones(1), ce, np.ones((1, 1), np.float16), 128, want_y=False)
    assert int(ae[0, 0, 0]) == 128 * 128 * 8 == 2 ** 17


def test_end_to_end_error_is_consistent_with_half_step_noise():
    from paper_2512_23367_b200 import synth
    x = synth.activations(64, 1024, seed=5)
    w = synth.weights(96, 1024, seed=5)
    q, s_tok = oracle.quantize_act(x)
    exact = x.astype(np.float64) @ w.astype(np.float64).T
    wq, s_ch = oracle.pack_w8(w)
    _, y8 = oracle.gemm_w8a8(q, s_tok, wq, s_ch)
    rel8 = np.linalg.norm(y8.astype(np.float64) - exact) / np.linalg.norm(exact)
    codes, sg = oracle.pack_w4(w, 128)
    _, y4 = oracle.gemm_w4a8(q, s_tok, codes, sg, 128)
    rel4 = np.linalg.norm(y4.astype(np.float64) - exact) / np.linalg.norm(exact)
    # activation half-step noise against outlier-dominated signal gives a few percent for W8A8;
    # 4-bit weights add roughly (1/sqrt(12)) * s/sigma ~ 10 %.
    assert rel8 < 0.10 and rel8 < rel4 < 0.25


# ---------------------------------------------------------------------------- Eq. 3 (SmoothQuant variant)

def test_smooth_scales_closed_forms_alpha_one_half():
    # s_j = sqrt(max|X_j|) / sqrt(max|W_j|): perfect squares give exact values
    xa = np.array([16.0, 4.0, 9.0, 1.0, 0.25, 0.0, 3.0], np.float32)
    wa = np.array([4.0, 4.0, 1.0, 4.0, 4.0, 2.0, 0.0], np.float32)
    s, s_inv = oracle.smooth_scales(xa, wa)
    assert s.tolist() == [2.0, 1.0, 3.0, 0.5, 0.25, 1.0, 1.0]       # dead channels (a zero maximum) keep s = 1
    assert s_inv.tolist() == [0.5, 1.0, np.float32(1.0) / np.float32(3.0), 2.0, 4.0, 1.0, 1.0]
    # the balance Eq. 3 is built for: after smoothing both sides have the same column maximum sqrt(ax * aw)
    rng = np.random.default_rng(3)
    xa = rng.uniform(0.1, 60.0, 512).astype(np.float32)
    wa = rng.uniform(0.01, 0.2, 512).astype(np.float32)
    s, s_inv = oracle.smooth_scales(xa, wa)
    geo = np.sqrt(xa.astype(np.float64) * wa.astype(np.float64))
    assert np.allclose(xa * s_inv, geo, rtol=1e-6) and np.allclose(wa * s, geo, rtol=1e-6)


def test_col_absmax_is_the_column_maximum():
    rng = np.random.default_rng(4)
    a = (rng.standard_normal((37, 200)) * 3).astype(np.float16)
    a[5, 7] = -1000.0
    got = oracle.col_absmax(a)
    assert np.array_equal(got, np.abs(a.astype(np.float32)).max(axis=0))
    assert got[7] == 1000.0


def test_unit_factors_change_nothing():
    from paper_2512_23367_b200 import synth
    x, w = synth.activations(9, 256, seed=11), synth.weights(24, 256, seed=11)
    one = np.ones(256, np.float32)
    for plain, smooth in ((oracle.quantize_act(x), oracle.quantize_act(x, one)),
                          (oracle.pack_w8(w), oracle.pack_w8(w, one)),
                          (oracle.pack_w4(w, 128), oracle.pack_w4(w, 128, one))):
        assert np.array_equal(plain[0], smooth[0])
        assert np.array_equal(plain[1].view(np.uint8), smooth[1].view(np.uint8))


def test_power_of_two_factors_reduce_to_the_plain_quantizers():
    """With s_k = 2^e_k the smoothed values are exactly representable in FP16, so quantizing X S^-1
    (or S W) must equal the already pinned plain quantizer applied to the pre-multiplied matrix; a
    factor applied to the wrong axis, inverted, or applied after the maximum fails this."""
    rng = np.random.default_rng(5)
    K = 256
    e = rng.integers(-3, 4, K)
    f = (2.0 ** e).astype(np.float32)
    x = rng.integers(-200, 201, (7, K)).astype(np.float16)          # small integers: products stay exact in FP16
    w = (rng.integers(-60, 61, (12, K)) * 2.0 ** -6).astype(np.float16)
    for got, want in ((oracle.quantize_act(x, f), oracle.quantize_act((x.astype(np.float32) * f).astype(np.float16))),
                      (oracle.pack_w8(w, f), oracle.pack_w8((w.astype(np.float32) * f).astype(np.float16))),
                      (oracle.pack_w4(w, 128, f), oracle.pack_w4((w.astype(np.float32) * f).astype(np.float16), 128))):
        assert np.array_equal(got[0], want[0])
        assert np.array_equal(got[1].view(np.uint8), want[1].view(np.uint8))
    # and the factors really matter here (the test would be vacuous otherwise)
    assert not np.array_equal(oracle.quantize_act(x, f)[0], oracle.quantize_act(x)[0])


def test_smoothed_codes_obey_the_half_step_bound_in_binary32():
    from paper_2512_23367_b200 import synth
    x = synth.activations(16, 512, seed=12)
    s_inv = np.random.default_rng(6).uniform(0.02, 3.0, 512).astype(np.float32)
    q, s_tok = oracle.quantize_act(x, s_inv)
    t = x.astype(np.float32) * s_inv                                   # one binary32 product per element
    err = np.abs(t.astype(np.float64) - q.astype(np.float64) * s_tok[:, None].astype(np.float64))
    assert (err <= s_tok[:, None].astype(np.float64) * (0.5 + 2.0 ** -14)).all()
    assert (np.abs(q.astype(np.int16)).max(axis=1) >= 127).all()       # the row maximum maps to the end of the range
    assert np.array_equal(s_tok, np.abs(t).max(axis=1) / np.float32(127.5))


def test_eq3_equivalence_and_smoothing_helps_on_outlier_channels():
    """Y = (X S^-1)(S W) equals X W exactly in real arithmetic; after quantization the smoothed W4A8
    product must be CLOSER to X W than the plain one when a few activation channels are outliers
    (what Eq. 3 is for).  A factor on the wrong side (X S, S^-1 W) would blow the error up instead."""
    from paper_2512_23367_b200 import synth
    M, K, N = 64, 1024, 96
    x, w = synth.activations(M, K, seed=13), synth.weights(N, K, seed=13)
    exact = x.astype(np.float64) @ w.astype(np.float64).T
    s, s_inv = oracle.smooth_scales(oracle.col_absmax(x), oracle.col_absmax(w))
    xs, ws = x.astype(np.float64) * s_inv, w.astype(np.float64) * s
    assert np.allclose(xs @ ws.T, exact, rtol=0, atol=1e-4 * np.abs(exact).max())   # binary32 factors: s * s_inv ~ 1

    def rel(q, s_tok, codes, sg):
        _, y = oracle.gemm_w4a8(q, s_tok, codes, sg, 128, want_acc=False)
        return np.linalg.norm(y.astype(np.float64) - exact) / np.linalg.norm(exact)

    plain = rel(*oracle.quantize_act(x), *oracle.pack_w4(w, 128))
    smooth = rel(*oracle.quantize_act(x, s_inv), *oracle.pack_w4(w, 128, s))
    swapped = rel(*oracle.quantize_act(x, s), *oracle.pack_w4(w, 128, s_inv))
    assert smooth < 0.8 * plain
    assert swapped > plain


# ---------------------------------------------------------------------------- Eq. 4 (Hadamard variant)

def test_hadamard_block_order():
    # a power of two: the row's own order; otherwise the largest power of two dividing K, at most 256
    assert [oracle.hadamard_block(K) for K in (16, 48, 208, 256, 512, 2048, 4096, 16384, 6144, 11008, 768, 32768)] == \
        [16, 16, 16, 256, 512, 2048, 4096, 16384, 256, 256, 256, 256]


def test_rotation_of_unit_rows_is_the_library_hadamard_matrix():
    """Row e_k times H is row k of H: compare the whole matrix with scipy's Sylvester construction."""
    from scipy.linalg import hadamard
    for K, B in ((16, 16), (64, 64), (256, 256), (48, 16), (768, 256), (512, 512), (1024, 1024)):
        eye = np.eye(K, dtype=np.float16)
        H = oracle.rotate_rows(eye).astype(np.float64)
        want = np.kron(np.eye(K // B), hadamard(B).astype(np.float64) / np.sqrt(B))
        assert np.allclose(H, want, rtol=0, atol=1e-7)
        assert np.allclose(H @ H.T, np.eye(K), atol=1e-6)                 # orthogonal
        if B in (16, 64, 256, 1024):                                     # 1/sqrt(B) is a power of two: exact
            assert np.array_equal(H, want)


def test_rotation_matches_the_dense_product_and_preserves_norms():
    from scipy.linalg import hadamard
    rng = np.random.default_rng(21)
    a = (rng.standard_normal((5, 768)) * 4).astype(np.float16)
    got = oracle.rotate_rows(a).astype(np.float64)
    H = np.kron(np.eye(3), hadamard(256) / 16.0)
    want = a.astype(np.float64) @ H
    assert np.allclose(got, want, rtol=0, atol=2e-5 * np.abs(want).max())
    assert np.allclose(np.linalg.norm(got, axis=1), np.linalg.norm(a.astype(np.float64), axis=1), rtol=1e-6)
    # a lone spike of height A in a block becomes +-A/16 across that block (exactly), nothing elsewhere
    spike = np.zeros((1, 768), np.float16)
    spike[0, 300] = 48.0
    r = oracle.rotate_rows(spike)
    assert (np.abs(r[0, 256:512]) == 3.0).all() and (r[0, :256] == 0).all() and (r[0, 512:] == 0).all()
    # a row whose length is a power of two is rotated as a whole: the spike spreads over all of it
    spike = np.zeros((1, 1024), np.float16)
    spike[0, 300] = 48.0
    assert (np.abs(oracle.rotate_rows(spike)) == 1.5).all()


def test_hadamard_quantizers_are_the_plain_rule_on_the_rotated_values():
    """Integer-valued rows keep the rotation exact in binary32 (and, scaled by 16, representable in
    FP16), so quantizing X H must equal the pinned plain quantizer applied to the rotated matrix."""
    from scipy.linalg import hadamard
    rng = np.random.default_rng(22)
    K = 768
    H = np.kron(np.eye(3), hadamard(256))
    x = rng.integers(-3, 4, (6, K)).astype(np.float16) * 16                 # x H / 16 is an integer below 2048
    xr = (x.astype(np.float64) @ H / 16.0)
    assert np.array_equal(xr, np.round(xr)) and np.abs(xr).max() < 2048
    q, s = oracle.quantize_act_hadamard(x)
    q2, s2 = oracle.quantize_act(xr.astype(np.float16))
    assert np.array_equal(q, q2) and np.array_equal(s, s2)
    w = rng.integers(-2, 3, (10, K)).astype(np.float16) * 16
    wr = (w.astype(np.float64) @ H / 16.0).astype(np.float16)
    for got, want in ((oracle.pack_w8_hadamard(w), oracle.pack_w8(wr)),
                      (oracle.pack_w4_hadamard(w, 128), oracle.pack_w4(wr, 128))):
        assert np.array_equal(got[0], want[0])
        assert np.array_equal(got[1].view(np.uint8), want[1].view(np.uint8))


def test_eq4_equivalence_and_rotation_helps_on_outlier_channels():
    from paper_2512_23367_b200 import synth
    M, K, N = 64, 1024, 96
    x, w = synth.activations(M, K, seed=23), synth.weights(N, K, seed=23)
    exact = x.astype(np.float64) @ w.astype(np.float64).T
    xr, wr = oracle.rotate_rows(x).astype(np.float64), oracle.rotate_rows(w).astype(np.float64)
    assert np.allclose(xr @ wr.T, exact, rtol=0, atol=1e-5 * np.abs(exact).max())    # (X H)(W H)^T = X W^T

    def rel8(q, s_tok, wq, s_ch):
        _, y = oracle.gemm_w8a8(q, s_tok, wq, s_ch, want_acc=False)
        return np.linalg.norm(y.astype(np.float64) - exact) / np.linalg.norm(exact)

    def rel4(q, s_tok, codes, sg):
        _, y = oracle.gemm_w4a8(q, s_tok, codes, sg, 128, want_acc=False)
        return np.linalg.norm(y.astype(np.float64) - exact) / np.linalg.norm(exact)

    # INT8 x INT8: the error is the activations' (outlier channels set the token scale); spreading every
    # outlier over its block of 256 removes most of it
    plain8 = rel8(*oracle.quantize_act(x), *oracle.pack_w8(w))
    rotated8 = rel8(*oracle.quantize_act_hadamard(x), *oracle.pack_w8_hadamard(w))
    assert rotated8 < 0.5 * plain8
    # INT4 weights: Gaussian weights gain nothing from the rotation, so the total only improves a little
    assert rel4(*oracle.quantize_act_hadamard(x), *oracle.pack_w4_hadamard(w, 128)) < \
        rel4(*oracle.quantize_act(x), *oracle.pack_w4(w, 128))
    # rotating only one operand destroys the product
    assert rel8(*oracle.quantize_act_hadamard(x), *oracle.pack_w8(w)) > 0.5


# ---------------------------------------------------------------------------- static (calibrated) activation scale

def test_static_scale_closed_forms_and_saturation():
    # s = 2^-2: codes are rne(4 x); ties to even; beyond +-127/4 the codes saturate
    x = np.array([[0.0, 0.125, 0.375, 0.625, -0.125, -0.375, 1.0, -1.0, 31.75, 31.875, 40.0, -32.0, -32.125, -100.0]],
                 np.float16)
    q, s_tok = oracle.quantize_act_static(x, 0.25)
    assert q[0].tolist() == [0, 0, 2, 2, 0, -2, 4, -4, 127, 127, 127, -128, -128, -128]
    assert s_tok.tolist() == [0.25]
    # a scale that is not positive: nothing can be represented
    q0, s0 = oracle.quantize_act_static(x, 0.0)
    assert (q0 == 0).all() and s0[0] == 0.0


def test_static_scale_error_bound_inside_the_calibrated_range():
    from paper_2512_23367_b200 import synth
    x = synth.activations(8, 512, seed=31)
    s = np.float32(np.abs(x.astype(np.float32)).max() / 127.5)       # calibrated on the data itself: nothing saturates low
    q, s_tok = oracle.quantize_act_static(x, s)
    assert (s_tok == s).all()
    err = np.abs(x.astype(np.float64) - q.astype(np.float64) * float(s))
    inside = np.abs(x.astype(np.float64)) <= 127.0 * float(s)
    assert (err[inside] <= float(s) * (0.5 + 2.0 ** -12)).all()
    # one scale for all tokens: rows without an outlier lose resolution against the per-token rule of Eq. 2
    qd, sd = oracle.quantize_act(x)
    assert (sd <= s * (1 + 1e-6)).all()


# ---------------------------------------------------------------------------- SwiGLU + per-token quantization

def _silu64(g):
    g = g.astype(np.float64)
    with np.errstate(over="ignore"):
        return g / (1.0 + np.exp(-g))


def test_swiglu_follows_the_definition_on_every_fp16_gate():
    """h = silu(gate) * up with silu(g) = g / (1 + e^-g): the fixed binary32 sequence (which multiplies by the
    rounded reciprocal of 1 + e^-g: two roundings where a quotient has one) stays within 2.5 ulp of
    the definition evaluated in binary64 for every finite FP16 gate value (up = 1), is exactly 0 at 0, equals
    g once e^-g no longer registers beside 1, and vanishes for large negative g."""
    g = np.arange(65536, dtype=np.uint16).view(np.float16)
    g = g[np.isfinite(g)].reshape(1, -1)
    _, _, h = oracle.swiglu_quantize(g, np.ones_like(g), want_h=True)
    true = _silu64(g)
    ulp = np.spacing(np.abs(true).astype(np.float32)).astype(np.float64)
    normal = np.abs(true) > 1e-30
    assert (np.abs(h - true)[normal] <= 2.5 * ulp[normal]).all()
    assert (np.abs(h - true)[~normal] <= 1e-33).all()
    gf = g.astype(np.float32)
    assert (h[gf == 0] == 0).all()
    assert np.array_equal(h[gf >= 17], gf[gf >= 17])              # e^-17 < 2^-24: 1 + e^-g rounds to 1
    assert (np.abs(h[gf <= -104]) <= 1e-33).all()
    # negative side: the minimum of silu is about -0.2785 near g = -1.2785
    assert abs(float(h.min()) + 0.27846) < 1e-4


def test_swiglu_is_gated_by_the_first_operand_and_scaled_by_the_second():
    g = np.array([[1.0, -1.0, 2.0, 0.5]], np.float16)
    u = np.array([[3.0, 3.0, -0.5, 0.0]], np.float16)
    _, _, h = oracle.swiglu_quantize(g, u, want_h=True)
    want = _silu64(g) * u.astype(np.float64)
    assert np.allclose(h, want, rtol=3e-7, atol=0)
    _, _, h_swapped = oracle.swiglu_quantize(u, g, want_h=True)
    assert not np.allclose(h_swapped, want, rtol=1e-3)             # silu(u) * g is a different function


def test_swiglu_quantize_reduces_to_the_pinned_quantizer_when_the_gate_factor_is_a_power_of_two():
    """With gate = 32 everywhere, silu(32) = 32 exactly, so h = 32 * up exactly (a power of two): the codes
    must be those of the pinned per-token quantizer on `up` and the scales 32 times its scales."""
    from paper_2512_23367_b200 import synth
    up = synth.activations(24, 640, seed=71)
    up[3] = 0                                                       # a zero row stays a zero row
    gate = np.full_like(up, 32.0)
    q, s = oracle.swiglu_quantize(gate, up)
    q_ref, s_ref = oracle.quantize_act(up)
    assert np.array_equal(q, q_ref)
    assert np.array_equal(s, 32.0 * s_ref)
    assert s[3] == 0 and (q[3] == 0).all()
    # gate = 0 closes every channel: the whole row is zero
    q0, s0 = oracle.swiglu_quantize(np.zeros_like(up), up)
    assert (q0 == 0).all() and (s0 == 0).all()
    # the operands are not interchangeable: gating by `up` and scaling by 32 gives other codes
    q_sw, _ = oracle.swiglu_quantize(up, gate)
    assert not np.array_equal(q_sw, q_ref)


def test_swiglu_quantize_closed_form_codes():
    # gate = 64 (silu = 64 exactly), up = multiples of 1/128 with maximum 127.5/128: h = up * 64, scale 0.5 * 64 / 64...
    up = np.array([[127.5 / 128, 0.5 / 128, 1.5 / 128, 2.5 / 128, -0.5 / 128, -1.5 / 128, -127.5 / 128, 64.0 / 128]], np.float16)
    gate = np.full_like(up, 64.0)
    q, s = oracle.swiglu_quantize(gate, up)
    # a = 127.5/128 * 64 = 63.75, s = a / 127.5 = 0.5, codes = rne(h / 0.5) = rne(up * 128): ties to even, +max clamps to 127
    assert s.tolist() == [0.5]
    assert q[0].tolist() == [127, 0, 2, 2, 0, -2, -128, 64]


def test_swiglu_quantize_half_step_bound_against_the_definition():
    from paper_2512_23367_b200 import synth
    rng = np.random.default_rng(5)
    gate = (rng.standard_normal((16, 1024)) * 3).astype(np.float16)
    up = synth.activations(16, 1024, seed=72)
    q, s, h = oracle.swiglu_quantize(gate, up, want_h=True)
    true = _silu64(gate) * up.astype(np.float64)
    assert np.allclose(h, true, rtol=4e-7, atol=1e-30)
    err = np.abs(true - q.astype(np.float64) * s.astype(np.float64)[:, None])
    assert (err <= s.astype(np.float64)[:, None] * (0.5 + 1e-4)).all()
    assert (np.abs(q.astype(np.int32)).max(axis=1) >= 127).all()    # every row uses the full range
    assert np.array_equal(s, (np.abs(h).max(axis=1) / np.float32(127.5)).astype(np.float32))


# ---------------------------------------------------------------------------- static scale per feature channel

def test_static_channel_scales_reduce_to_the_per_tensor_rule_and_follow_closed_forms():
    from paper_2512_23367_b200 import synth
    x = synth.activations(6, 256, seed=33)
    # the same power-of-two scale in every channel: exactly the per-tensor static quantizer
    q, s_tok = oracle.quantize_act_static_channel(x, np.full((256,), 8.0, np.float32))
    q_ref, _ = oracle.quantize_act_static(x, 0.125)
    assert np.array_equal(q, q_ref) and (s_tok == 1.0).all()
    # channel k has its own scale: closed forms with ties and saturation
    xs = np.array([[0.5, 0.5, 2.5, -2.5, 100.0, -100.0, 1.0, 1.0]], np.float16)
    inv = np.array([1.0, 3.0, 1.0, 1.0, 2.0, 2.0, 0.0, -1.0], np.float32)
    q2, _ = oracle.quantize_act_static_channel(np.tile(xs, (1, 2)), np.tile(inv, 2))
    assert q2[0, :8].tolist() == [0, 2, 2, -2, 127, -128, 0, 0]      # 0.5 -> 0 (tie to even), 1.5 -> 2, 2.5 -> 2, saturation, dead channels
    # the scale really is applied per COLUMN: scaling the factor of one channel changes that channel's codes only
    inv2 = np.full((256,), 8.0, np.float32)
    inv2[7] = 16.0
    q3, _ = oracle.quantize_act_static_channel(x, inv2)
    assert np.array_equal(np.delete(q3, 7, axis=1), np.delete(q_ref, 7, axis=1)) and not np.array_equal(q3[:, 7], q_ref[:, 7])
    # folded into the weights, the product is that of the plain operands: x ~ q / inv_s, (q) . (w * s) ~ x . w
    w = synth.weights(8, 256, seed=34).astype(np.float64)
    a = np.abs(x.astype(np.float32)).max(axis=0)
    inv_s = (np.float32(127.0) / np.maximum(a, np.float32(1e-6))).astype(np.float32)
    q4, _ = oracle.quantize_act_static_channel(x, inv_s)
    approx = (q4.astype(np.float64) / inv_s.astype(np.float64)) @ w.T
    exact = x.astype(np.float64) @ w.T
    assert np.abs(approx - exact).max() <= 0.02 * np.abs(exact).max()


def test_full_order_hadamard_quantizers_are_the_plain_rule_on_the_rotated_values():
    """K a power of two: H is the Sylvester matrix of order K.  Integer rows scaled by sqrt(K) keep the
    rotation exact, so the quantizers of X H and W H must equal the pinned plain ones on X H_K / sqrt(K)."""
    from scipy.linalg import hadamard
    rng = np.random.default_rng(23)
    K = 1024
    H = hadamard(K).astype(np.float64)
    x = rng.integers(-2, 3, (5, K)).astype(np.float16) * 32                 # x H / 32 is an integer below 2048
    xr = x.astype(np.float64) @ H / 32.0
    assert np.array_equal(xr, np.round(xr)) and np.abs(xr).max() < 2048
    assert np.array_equal(oracle.rotate_rows(x).astype(np.float64), xr)
    q, s = oracle.quantize_act_hadamard(x)
    q2, s2 = oracle.quantize_act(xr.astype(np.float16))
    assert np.array_equal(q, q2) and np.array_equal(s, s2)
    w = rng.integers(-2, 3, (6, K)).astype(np.float16) * 32
    wr = (w.astype(np.float64) @ H / 32.0).astype(np.float16)
    for got, want in ((oracle.pack_w8_hadamard(w), oracle.pack_w8(wr)),
                      (oracle.pack_w4_hadamard(w, 128), oracle.pack_w4(wr, 128))):
        assert np.array_equal(got[0], want[0])
        assert np.array_equal(got[1].view(np.uint8), want[1].view(np.uint8))
    # (X H)(W H)^T = X W^T with the full matrix too
    xf, wf = oracle.rotate_rows(x).astype(np.float64), oracle.rotate_rows(w).astype(np.float64)
    assert np.allclose(xf @ wf.T, x.astype(np.float64) @ w.astype(np.float64).T, rtol=1e-9)


# ---------------------------------------------------------------------------- Eq. 3 with alpha a multiple of 1/4

def test_smooth_scales_for_quarter_alphas():
    """s_j = max|X_j|^alpha / max|W_j|^(1-alpha): closed forms on fourth powers, the alpha = 1/2 case is the
    pinned pqo_smooth_scales bit for bit, the extremes put all of the range on one side, and the binary64
    power agrees to rounding."""
    xa = np.array([16.0, 81.0, 256.0, 1.0, 0.0, 625.0], np.float32)
    wa = np.array([1.0, 16.0, 81.0, 16.0, 4.0, 0.0], np.float32)
    want = {0: [1 / 1.0, 1 / 16.0, 1 / 81.0, 1 / 16.0, 1, 1],          # 1 / max|W|
            1: [2 / 1.0, 3 / 8.0, 4 / 27.0, 1 / 8.0, 1, 1],            # x^(1/4) / w^(3/4)
            2: [4 / 1.0, 9 / 4.0, 16 / 9.0, 1 / 4.0, 1, 1],
            3: [8 / 1.0, 27 / 2.0, 64 / 3.0, 1 / 2.0, 1, 1],           # x^(3/4) / w^(1/4)
            4: [16.0, 81.0, 256.0, 1.0, 1, 1]}                          # max|X|
    for a, vals in want.items():
        s, s_inv = oracle.smooth_scales_alpha(xa, wa, a)
        assert np.array_equal(s, np.array(vals, np.float64).astype(np.float32)), a
        assert np.array_equal(s_inv, (np.float32(1.0) / s).astype(np.float32))
    rng = np.random.default_rng(9)
    xr = (rng.random(512) * 50 + 0.01).astype(np.float32)
    wr = (rng.random(512) * 0.3 + 0.001).astype(np.float32)
    s2, i2 = oracle.smooth_scales_alpha(xr, wr, 2)
    s_ref, i_ref = oracle.smooth_scales(xr, wr)
    assert np.array_equal(s2, s_ref) and np.array_equal(i2, i_ref)
    for a in range(5):
        s, _ = oracle.smooth_scales_alpha(xr, wr, a)
        true = xr.astype(np.float64) ** (a / 4) / wr.astype(np.float64) ** (1 - a / 4)
        assert np.allclose(s, true, rtol=4e-7)
    # what alpha does: the smoothed maxima are (x w)^(1-alpha) on the activation side and (x w)^alpha on the
    # weight side -- their product stays x w, and they meet at alpha = 1/2
    for a in range(5):
        s, _ = oracle.smooth_scales_alpha(xr, wr, a)
        xw = xr.astype(np.float64) * wr.astype(np.float64)
        assert np.allclose(xr / s, xw ** (1 - a / 4), rtol=1e-6) and np.allclose(wr * s, xw ** (a / 4), rtol=1e-6)
