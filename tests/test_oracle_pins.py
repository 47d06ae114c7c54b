"""CPU-only tests that pin the oracle to what the paper and the mathematics fix.

Each test names the passage it checks.  None of them re-types the oracle's own formula: they use
the paper's printed values (Table II, Theorem 1), invariants stated in the Appendix proof, closed
forms, special cases that reduce to a library routine, and brute-force search over the explicit
set of representable values with exact rational arithmetic.
"""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import oracle as orc
from paper_2302_08007_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
Cfg = orc.Config

GRID = [Cfg(k1, 8, k2, d2, m) for k1 in (1, 2, 4, 8, 16, 32, 64, 1024) for k2 in (1, 2, 4, 8)
        for d2 in (0, 1, 2, 3) for m in (1, 2, 4, 7, 8) if k2 <= k1]
SMALL_GRID = GRID[::7]


def _golden_rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]


# ---- Table II: bits per element -----------------------------------------------------------------
def test_table2_bits_per_element_formula_and_packed_bytes():
    for row in _golden_rows("table2_formats.txt"):
        name, k1, k2, d1, d2, m, bits = row.split()
        cfg = Cfg(int(k1), int(d1), int(k2), int(d2), int(m))
        assert orc.bits_per_element(cfg) == float(bits)
        # the packed planes spend exactly that many bits when the line needs no padding
        rows, cols = 3, 1024
        _, nbytes = orc.packed_sizes(cfg, rows, cols, axis=1)
        assert sum(nbytes) * 8 == int(bits) * rows * cols
        _, nbytes = orc.packed_sizes(cfg, cols, rows, axis=0)
        assert sum(nbytes) * 8 == int(bits) * rows * cols


def test_bits_per_element_general():
    # Section III: (m+1) + d1/k1 + d2/k2, e.g. MSFP16-like k1=16, d2=0, m=7 -> 8.5 bits
    assert orc.bits_per_element(Cfg(16, 8, 1, 0, 7)) == 8.5
    assert orc.bits_per_element(Cfg(8, 8, 8, 2, 3)) == 4 + 1 + 0.25


# ---- Theorem 1 -----------------------------------------------------------------------------------
def test_theorem1_closed_form_values():
    for row in _golden_rows("theorem1_bounds.txt"):
        name, m, bound = row.split()
        cfg = Cfg(16, 8, 2, 1, int(m))
        assert abs(orc.theorem1_bound_db(cfg, 1 << 20) - float(bound)) < 1e-3
    # N < k1 replaces k1 by N (end of the proof)
    assert orc.theorem1_bound_db(Cfg(16, 8, 2, 1, 4), 4) > orc.theorem1_bound_db(Cfg(16, 8, 2, 1, 4), 16)


def test_theorem1_holds_on_random_and_adversarial_inputs():
    rng = np.random.default_rng(5)
    inputs = [synth.normal(4096, 1), synth.laplace(4096, 2), synth.student_t(4096, 3),
              synth.normal_with_outliers(4096, 4, frac=0.01),
              (rng.standard_normal(4096) * np.exp2(rng.integers(-6, 6, 4096))).astype(np.float32)]
    for cfg in GRID:
        if cfg.m < 2:
            continue
        for x in inputs:
            assert orc.qsnr(cfg, x) >= orc.theorem1_bound_db(cfg, x.size) - 1e-9, cfg


def test_theorem1_worst_case_search_tiny_blocks():
    # every block from a grid of magnitudes in a few binades; k1=4, k2=2
    vals = np.array([0.0] + [m * 2.0 ** e for e in (-3, -2, -1, 0) for m in (1.0, 1.24, 1.26, 1.5, 1.74, 1.99)],
                    dtype=np.float32)
    blocks = np.array(list(itertools.product(vals, repeat=4)), dtype=np.float32)
    blocks = blocks[np.abs(blocks).max(axis=1) > 0]
    for d2 in (0, 1, 2):
        for m in (2, 3):
            cfg = Cfg(4, 8, 2, d2, m)
            y, _ = orc.quant_dequant(cfg, blocks)
            e2 = ((y.astype(np.float64) - blocks) ** 2).sum(axis=1)
            s2 = (blocks.astype(np.float64) ** 2).sum(axis=1)
            worst = (-10 * np.log10(np.maximum(e2, 1e-300) / s2)).min()
            assert worst >= orc.theorem1_bound_db(cfg, 4) - 1e-9


# ---- hand-worked blocks ---------------------------------------------------------------------------
def test_hand_worked_blocks():
    for row in _golden_rows("hand_blocks.txt"):
        rnd, xs, qs, F, taus, codes = [f.strip() for f in row.split("|")]
        cfg = Cfg(8, 8, 2, 1, 4, orc.POW2, int(rnd))
        x = np.array([float(v) for v in xs.split()], dtype=np.float32)
        want = np.array([float(v) for v in qs.split()], dtype=np.float32)
        y, _ = orc.quant_dequant(cfg, x)
        assert y.view(np.uint32).tolist() == want.view(np.uint32).tolist()
        Fo, tauo, codeo = orc.encode(cfg, x)
        assert Fo.ravel().tolist() == [int(F)]
        assert tauo.ravel().tolist() == [int(t) for t in taus.split()]
        assert codeo.ravel().tolist() == [int(c, 16) for c in codes.split()]


def test_hand_worked_packed_bytes():
    # 5-bit codes 08 16 05 04 02 11 0f 04, LSB first: bits written out by hand
    x = np.array([1.0, -0.75, 0.3, 0.26, 0.124, -0.06, 1.9, 0.49], dtype=np.float32)
    exps, micro, elems = orc.pack(Cfg(8, 8, 2, 1, 4), x)
    bits = "".join(format(c, "05b")[::-1] for c in (0x08, 0x16, 0x05, 0x04, 0x02, 0x11, 0x0F, 0x04))
    want = bytes(int(bits[i:i + 8][::-1], 2) for i in range(0, 40, 8))
    assert bytes(elems[0, :5]) == want == bytes.fromhex("c81622e223")
    assert exps[0, 0] == 127 and micro[0, 0] == 0b0110
    assert not elems[0, 5:].any() and not exps[0, 1:].any() and not micro[0, 1:].any()


# ---- Appendix invariants ---------------------------------------------------------------------------
def _fields(cfg, x):
    F, tau, code = orc.encode(cfg, x)
    y, _ = orc.quant_dequant(cfg, x)
    n = x.size
    nb = F.shape[1]
    q = (code & ((1 << cfg.m) - 1)).astype(np.int64).ravel()[:n]
    s = (code >> cfg.m).astype(np.int64).ravel()[:n]
    Fe = np.repeat(F.ravel().astype(np.int64), cfg.k1)[:n]
    te = np.repeat(tau.ravel().astype(np.int64), cfg.k2)[:n]
    return F, tau, q, s, Fe, te, y, nb


@pytest.mark.parametrize("cfg", SMALL_GRID, ids=str)
def test_representation_form_and_error_bounds(cfg):
    """Q(x) = +-q * 2^(E-tau-m+1) with integer q < 2^m; |Q(x)-x| <= 2^(E-tau-m) unless clamped."""
    for x in (synth.normal(2048, 7), synth.edge_case_values(2048, 8)):
        F, tau, q, s, Fe, te, y, nb = _fields(cfg, x)
        assert q.max() < (1 << cfg.m) and tau.max() <= (1 << cfg.d2) - 1
        p = Fe - 127 - te - (cfg.m - 1)
        recon = np.ldexp(q.astype(np.float64), p) * np.where(s == 1, -1.0, 1.0)
        assert np.array_equal(recon.astype(np.float32).view(np.uint32), y.view(np.uint32))
        assert np.array_equal(s, (x.view(np.uint32) >> 31).astype(np.int64))      # sign kept, also for zeros
        err = np.abs(y.astype(np.float64) - x.astype(np.float64))
        half = np.ldexp(1.0, p - 1)
        clamped = np.abs(x.astype(np.float64)) > np.ldexp(float((1 << cfg.m) - 1), p)
        assert (err[~clamped] <= half[~clamped]).all()
        assert (err[clamped] <= 2 * half[clamped]).all()
        assert (q[clamped] == (1 << cfg.m) - 1).all()


@pytest.mark.parametrize("cfg", SMALL_GRID, ids=str)
def test_shared_exponent_and_microexponent_structure(cfg):
    """E is the largest private exponent; the block's largest element sits in a sub-block with
    tau = 0; a sub-block with tau < beta holds an element whose private exponent is E - tau."""
    x = synth.edge_case_values(4096, 11)
    F, tau, q, s, Fe, te, y, nb = _fields(cfg, x)
    f = ((x.view(np.uint32) >> 23) & 0xFF).astype(np.int64)
    beta = (1 << cfg.d2) - 1
    fb = f.reshape(-1, cfg.k1)
    assert np.array_equal(F.ravel(), fb.max(axis=1))
    fs = f.reshape(-1, cfg.k2).max(axis=1)
    t = tau.ravel().astype(np.int64)
    Fs = np.repeat(F.ravel().astype(np.int64), cfg.k1 // cfg.k2)
    assert (t.reshape(-1, cfg.k1 // cfg.k2).min(axis=1) == 0).all()
    assert np.array_equal(fs[t < beta], (Fs - t)[t < beta])
    assert (fs[t == beta] <= (Fs - beta)[t == beta]).all()


@pytest.mark.parametrize("cfg", SMALL_GRID, ids=str)
def test_idempotence_values_and_bytes(cfg):
    for x in (synth.laplace(1536, 3), synth.edge_case_values(1536, 4)):
        y, _ = orc.quant_dequant(cfg, x)
        y2, (e2, _) = orc.quant_dequant(cfg, y)
        assert np.array_equal(y.view(np.uint32), y2.view(np.uint32)) and e2 == 0.0
        for a, b in zip(orc.pack(cfg, x), orc.pack(cfg, y)):
            assert np.array_equal(a, b)


def test_powers_of_two_inside_the_window_are_exact():
    for cfg in (orc.MX4, orc.MX6, orc.MX9, Cfg(32, 8, 4, 2, 3)):
        for E in (-126, -20, 0, 100):
            x = np.zeros(cfg.k1, dtype=np.float32)
            x[0] = np.ldexp(1.5, E)                       # pins the shared exponent, tau_0 = 0
            for t in range(E - cfg.m + 1, E + 1):
                x[1] = np.ldexp(1.0, t)                   # same sub-block (k2 >= 2) -> tau = 0
                y, _ = orc.quant_dequant(cfg, x)
                assert y[1] == x[1], (cfg, E, t)
            x[1] = np.ldexp(1.0, E - cfg.m - 1)           # below half a step: flushed to zero
            assert orc.quant_dequant(cfg, x)[0][1] == 0.0


@pytest.mark.parametrize("cfg", SMALL_GRID, ids=str)
def test_power_of_two_scale_equivariance(cfg):
    x = synth.student_t(2048, 9)
    y, (e2, s2) = orc.quant_dequant(cfg, x)
    for t in (-40, -3, 5, 60):
        yt, (e2t, s2t) = orc.quant_dequant(cfg, np.ldexp(x, t))
        assert np.array_equal(yt, np.ldexp(y, t))
        assert orc.qsnr_db(e2t, s2t) == pytest.approx(orc.qsnr_db(e2, s2), abs=1e-9)


def test_qsnr_monotone_in_m_and_six_db_per_bit():
    x = synth.normal(1 << 16, 0)
    for k1, k2, d2 in ((16, 2, 1), (16, 1, 0), (64, 8, 2), (8, 1, 1)):
        q = [orc.qsnr(Cfg(k1, 8, k2, d2, m), x) for m in range(1, 9)]
        assert all(b > a for a, b in zip(q, q[1:]))
        steps = np.diff(q[2:])
        assert np.all(np.abs(steps - 6.02) < 0.35), steps


def test_d2_zero_is_plain_block_floating_point():
    """d2 = 0 is conventional BFP: the result cannot depend on k2 and every element of a block
    shares one step."""
    x = synth.laplace(4096, 12)
    base, _ = orc.quant_dequant(Cfg(16, 8, 1, 0, 5), x)
    for k2 in (2, 4, 8, 16):
        y, _ = orc.quant_dequant(Cfg(16, 8, k2, 0, 5), x)
        assert np.array_equal(y.view(np.uint32), base.view(np.uint32))
    blk = base.reshape(-1, 16).astype(np.float64)
    E = np.floor(np.log2(np.abs(x.reshape(-1, 16)).max(axis=1)))
    ratio = blk / np.ldexp(1.0, (E - 4).astype(int))[:, None]
    assert np.array_equal(ratio, np.round(ratio))


def test_scalar_case_matches_bf16_rounding_except_binade_carries():
    """k1 = k2 = 1, d2 = 0, m = 8 is a scalar float with 8 significant bits, i.e. bf16 rounding
    (a library routine here: torch's cast), except that BDR never bumps the exponent."""
    import torch
    x = synth.normal(1 << 16, 21)
    y, _ = orc.quant_dequant(Cfg(1, 8, 1, 0, 8), x)
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    differs = y != ref
    assert 0 < differs.mean() < 0.01
    # where they differ, bf16 carried into the next binade and BDR clamped to the top code
    assert np.array_equal(np.abs(ref[differs]), np.exp2(np.floor(np.log2(np.abs(x[differs]))) + 1))
    assert np.array_equal(np.abs(y[differs]), np.abs(ref[differs]) * (1 - 2.0 ** -8))


# ---- brute force against the explicit value set -----------------------------------------------------
def _brute_block(cfg, xs):
    """Nearest representable value by exact rational search over the explicit code set."""
    def pexp(v):
        v = abs(Fraction(float(v)))
        if v < Fraction(1, 2 ** 126):
            return -127
        e = math.floor(math.log2(v))
        while Fraction(2) ** e > v:
            e -= 1
        while Fraction(2) ** (e + 1) <= v:
            e += 1
        return e
    E = max(pexp(v) for v in xs)
    beta = 2 ** cfg.d2 - 1
    out = []
    for j in range(0, len(xs), cfg.k2):
        sub = xs[j:j + cfg.k2]
        tau = min(E - max(pexp(v) for v in sub), beta)
        step = Fraction(2) ** (E - tau - cfg.m + 1)
        for v in sub:
            a = abs(Fraction(float(v)))
            best = min(range(2 ** cfg.m), key=lambda q: (abs(q * step - a), q % 2 if cfg.rounding == 0 else -q))
            out.append(float(best * step) * (-1.0 if math.copysign(1.0, float(v)) < 0 else 1.0))
    return out


@pytest.mark.parametrize("rounding", [orc.RNE, orc.RNA])
def test_brute_force_all_bf16_values_in_a_few_binades(rounding):
    # every bf16 value with exponent in [-3, 1] (plus zero), paired with fixed companions
    mags = [0.0] + [(1 + k / 128.0) * 2.0 ** e for e in range(-3, 2) for k in range(128)]
    comps = [0.0, 0.3, -1.0, 1.99, 0.06]
    for m, d2, k1, k2 in ((1, 1, 2, 1), (2, 1, 2, 2), (3, 0, 2, 1), (3, 2, 4, 2), (2, 1, 4, 1)):
        cfg = Cfg(k1, 8, k2, d2, m, orc.POW2, rounding)
        blocks = []
        for v in mags:
            for c in comps:
                blk = [v, c] + [0.25, -0.01][: k1 - 2]
                blocks.append(blk)
        x = np.array(blocks, dtype=np.float32)
        y, _ = orc.quant_dequant(cfg, x)
        ya, _ = orc.quant_dequant(cfg, x, alt=True)
        assert np.array_equal(y.view(np.uint32), ya.view(np.uint32))
        want = np.array([_brute_block(cfg, list(b)) for b in x], dtype=np.float32)
        assert np.array_equal(y.view(np.uint32), want.view(np.uint32)), cfg


def test_two_formulations_agree_everywhere():
    for cfg in GRID[::3]:
        for rounding in (orc.RNE, orc.RNA):
            c = Cfg(cfg.k1, 8, cfg.k2, cfg.d2, cfg.m, orc.POW2, rounding)
            for x in (synth.edge_case_values(2048, 31), synth.f32_to_bf16_bits(synth.normal(2048, 32))):
                if x.dtype == np.uint16:
                    x = synth.bf16_bits_to_f32(x)        # bf16-valued inputs: ties are common
                a, _ = orc.quant_dequant(c, x)
                b, _ = orc.quant_dequant(c, x, alt=True)
                assert np.array_equal(a.view(np.uint32), b.view(np.uint32)), c


# ---- layout, axes, tails ------------------------------------------------------------------------------
@pytest.mark.parametrize("cfg", [orc.MX4, orc.MX6, orc.MX9, Cfg(8, 8, 4, 2, 3), Cfg(32, 8, 1, 3, 6), Cfg(16, 8, 16, 0, 7)], ids=str)
def test_pack_unpack_round_trip(cfg):
    x = synth.edge_case_values(5 * 200, 40).reshape(5, 200)        # 200 is not a multiple of 16 or 32
    for axis in (0, 1):
        y, _ = orc.quant_dequant(cfg, x, axis=axis)
        planes = orc.pack(cfg, x, axis=axis)
        back = orc.unpack(cfg, planes, 5, 200, axis=axis)
        assert np.array_equal(back.view(np.uint32), y.view(np.uint32))
        again = orc.pack(cfg, back, axis=axis)
        for a, b in zip(planes, again):
            assert np.array_equal(a, b)


def test_column_direction_is_row_direction_of_the_transpose():
    x = synth.normal_matrix(48, 80, 50)
    for cfg in (orc.MX6, Cfg(32, 8, 8, 2, 3)):
        y0, s0 = orc.quant_dequant(cfg, x, axis=0)
        y1, s1 = orc.quant_dequant(cfg, np.ascontiguousarray(x.T), axis=1)
        assert np.array_equal(y0, y1.T) and s0 == pytest.approx(s1, rel=1e-12)
        for a, b in zip(orc.pack(cfg, x, axis=0), orc.pack(cfg, np.ascontiguousarray(x.T), axis=1)):
            assert np.array_equal(a, b)


def test_short_last_block_behaves_as_zero_padded():
    x = synth.normal(100, 60)
    for cfg in (orc.MX6, Cfg(64, 8, 8, 2, 5)):
        pad = np.zeros(-(-100 // cfg.k1) * cfg.k1, dtype=np.float32)
        pad[:100] = x
        y, s = orc.quant_dequant(cfg, x)
        yp, sp = orc.quant_dequant(cfg, pad)
        assert np.array_equal(y, yp[:100]) and s == pytest.approx(sp, rel=1e-12)
        for a, b in zip(orc.pack(cfg, x), orc.pack(cfg, pad)):
            assert np.array_equal(a, b)


def test_nonfinite_block_becomes_nan_block():
    x = synth.normal(64, 61)
    x[17] = np.inf
    y, (e2, s2) = orc.quant_dequant(orc.MX6, x)
    assert np.isnan(y[16:32]).all() and np.isfinite(y[:16]).all() and np.isfinite(y[32:]).all()
    assert np.isnan(orc.qsnr_db(e2, s2))
    exps, _, _ = orc.pack(orc.MX6, x)
    assert exps[0, 1] == 0xFF
    assert np.isnan(orc.unpack(orc.MX6, orc.pack(orc.MX6, x), 1, 64)[0, 16:32]).all()


# ---- QSNR (Eq. 3) ---------------------------------------------------------------------------------------
def test_qsnr_definition_closed_forms():
    assert orc.qsnr_db(1.0, 100.0) == pytest.approx(20.0, abs=1e-12)
    assert orc.qsnr_db(0.5, 0.5) == 0.0
    assert math.isinf(orc.qsnr_db(0.0, 1.0)) and math.isnan(orc.qsnr_db(0.0, 0.0))
    # an input made of representable values has infinite QSNR; sums are plain fp64 sums
    x = np.array([1.0, 0.5, -0.25, 1.75] * 4, dtype=np.float32)
    _, (e2, s2) = orc.quant_dequant(orc.MX6, x)
    assert e2 == 0.0 and s2 == 4 * (1 + 0.25 + 0.0625 + 3.0625)
    # one element off by exactly half a step: err^2 known in closed form
    x = np.zeros(16, dtype=np.float32); x[0] = 1.0; x[1] = 1.0 + 1.0 / 16           # MX6 step at E=0 is 1/8
    _, (e2, s2) = orc.quant_dequant(orc.MX6, x)
    assert e2 == (1.0 / 16) ** 2 and s2 == 1.0 + (17.0 / 16) ** 2


def test_soft_pins_from_the_pareto_discussion():
    """Section IV-C quotes approximate QSNR gaps on X ~ N(0,|N(0,1)|); hold them to +-1 dB."""
    x = synth.variable_variance_vectors(2048, 1024, seed=3)
    q = lambda *a, **k: orc.qsnr(Cfg(*a, **k), x)
    mx9, mx6, msfp16 = q(16, 8, 2, 1, 7), q(16, 8, 2, 1, 4), q(16, 8, 1, 0, 7)
    assert abs((mx9 - msfp16) - 3.6) < 1.0
    for m in (2, 4, 7):
        assert abs((q(16, 8, 2, 2, m) - q(16, 8, 2, 1, m)) - 0.5) < 0.5
        assert abs((q(16, 8, 2, 1, m) - q(16, 8, 8, 1, m)) - 2.0) < 1.0
        assert abs((q(16, 8, 1, 1, m) - q(16, 8, 2, 1, m)) - 0.7) < 0.5
    e4m3 = q(0, 32, 1, 4, 3, scale_kind=orc.FP32_FP)
    e5m2 = q(0, 32, 1, 5, 2, scale_kind=orc.FP32_FP)
    assert e5m2 < mx6 < e4m3
    assert 13.0 < mx9 - e4m3 < 18.0


# ---- comparator kinds --------------------------------------------------------------------------------------
def test_fp8_casts_match_library_casts():
    import torch
    x = np.concatenate([synth.normal(20000, 70) * 30, synth.edge_case_values(4000, 71),
                        np.array([0.0, -0.0, 448.0, 463.9, -448.0, 2 ** -9, 2 ** -10, 1.5 * 2 ** -10, 57344.0, 6e4,
                                  2 ** -16, 2 ** -17, 3 * 2 ** -17], dtype=np.float32)]).astype(np.float32)
    for (eb, mb, dt, lim) in ((4, 3, torch.float8_e4m3fn, 464.0), (5, 2, torch.float8_e5m2, 61440.0)):
        xs = x[np.abs(x) < lim]
        want = torch.from_numpy(xs).to(dt).to(torch.float32).numpy()
        got = orc.minifloat_round(xs, eb, mb)
        assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # saturation beyond the largest finite value
    assert orc.minifloat_round(np.array([1e9, -1e9], dtype=np.float32), 4, 3).tolist() == [448.0, -448.0]
    assert orc.minifloat_round(np.array([1e9], dtype=np.float32), 5, 2).tolist() == [57344.0]


def test_minifloat_rounding_by_nearest_value_search_over_the_explicit_code_set():
    # every (exponent bits, mantissa bits) shape the FP32_FP kind accepts, not only the two FP8 formats that have a
    # library cast: enumerate the format's finite values (bias 2^(eb-1)-1, gradual underflow, top exponent
    # reserved as in IEEE -- except E4M3, whose top exponent is finite up to 448), then find the nearest one to
    # each input with exact rationals; ties go to the even mantissa code (or away from zero); beyond the largest
    # value the cast saturates.
    for eb, mb in ((2, 1), (3, 2), (2, 3), (4, 3), (5, 2), (3, 4), (4, 1), (5, 7)):
        bias = (1 << (eb - 1)) - 1
        codes = []                                                   # (value, mantissa code) in ascending order
        top = (1 << eb) - 1 if (eb, mb) != (4, 3) else (1 << eb)
        for e in range(0, top):
            for f in range(1 << mb):
                if (eb, mb) == (4, 3) and e == 15 and f == 7:
                    continue                                          # the one NaN code of E4M3
                val = Fraction(f, 1 << mb) * Fraction(2) ** (1 - bias) if e == 0 else \
                    (1 + Fraction(f, 1 << mb)) * Fraction(2) ** (e - bias)
                codes.append((val, f))
        vals = [v for v, _ in codes]
        assert vals == sorted(vals) and len(set(vals)) == len(vals)
        fmax = vals[-1]
        if (eb, mb) == (4, 3):
            assert fmax == 448
        if (eb, mb) == (5, 2):
            assert fmax == 57344
        rng = np.random.default_rng(1000 + 10 * eb + mb)
        xs = np.concatenate([
            rng.normal(size=300).astype(np.float32) * np.float32(float(fmax) / 3),
            (rng.normal(size=300) * float(vals[1 << mb]) * 2).astype(np.float32),      # around the subnormal range
            np.array([float((a + b) / 2) for (a, _), (b, _) in zip(codes[:-1], codes[1:])], dtype=np.float32),  # exact ties
            np.array([float(fmax) * 1.5, -float(fmax) * 4, 0.0, float(vals[1]) / 2, float(vals[1]) / 4], dtype=np.float32)])
        for rnd in (orc.RNE, orc.RNA):
            got = orc.minifloat_round(xs, eb, mb, rnd)
            for x, g in zip(xs.tolist(), got.tolist()):
                a = abs(Fraction(x))
                if a >= fmax:
                    want = fmax
                else:
                    import bisect
                    hi = bisect.bisect_right(vals, a)                 # vals[hi-1] <= a < vals[hi]
                    lo_v, hi_v = vals[hi - 1], vals[hi]
                    if a - lo_v < hi_v - a:
                        want = lo_v
                    elif a - lo_v > hi_v - a:
                        want = hi_v
                    elif rnd == orc.RNA:
                        want = hi_v
                    else:
                        want = lo_v if codes[hi - 1][1] % 2 == 0 else hi_v
                assert Fraction(abs(g)) == want, (eb, mb, rnd, x, g, float(want))
                assert math.copysign(1, g) == math.copysign(1, x)


def test_fp8_kind_is_scale_then_cast():
    import torch
    x = synth.normal(4096, 72)
    x[0] = 448.0                                       # amax = 448 -> s = 1 -> the kind is the bare cast
    x = np.clip(x, -448, 448)
    y, _ = orc.quant_dequant(Cfg(0, 32, 1, 4, 3, orc.FP32_FP), x)
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).to(torch.float32).numpy()
    assert np.array_equal(y.view(np.uint32), want.view(np.uint32))
    assert orc.bits_per_element(Cfg(0, 32, 1, 4, 3, orc.FP32_FP)) == 8.0


def test_int_kind_reduces_to_integer_rounding_when_scale_is_one():
    # Eq. 1: s = max/(2^(b-1)-1); with max = 127 (INT8) s = 1 and Eq. 2 is RoundToInt(x)
    x = (synth.normal(4096, 73) * 40).clip(-127, 127).astype(np.float32)
    x[0] = 127.0
    y, _ = orc.quant_dequant(Cfg(0, 32, 1, 0, 7, orc.FP32_INT), x)
    assert np.array_equal(y, np.rint(x))
    # and is scale-equivariant under powers of two (s scales exactly)
    y2, _ = orc.quant_dequant(Cfg(0, 32, 1, 0, 7, orc.FP32_INT), x * np.float32(2.0 ** -9))
    assert np.array_equal(y2, y * np.float32(2.0 ** -9))
    # INT4: values are multiples of max/7
    x4 = synth.normal(1024, 74)
    y4, _ = orc.quant_dequant(Cfg(0, 32, 1, 0, 3, orc.FP32_INT), x4)
    k = y4 / (np.abs(x4).max() / np.float32(7))
    assert np.allclose(k, np.round(k), atol=1e-5) and np.abs(k).max() <= 7 + 1e-5


def test_vsq_reductions():
    # all 16-vectors share the same maximum -> every integer sub-scale is 2^d2-1 -> per-tensor INT
    x = synth.normal(2048, 75).reshape(-1, 16)
    x = (x / np.abs(x).max(axis=1, keepdims=True)).astype(np.float32)
    x[:, 0] = 1.0
    x = x.ravel()
    for m in (3, 7):
        yv, _ = orc.quant_dequant(Cfg(0, 32, 16, 8, m, orc.FP32_VSQ), x)
        yi, _ = orc.quant_dequant(Cfg(0, 32, 1, 0, m, orc.FP32_INT), x)
        assert np.allclose(yv, yi, rtol=3e-7, atol=0)
    # a finer sub-scale can only help on data with varied per-vector maxima
    x = synth.variable_variance_vectors(256, 16, 76).ravel()
    qs = [orc.qsnr(Cfg(0, 32, 16, d2, 3, orc.FP32_VSQ), x) for d2 in (4, 6, 8, 10)]
    assert qs[-1] > orc.qsnr(Cfg(0, 32, 1, 0, 3, orc.FP32_INT), x)
    assert qs == sorted(qs) or max(qs) - min(qs) < 1.0


def _vsq_cases():
    """tests/golden/vsq_blocks.txt -> [(name, rounding, k1, m, d2, gammas, [(u, x, q, Q), ...])]."""
    def expand(field):
        out = []
        for tok in field.split():
            out += [0.0] * int(tok[1:]) if tok[0] == "z" else [float(tok)]
        assert len(out) == 16, field
        return out
    cases = []
    for row in _golden_rows("vsq_blocks.txt"):
        if row.startswith("case"):
            _, name, rnd, k1, m, d2, gam = row.split()
            cases.append((name, int(rnd), int(k1), int(m), int(d2), [float(g) for g in gam.split(",")], []))
        else:
            u, xs, qs, Qs = [f.strip() for f in row[3:].split("|")]
            cases[-1][-1].append((int(u), expand(xs), expand(qs), expand(Qs)))
    return cases


def test_vsq_hand_worked_groups():
    # vectors with different maxima: an integer sub-scale that rounds up, one that rounds down (and makes its
    # largest element clamp), an exact tie in the sub-scale under both tie rules, the top code, an all-zero
    # vector, a vector flushed by u = 0, ties and clamps of the elements, and the scope of the first-level scale
    names = set()
    for name, rnd, k1, m, d2, gammas, vecs in _vsq_cases():
        names.add(name)
        x = np.array([v for _, xs, _, _ in vecs for v in xs], dtype=np.float32)
        want = np.array([v for _, _, _, Qs in vecs for v in Qs], dtype=np.float32)
        # the file is consistent with itself: Q = sign(x) * q * u * gamma, every product exact
        for i, (u, xs, qs, Qs) in enumerate(vecs):
            g = gammas[0] if k1 == 0 else gammas[i * 16 // k1]
            assert u <= 2 ** d2 - 1 and max(qs) <= 2 ** m - 1
            assert [abs(v) for v in Qs] == [q * u * g for q in qs], (name, i)
            assert [math.copysign(1, a) for a in Qs] == [math.copysign(1, a) for a in xs], (name, i)
        y, _ = orc.quant_dequant(Cfg(k1, 32, 16, d2, m, orc.FP32_VSQ, rnd), x)
        assert y.view(np.uint32).tolist() == want.view(np.uint32).tolist(), (name, y.tolist(), want.tolist())
    assert names == {"d4_even", "d4_away", "d6_even", "d6_away", "group32"}


def test_vsq_with_a_wide_sub_scale_approaches_int_with_one_fp32_scale_per_vector():
    # d2 = 16: u_v = RN(s_v / gamma) with gamma = s_max / 65535, so the effective scale u_v * gamma differs from
    # the vector's ideal scale s_v = amax_v / qmax by |delta| <= 0.5 / u_v (+ fp32 rounding).  With every vector
    # maximum within a factor 4 of the largest, u_v >= 16383 and |delta| <= 3.1e-5.  An element keeps its code q
    # unless |x|/s_v lies within qmax * |delta| of a half-integer; then |Q' - Q| <= q * s_v * |delta| <=
    # 7 * 3.1e-5 * s_v = 2.2e-4 s_v (m = 3); the rare element whose code flips moves by one step s_v (1 + delta).
    rng = np.random.default_rng(77)
    x = synth.normal(4096 * 16, 77).reshape(-1, 16)
    x = (x / np.abs(x).max(axis=1, keepdims=True) * rng.uniform(0.25, 1.0, (4096, 1))).astype(np.float32)
    m = 3
    qmax = 2 ** m - 1
    yv, (ev, sv) = orc.quant_dequant(Cfg(0, 32, 16, 16, m, orc.FP32_VSQ), x.ravel())
    yi, (ei, si) = orc.quant_dequant(Cfg(16, 32, 1, 0, m, orc.FP32_INT), x.ravel())
    s_v = (np.abs(x).max(axis=1, keepdims=True) / qmax).astype(np.float64)
    diff = np.abs(yv.reshape(-1, 16).astype(np.float64) - yi.reshape(-1, 16)) / s_v
    same_code = diff <= qmax * 3.2e-5
    flipped = ~same_code
    assert flipped.mean() < 2 * qmax * 3.2e-5 * 2            # half-integers are hit with probability ~2 q |delta|
    assert np.all(diff[flipped] <= 1.0 + 1e-3)
    # RMS error ~ s/sqrt(12); per-element change <= 2.2e-4 s (same code) => |dQSNR| <= 20 log10(1 + 8e-4) < 0.01 dB
    # for those, plus the flipped ones (error stays about half a step): bound the total by 0.02 dB
    assert sv == si and abs(orc.qsnr_db(ev, sv) - orc.qsnr_db(ei, si)) < 0.02
    # and the narrow sub-scales are measurably worse on the same data (the reduction is not vacuous)
    assert orc.qsnr(Cfg(0, 32, 16, 4, m, orc.FP32_VSQ), x.ravel()) < orc.qsnr_db(ei, si) - 0.1


# ---- first-level scale from elsewhere (delayed scaling), packing efficiency -------------------------------------
def test_supplied_first_level_maximum():
    import torch
    x = synth.normal(8192, 90) * np.float32(3.0)
    cur = float(np.abs(x).max())
    kinds = [Cfg(0, 32, 1, 0, 7, orc.FP32_INT), Cfg(0, 32, 1, 4, 3, orc.FP32_FP), Cfg(0, 32, 16, 6, 3, orc.FP32_VSQ)]
    for cfg in kinds:     # the current tensor's own maximum, supplied from outside: the same function
        a, sa = orc.quant_dequant(cfg, x)
        b, sb = orc.quant_dequant(cfg, x, amax=cur)
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32)) and sa == sb
    # INT8 with a supplied maximum of 127: s = 1, so Eq. 2 is rint(x) and values beyond the maximum saturate
    xi = (synth.normal(4096, 91) * 80).astype(np.float32)
    y, _ = orc.quant_dequant(Cfg(0, 32, 1, 0, 7, orc.FP32_INT), xi, amax=127.0)
    assert np.abs(xi).max() > 200 and np.array_equal(y, np.clip(np.rint(xi), -127, 127))
    # E4M3 with a supplied maximum of 448: s = 1, the library's saturating cast
    xf = (synth.normal(4096, 92) * 300).astype(np.float32)
    y, _ = orc.quant_dequant(Cfg(0, 32, 1, 4, 3, orc.FP32_FP), xf, amax=448.0)
    want = torch.from_numpy(np.clip(xf, -448, 448)).to(torch.float8_e4m3fn).to(torch.float32).numpy()
    assert np.abs(xf).max() > 448 and np.array_equal(y.view(np.uint32), want.view(np.uint32))
    # VSQ: the hand-worked group without its largest vector, with that vector's maximum supplied: same results
    for name, rnd, k1, m, d2, gammas, vecs in _vsq_cases():
        if name != "d4_even":
            continue
        xs = np.array([v for _, xx, _, _ in vecs[1:] for v in xx], dtype=np.float32)
        want = np.array([v for _, _, _, Q in vecs[1:] for v in Q], dtype=np.float32)
        y, _ = orc.quant_dequant(Cfg(0, 32, 16, d2, m, orc.FP32_VSQ, rnd), xs, amax=6.5625)
        assert y.view(np.uint32).tolist() == want.view(np.uint32).tolist()
        # a window maximum SMALLER than a vector's own (105/64: gamma = 1/64): (2/7) x 64 = 18.3 clamps at the top
        # sub-scale 15, scale 15/64; 2.0 / (15/64) = 8.5 saturates at 7; 0.78125 / (15/64) = 3.33 -> 3
        y, _ = orc.quant_dequant(Cfg(0, 32, 16, d2, m, orc.FP32_VSQ, rnd), xs[:16], amax=1.640625)
        assert y[0] == np.float32(7 * 15 / 64) and y[1] == np.float32(3 * 15 / 64)
    # a supplied maximum is refused where it has no meaning
    with pytest.raises(ValueError):
        orc.quant_dequant(orc.MX6, x, amax=1.0)


def test_tile_packing_efficiency_closed_form():
    # Section IV-B: a 256-element tile into 64-byte lines.  MX9: 288 bytes in 5 lines = 0.9; MX6 192 B, MX4 128 B and
    # FP8 256 B fill whole lines; MSFP12 (4.5 bits: 144 B in 3 lines) 0.75
    assert orc.tile_packing_efficiency(orc.MX9) == 288 / 320
    assert orc.tile_packing_efficiency(orc.MX6) == 1.0 and orc.tile_packing_efficiency(orc.MX4) == 1.0
    assert orc.tile_packing_efficiency(Cfg(0, 32, 1, 4, 3, orc.FP32_FP)) == 1.0
    assert orc.tile_packing_efficiency(Cfg(16, 8, 1, 0, 3)) == 144 / 192
    for cfg in (orc.MX9, Cfg(64, 8, 8, 2, 5), Cfg(8, 8, 1, 3, 2)):
        for tile, line in ((256, 64), (100, 32), (16, 128)):
            bits = orc.bits_per_element(cfg) * tile
            lines = math.ceil(bits / (8 * line))
            assert orc.tile_packing_efficiency(cfg, tile, line) == pytest.approx(bits / (lines * 8 * line), rel=1e-15)


def test_pareto_frontier_against_brute_force():
    from paper_2302_08007_b200 import sweep
    rng = np.random.default_rng(93)
    pts = [("p%d" % i, float(rng.integers(2, 12)) / 2, float(rng.normal(30, 10))) for i in range(200)]
    got = sweep.pareto_frontier(pts)
    brute = [p for p in pts if not any((q[1] <= p[1] and q[2] > p[2]) or (q[1] < p[1] and q[2] >= p[2]) for q in pts)]
    assert sorted(got) == sorted(brute)
    assert [g[1] for g in got] == sorted(g[1] for g in got) and [g[2] for g in got] == sorted(g[2] for g in got)
    assert sweep.bits_per_element(sweep.Config(16, 8, 2, 1, 7)) == 9.0


# ---- the dot product as the hardware pipeline computes it (Section IV-B, Fig. 6) --------------------------------
def _exact_dot_f32(qa, qb):
    """float32(sum_k qa[k] qb[k]) with the sum formed exactly (rationals), for dequantized fp32 operands."""
    out = np.empty((qa.shape[0], qb.shape[0]), dtype=np.float32)
    for i in range(qa.shape[0]):
        for j in range(qb.shape[0]):
            out[i, j] = np.float32(float(sum(Fraction(float(x)) * Fraction(float(y)) for x, y in zip(qa[i], qb[j]))))
    return out


def test_hw_dot_hand_worked_passes():
    cfg = Cfg(4, 8, 2, 1, 3)
    for row in _golden_rows("hw_dot_blocks.txt"):
        f, a, b, want = [t.strip() for t in row.split("|")]
        a = np.array([float(v) for v in a.split()], dtype=np.float32).reshape(1, -1)
        b = np.array([float(v) for v in b.split()], dtype=np.float32).reshape(1, -1)
        got = orc.gemm_hw(cfg, a, cfg, b, r=8, f=int(f))
        assert got.shape == (1, 1) and got[0, 0] == np.float32(float(want)), (row, got)


def test_hw_dot_is_the_exact_dot_product_when_nothing_is_shifted_out():
    rng = np.random.default_rng(95)
    # (1) MX9, one pass of 64: every block holds an element of magnitude 1.5, so all block exponents are equal and the
    # 25-bit frame keeps every bit of the 20-bit block results: the pass is the exact dot product, rounded once
    a = rng.normal(size=(5, 64)).astype(np.float32).clip(-1.4, 1.4)
    b = rng.normal(size=(4, 64)).astype(np.float32).clip(-1.4, 1.4)
    a[:, ::16] = 1.5
    b[:, 5::16] = -1.5
    qa, qb = orc.quant_dequant(orc.MX9, a)[0], orc.quant_dequant(orc.MX9, b)[0]
    assert np.array_equal(orc.gemm_hw(orc.MX9, a, orc.MX9, b, r=64, f=25), _exact_dot_f32(qa, qb))
    # (2) no microexponents (d2 = 0: plain block floating point), m = 7 x m = 4, block exponents up to 3 + 3 binades apart:
    # W = 7 + 4 + 4 = 15, the frame has 10 spare bits, nothing is lost
    ca, cb = Cfg(16, 8, 1, 0, 7), Cfg(16, 8, 1, 0, 4)
    a = (rng.normal(size=(3, 128)) * np.repeat(2.0 ** rng.integers(0, 4, (3, 8)), 16, axis=1)).astype(np.float32)
    b = (rng.normal(size=(6, 128)) * np.repeat(2.0 ** rng.integers(0, 4, (6, 8)), 16, axis=1)).astype(np.float32)
    qa, qb = orc.quant_dequant(ca, a)[0], orc.quant_dequant(cb, b)[0]
    assert np.array_equal(orc.gemm_hw(ca, a, cb, b, r=128, f=25), _exact_dot_f32(qa, qb))
    # and equals the integer dot product of the codes, block by block
    Fa, _, codea = orc.encode(ca, a)
    Fb, _, codeb = orc.encode(cb, b)
    sa = np.where(codea >> 7 & 1, -1, 1) * (codea & 127).astype(np.int64)
    sb = np.where(codeb >> 4 & 1, -1, 1) * (codeb & 15).astype(np.int64)
    i, j = 1, 4
    D = (sa[i] * sb[j]).reshape(8, 16).sum(axis=1)
    val = sum(Fraction(int(D[k])) * Fraction(2) ** (int(Fa[i, k]) + int(Fb[j, k]) - 254 - 6 - 3) for k in range(8))
    assert orc.gemm_hw(ca, a, cb, b, r=128, f=25)[i, j] == np.float32(float(val))


def test_hw_dot_truncation_is_bounded_ordered_and_pass_structured():
    rng = np.random.default_rng(96)
    a = (rng.normal(size=(4, 64)) * np.repeat(2.0 ** rng.integers(-6, 7, (4, 4)), 16, axis=1)).astype(np.float32)
    b = (rng.normal(size=(5, 64)) * np.repeat(2.0 ** rng.integers(-6, 7, (5, 4)), 16, axis=1)).astype(np.float32)
    qa, qb = orc.quant_dequant(orc.MX6, a)[0], orc.quant_dequant(orc.MX6, b)[0]
    exact = qa.astype(np.float64) @ qb.astype(np.float64).T          # exact in fp64: 64 products of 5-bit numbers
    Fa, Fb = orc.encode(orc.MX6, a)[0].astype(int), orc.encode(orc.MX6, b)[0].astype(int)
    W = 4 + 4 + 4 + 2
    lost = False
    for f in (6, 10, 14, 25):
        c = orc.gemm_hw(orc.MX6, a, orc.MX6, b, r=64, f=f).astype(np.float64)
        emax = (Fa[:, None, :] + Fb[None, :, :]).max(axis=2)
        unit = 2.0 ** (emax - 254 - 3 - 3 - 2 - (f - W))
        # each of the 4 blocks loses less than one unit of the frame (toward zero); the largest block loses nothing when f >= W
        err = np.abs(c - exact)
        assert np.all(err <= 4 * unit + 2.0 ** -23 * np.abs(exact)), f
        lost |= bool(np.any(err > 0))
    assert lost                                                       # the narrow frames do drop bits on this input
    # blocks of a pass may come in any order: the fixed-point sum is exact
    perm = np.array([2, 0, 3, 1])
    idx = (perm[:, None] * 16 + np.arange(16)[None, :]).ravel()
    assert np.array_equal(orc.gemm_hw(orc.MX6, a[:, idx], orc.MX6, b[:, idx], r=64, f=10), orc.gemm_hw(orc.MX6, a, orc.MX6, b, r=64, f=10))
    # K = 2 r: two passes, added in fp32 in order
    a2, b2 = np.concatenate([a, a[::-1]], axis=1), np.concatenate([b, 3 * b], axis=1)
    p1 = orc.gemm_hw(orc.MX6, a2[:, :64], orc.MX6, b2[:, :64], r=64, f=10)
    p2 = orc.gemm_hw(orc.MX6, a2[:, 64:], orc.MX6, b2[:, 64:], r=64, f=10)
    assert np.array_equal(orc.gemm_hw(orc.MX6, a2, orc.MX6, b2, r=64, f=10), p1 + p2)
    # shorter passes align fewer blocks to a common exponent: r = 16 (one block per pass) loses nothing in the frame
    one = orc.gemm_hw(orc.MX6, a, orc.MX6, b, r=16, f=14)
    blocks = sum((qa[:, k:k + 16].astype(np.float64) @ qb[:, k:k + 16].astype(np.float64).T).astype(np.float32) for k in range(0, 64, 16))
    assert np.array_equal(one, blocks.astype(np.float32))
    # an Inf/NaN block poisons the outputs of its row only
    an = a.copy()
    an[2, 17] = np.inf
    cn = orc.gemm_hw(orc.MX6, an, orc.MX6, b, r=64, f=25)
    assert np.isnan(cn[2]).all() and not np.isnan(np.delete(cn, 2, axis=0)).any()
    with pytest.raises(ValueError):
        orc.gemm_hw(orc.MX6, a, orc.MX9._replace(k2=4) if hasattr(orc.MX9, "_replace") else Cfg(16, 8, 4, 1, 7), b)


# ---- three-level scaling: FP32 parent scale above the block scale (Section III, extension) ---------------------------
def test_parent_scale_hand_worked_group_and_reductions():
    # k1 = 4, k2 = 2, d2 = 1, m = 3: V = 7/4.  Group maximum 5.25 -> s = 3 exactly; x/3 = [1.75 1 | -.5 .25] [.2 -.3 | .1 .0333]
    # block 0: F 127, tau [0 1], q [7 4 | -4 2]: exact.  block 1: F 125 (0.3), units 1/16 and 1/32: 3.2 -> 3, 4.8 -> 5, 3.2 -> 3,
    # 1.07 -> 1: [.1875 -.3125 | .09375 .03125]; times 3.  (Worked by hand; without the parent scale 5.25 -> 5 and 0.75 -> 1.)
    cfg = Cfg(4, 8, 2, 1, 3)
    x = np.array([5.25, 3.0, -1.5, 0.75, 0.6, -0.9, 0.3, 0.1], dtype=np.float32)
    y, _ = orc.quant_dequant_parent(cfg, 8, x)
    assert y.tolist() == [5.25, 3.0, -1.5, 0.75, 0.5625, -0.9375, 0.28125, 0.09375]
    assert orc.quant_dequant(cfg, x)[0].tolist()[:4] == [5.0, 3.0, -1.5, 1.0]
    # a group maximum of V 2^t makes the parent scale a power of two: the two-level quantizer itself (scale equivariance)
    for cfg in (orc.MX4, orc.MX6, orc.MX9, Cfg(16, 8, 4, 2, 5)):
        V = (2 ** cfg.m - 1) * 2.0 ** -(cfg.m - 1)
        x = synth.normal_matrix(8, 512, 97).clip(-1.7, 1.7)
        for r in range(8):
            x[r, 37 * r] = V * 2.0 ** (r - 3)
            x[r] = np.clip(x[r], -V * 2.0 ** (r - 3), V * 2.0 ** (r - 3))
        for kp in (512, 128):
            xx = x.copy()
            if kp == 128:                                   # every group of 128 needs its own maximum of that form
                xx[:, ::128] = (V * 2.0 ** (np.arange(8) - 3))[:, None]
            y3, s3 = orc.quant_dequant_parent(cfg, kp, xx)
            y2, s2 = orc.quant_dequant(cfg, xx)
            assert np.array_equal(y3.view(np.uint32), y2.view(np.uint32)) and s3 == s2
    # the group's largest element comes back within a rounding of the two divisions / multiplications; zeros stay zeros
    x = synth.variable_variance_vectors(64, 1024, 98)
    x[5] = 0.0
    x[5, 3] = -0.0
    for cfg in (orc.MX4, orc.MX9):
        y, _ = orc.quant_dequant_parent(cfg, 1024, x)
        i = np.abs(x).argmax(axis=1)
        top, got = x[np.arange(64), i], y[np.arange(64), i]
        ok = top != 0
        assert np.all(np.abs(got[ok] - top[ok]) <= 4 * np.spacing(np.abs(top[ok])))
        assert not y[5].any() and np.signbit(y[5, 3])
    # lines are independent and the column direction is the row direction of the transpose
    xm = synth.normal_matrix(64, 48, 99)
    a, sa = orc.quant_dequant_parent(orc.MX6, 32, xm, axis=0)
    b, sb = orc.quant_dequant_parent(orc.MX6, 32, np.ascontiguousarray(xm.T), axis=1)
    assert np.array_equal(a, b.T) and sa == pytest.approx(sb, rel=1e-12)
    with pytest.raises(ValueError):
        orc.quant_dequant_parent(orc.MX6, 24, xm)


# ---- GEMM reference ---------------------------------------------------------------------------------------------
def test_gemm_reference_is_the_plain_definition():
    rng = np.random.default_rng(80)
    a = rng.integers(-8, 9, (7, 33)).astype(np.float32)
    b = rng.integers(-8, 9, (5, 33)).astype(np.float32)
    c = orc.gemm_nt_f64(a, b)
    assert np.array_equal(c, (a.astype(np.int64) @ b.astype(np.int64).T).astype(np.float64))
    assert np.array_equal(orc.gemm_nt_f64(a, b, nthreads=3), c)
    ri, ci = np.array([0, 6, 3]), np.array([4, 0, 2])
    assert np.array_equal(orc.gemm_nt_f64_sampled(a, b, ri, ci), c[ri, ci])


def test_multithreaded_oracle_is_the_same_function():
    x = synth.normal_matrix(64, 256, 81)
    for axis in (0, 1):
        a, sa = orc.quant_dequant(orc.MX6, x, axis=axis)
        b, sb = orc.quant_dequant(orc.MX6, x, axis=axis, nthreads=4)
        assert np.array_equal(a, b) and sa == sb


# ---- re-encoding onto E4M3 + power-of-two block scales (library extension; oracle/reencode.py) ----------------
def test_e4m3_byte_table_matches_the_library_cast():
    torch = pytest.importorskip("torch")
    from oracle import reencode as R
    lib_vals = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).to(torch.float32).numpy().astype(np.float64)
    table = R.e4m3_value_table()
    assert np.array_equal(table[:0x7F], lib_vals[:0x7F]) and np.isnan(table[0x7F]) and np.isnan(lib_vals[0x7F])
    both = np.concatenate([lib_vals[:0x7F], -lib_vals[:0x7F]])
    got, hit = R.e4m3_bytes(both)
    assert hit.all() and np.array_equal(got, np.concatenate([np.arange(0x7F), 0x80 + np.arange(0x7F)]).astype(np.uint8))
    _, hit = R.e4m3_bytes(np.array([17.0, 2.0 ** -10, 3.0 * 2.0 ** -10, 449.0, 0.3]))     # five significant bits, below the
    assert not hit.any()                                                                  # finest step, above the range


def test_reencoding_reconstructs_the_decoded_operand_and_knows_its_limits():
    from oracle import reencode as R
    rng = np.random.default_rng(8)
    table = R.e4m3_value_table()
    for cfg, m in ((orc.MX6, 4), (orc.MX4, 2)):
        x = rng.standard_normal((128, 256)).astype(np.float32)
        x[:, 64:80] = 0.0                                            # an all-zero block beside a normal one
        out, scales, inexact = R.reencode_e4m3(cfg, x)
        assert not inexact
        y, _ = orc.quant_dequant(cfg, x)
        sb = scales.reshape(2, 1, 32, 4, 4).transpose(1, 3, 2, 0, 4).reshape(128, 8).astype(np.int64)
        val = np.where(out & 0x80, -1.0, 1.0) * table[out & 0x7F] * np.repeat(np.ldexp(1.0, sb - 127), 32, axis=1)
        assert np.array_equal(val, y.astype(np.float64))
        # scale byte = larger block exponent of the pair minus 7
        F, _, _ = orc.encode(cfg, x)
        assert np.array_equal(sb, F.astype(np.int64).reshape(128, 8, 2).max(axis=2) - 7)
        # neighbouring blocks d binades apart, every magnitude in [1, 2) * 2^F (so tau = 0): exact up to d = 16 - (m - 1)
        for d, want_inexact in ((16 - (m - 1), False), (17 - (m - 1), True)):
            z = ((1.0 + rng.integers(0, 8, (128, 128)) / 8.0) * np.where(rng.random((128, 128)) < 0.5, -1, 1)).astype(np.float32)
            z[:, 16:32] *= np.float32(2.0 ** -d)
            assert R.reencode_e4m3(cfg, z)[2] == want_inexact, (m, d)
    tiny = np.full((128, 128), 1.0, np.float32)
    tiny[3, 0:16] = np.float32(1e-38)                                # block exponent below 16
    assert R.reencode_e4m3(orc.MX6, tiny)[2]
