"""Pins for the CPU oracle: what the paper and the mathematics fix, checked without a GPU.

Each test is chosen so that a plausible slip in the oracle (dropped term, wrong sign or
index, wrong grid bound, transposed layout) makes it fail.
"""
import os

import numpy as np
import pytest

from oracle import omse_oracle as orc
from paper_1902_06822_b200 import synth
from exact_opt import exact_optimum

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _bounds(bits, signed):
    return (-(1 << (bits - 1)), (1 << (bits - 1)) - 1) if signed else (0, (1 << bits) - 1)


# ---------------------------------------------------------------- Section 3.1: grids, operator
def test_grid_bounds_match_section_3_1():
    assert orc.grid_bounds(4, True) == (-8, 7)
    assert orc.grid_bounds(4, False) == (0, 15)
    assert orc.grid_bounds(2, True) == (-2, 1)
    assert orc.grid_bounds(8, True) == (-128, 127)
    assert orc.grid_bounds(8, False) == (0, 255)


def test_rounding_is_half_to_even_then_saturates():
    # x/alpha with alpha = 1: 0.5 -> 0, 1.5 -> 2, 2.5 -> 2, -0.5 -> 0, -1.5 -> -2, 7.5 -> 8 -> 7, -9 -> -8
    x = np.array([0.5, 1.5, 2.5, -0.5, -1.5, 7.5, -9.0, 6.5, 100.0], np.float32)
    assert orc.codes(x, 1.0, 4, True).tolist() == [0, 2, 2, 0, -2, 7, -8, 6, 7]
    assert orc.codes(x, 1.0, 4, False).tolist() == [0, 2, 2, 0, 0, 8, 0, 6, 15]


# ---------------------------------------------------------------- hand-worked example
def test_hand_worked_two_bit_example():
    """x = (0.9, -0.35, 0.1, 0.5), signed 2-bit grid {-2..1}, 4 candidates in (0, 0.9].

    By hand: alpha = 0.225, 0.45, 0.675, 0.9 give squared errors 0.55125, 0.225, 0.196875, 0.2925
    (codes (1,-2,0,1), (1,-1,0,1), (1,-1,0,1), (1,0,0,1)); the third wins.  With codes (1,-1,0,1)
    the least-squares scale is (0.9+0.35+0.5)/3 = 0.58333..., which re-quantizes to the same codes,
    and the error is 0.31667^2 + 0.23333^2 + 0.1^2 + 0.08333^2 = 0.171667.
    """
    x = np.array([0.9, -0.35, 0.1, 0.5], np.float32)
    r0 = orc.phi(x, bits=2, is_signed=True, n_cand=4, refine_iters=0, want_curve=True)
    np.testing.assert_allclose(r0.sse_curve, [0.55125, 0.225, 0.196875, 0.2925], rtol=1e-6)
    assert r0.best_idx == 2 and r0.codes.tolist() == [1, -1, 0, 1]
    np.testing.assert_allclose(r0.alpha, 0.675, rtol=1e-6)
    r3 = orc.phi(x, bits=2, is_signed=True, n_cand=4, refine_iters=3)
    np.testing.assert_allclose(r3.alpha, 1.75 / 3.0, rtol=1e-6)
    np.testing.assert_allclose(r3.sse, 0.1716667, rtol=1e-5)
    assert r3.codes.tolist() == [1, -1, 0, 1] and r3.best_idx == 2


def test_lowest_index_wins_exact_ties():
    # K = 1, x = 1: candidates 1/4, 1/2, 3/4, 1 reproduce x with codes 4, 2, (1), 1: three exact zeros.
    r = orc.phi(np.array([1.0], np.float32), bits=4, n_cand=4, refine_iters=0, want_curve=True)
    assert r.sse_curve.tolist() == [0.0, 0.0, 0.0625, 0.0]
    assert r.best_idx == 0 and r.alpha == 0.25 and r.codes.tolist() == [4]


# ---------------------------------------------------------------- Section 3.4: exact optimum (brute force)
def _tiny_cases():
    rng = np.random.default_rng(1234)
    for trial in range(60):
        k = int(rng.choice([1, 2, 3, 8, 27, 64]))
        bits = int(rng.choice([2, 3, 4]))
        signed = bool(rng.integers(0, 2))
        n_cand = int(rng.choice([16, 64, 256]))
        if trial % 2:
            x = rng.laplace(0.0, 0.02, k)
        else:
            x = rng.standard_t(3, k)
        if not signed and trial % 3 == 0:
            x = np.abs(x)
        yield x.astype(np.float32), bits, signed, n_cand


@pytest.mark.parametrize("case", list(_tiny_cases()), ids=lambda c: f"K{c[0].size}-p{c[1]}-{'s' if c[2] else 'u'}-C{c[3]}")
def test_grid_search_within_grid_resolution_of_exact_optimum(case):
    x, bits, signed, n_cand = case
    lo, hi = _bounds(bits, signed)
    m = float(np.max(np.abs(x)))
    step = m / n_cand
    r0 = orc.phi(x, bits, signed, n_cand, 1.0, 0, want_curve=True)
    r3 = orc.phi(x, bits, signed, n_cand, 1.0, 3)
    # (a) nothing on (0, max|x|] beats the grid answer by more than the grid resolution allows:
    #     ||x - a_c q*|| <= ||x - a* q*|| + |a_c - a*| ||q*||, and rounding at a_c can only do better.
    sse_star, a_star, q_star = exact_optimum(x, lo, hi, a_max=m)
    grid = (np.arange(n_cand) + 1) * step
    dist = float(np.min(np.abs(grid - a_star)))
    assert dist <= step * (1 + 1e-9)
    bound = (np.sqrt(sse_star) + dist * np.linalg.norm(q_star)) ** 2
    assert r0.sse <= bound * (1 + 1e-5) + 1e-30
    # (b) the polished answer never gets worse than the grid answer
    assert r3.sse <= r0.sse * (1 + 1e-6) + 1e-30
    # (c) and no answer can be better than the true optimum over all alpha > 0
    sse_glob, _, _ = exact_optimum(x, lo, hi)
    assert sse_glob <= sse_star * (1 + 1e-12)
    assert r3.sse >= sse_glob * (1 - 1e-6) - 1e-30
    assert r0.sse >= sse_star * (1 - 1e-6) - 1e-30
    # (d) the reported minimum is the minimum of the reported curve, lowest index first
    assert r0.best_idx == int(np.argmin(r0.sse_curve))
    assert r0.sse == pytest.approx(r0.sse_curve[r0.best_idx], rel=1e-12)


def test_sse_curve_matches_definition_in_numpy():
    """Section 3.4 objective at every candidate, recomputed with numpy (fp32 divide, fp64 error)."""
    x = synth.laplace(576, 0.02, seed=11)
    for bits, signed in [(4, True), (4, False), (3, True), (8, True)]:
        lo, hi = _bounds(bits, signed)
        r = orc.phi(x, bits, signed, 128, 1.0, 0, want_curve=True)
        m = np.float32(np.max(np.abs(x)))
        step = np.float32(m) / np.float32(128)
        for c in (0, 1, 17, 63, 127, r.best_idx):
            a = np.float32(c + 1) * step
            q = np.clip(np.rint(x / a), lo, hi).astype(np.float64)
            sse = np.sum((x.astype(np.float64) - np.float64(a) * q) ** 2)
            assert r.sse_curve[c] == pytest.approx(sse, rel=1e-12)
            assert orc.candidate(m, 1.0, 128, c) == float(a)


# ---------------------------------------------------------------- special cases with closed forms
def test_input_already_on_a_candidate_grid_is_reproduced_exactly():
    a = 2.0 ** -5
    k = np.array([-8, 7, 3, 0, -1, 5, 7, -8, 2, 1, -4, 6], np.float32)
    x = k * np.float32(a)          # max|x| = 8a; with 64 candidates the step is a/8, so candidate 7 is a
    r = orc.phi(x, 4, True, 64, 1.0, 3, want_curve=True)
    assert r.best_idx == 7 and r.sse == 0.0 and r.alpha == a
    assert r.codes.tolist() == k.astype(int).tolist()
    assert np.count_nonzero(r.sse_curve == 0.0) == 1


def test_single_element_segment_is_reproduced_after_polish():
    for v in (0.37, -1.9, 3e-5):
        r = orc.phi(np.array([v], np.float32), 4, True, 16, 1.0, 1)
        assert abs(r.alpha * int(r.codes[0]) - np.float32(v)) <= 1e-6 * abs(v)
        assert r.sse <= (1e-6 * v) ** 2


@pytest.mark.parametrize("bits,signed", [(4, True), (3, True), (8, True), (4, False)])
def test_one_candidate_at_max_over_L_is_the_uniform_quantizer(bits, signed):
    """Section 3.1 without offset: alpha = max|T| / (2^(p-1) - 1), codes = [T/alpha]."""
    lo, hi = _bounds(bits, signed)
    x = synth.student_t3(300, seed=7, tensor_id=bits)
    if not signed:
        x = np.abs(x)
    r = orc.phi(x, bits, signed, 1, 1.0 / hi, 0)
    a_paper = float(np.max(np.abs(x))) / hi
    assert r.alpha == pytest.approx(a_paper, rel=3e-7) and r.best_idx == 0
    q = np.clip(np.rint(x / np.float32(r.alpha)), lo, hi).astype(np.float64)
    assert np.array_equal(r.codes, q.astype(np.int8))
    assert r.sse == pytest.approx(np.sum((x.astype(np.float64) - r.alpha * q) ** 2), rel=1e-12)
    assert r.sse <= float(np.sum(x.astype(np.float64) ** 2))


def test_eight_bit_error_follows_uniform_noise_model():
    """No saturation, fine grid: squared error per element ~ alpha^2 / 12 (textbook rounding noise)."""
    rng = np.random.default_rng(5)
    x = rng.uniform(-1.0, 1.0, 20000).astype(np.float32)
    r = orc.phi(x, 8, True, 1, 1.0 / 127, 0)
    assert r.sse / x.size == pytest.approx(r.alpha ** 2 / 12.0, rel=0.05)


# ---------------------------------------------------------------- invariants
def test_invariants_on_cnn_shaped_rows():
    w = synth.conv_layer(seed=1)[:16]
    prev = None
    for bits in (2, 3, 4, 8):
        lo, hi = _bounds(bits, True)
        res = orc.quantize_rows(w, bits, True, 256, 1.0, 3)
        res0 = orc.quantize_rows(w, bits, True, 256, 1.0, 0)
        assert res.codes.min() >= lo and res.codes.max() <= hi
        assert np.all(res.sse <= res0.sse * (1 + 1e-9))             # polish never hurts
        assert np.all(res.sse <= np.sum(w.astype(np.float64) ** 2, axis=1))
        assert np.array_equal(res.best_idx, res0.best_idx)
        if prev is not None:
            assert res.sse.mean() < prev                              # error shrinks with bit width
        prev = res.sse.mean()


def test_power_of_two_scaling_is_exact_and_permutation_keeps_alpha():
    x = synth.student_t3(147, seed=9)
    r = orc.phi(x, 4, True, 256, 1.0, 3)
    r8 = orc.phi(x * np.float32(8.0), 4, True, 256, 1.0, 3)
    assert r8.alpha == r.alpha * 8.0 and np.array_equal(r8.codes, r.codes) and r8.best_idx == r.best_idx
    assert r8.sse == pytest.approx(64.0 * r.sse, rel=1e-12)
    perm = np.random.default_rng(0).permutation(x.size)
    rp = orc.phi(x[perm], 4, True, 256, 1.0, 0)
    r0 = orc.phi(x, 4, True, 256, 1.0, 0)
    assert rp.alpha == r0.alpha and rp.best_idx == r0.best_idx and np.array_equal(rp.codes, r0.codes[perm])
    assert rp.sse == pytest.approx(r0.sse, rel=1e-12)


def test_grid_search_beats_alternation_from_the_uniform_start_somewhere():
    """Section 3.4: alternation alone can stop in a local minimum of the non-convex objective; the grid cannot."""
    w = synth.resnet50_weights(seed=2)[1][1][:64]       # 64 rows of a 1x1 convolution
    grid = orc.quantize_rows(w, 4, True, 256, 1.0, 3).sse
    alt = orc.quantize_rows(w, 4, True, 1, 1.0 / 7, 10).sse   # uniform start + 10 alternations
    assert np.all(grid <= alt * 1.05)
    assert np.mean(grid < alt * 0.999) > 0.25


def test_degenerate_rows():
    r = orc.phi(np.zeros(9, np.float32), 4, True, 16, 1.0, 3)
    assert r.alpha == 0.0 and r.best_idx == -1 and r.sse == 0.0 and not r.codes.any()
    assert r.status & orc.STATUS_DEGENERATE
    r = orc.phi(np.array([1.0, np.nan, 0.5], np.float32), 4, True, 16, 1.0, 0)
    assert r.status & orc.STATUS_NONFINITE


# ---------------------------------------------------------------- layouts: rows, per tensor, restart
def test_rows_per_tensor_and_restart_agree_with_single_segment_phi():
    w = synth.sweep_tensor(27, seed=5, n_kernels=10)
    res = orc.quantize_rows(w, 3, True, 64, 1.0, 2)
    for s in (0, 4, 9):
        r = orc.phi(w[s], 3, True, 64, 1.0, 2)
        assert (r.alpha, r.sse, r.best_idx) == (res.alpha[s], res.sse[s], res.best_idx[s])
        assert np.array_equal(r.codes, res.codes[s])
    again = orc.quantize_rows(w, 3, True, 64, 1.0, 2, start_idx=res.best_idx)
    assert np.array_equal(again.alpha, res.alpha) and np.array_equal(again.codes, res.codes)
    x = synth.relu_activations(5000, seed=3)
    a = orc.activation_scale(x, 4, False, 128, 1.0, 3)
    r = orc.phi(x, 4, False, 128, 1.0, 3, want_curve=True)
    assert (a.alpha, a.sse, a.best_idx) == (r.alpha, r.sse, r.best_idx)
    assert np.array_equal(a.sse_curve, r.sse_curve)


# ---------------------------------------------------------------- Section 3.5 / 3.7: residual, Algorithm 1
def test_residual_quantization_bookkeeping_and_gain():
    t = synth.laplace_with_outliers(12 * 200, 0.005, seed=4, outlier_prob=0.01).reshape(12, 200)
    res = orc.residual_rows(t, (4, 4), True, 128, 1.0, 3, n_sweeps=1)
    t64 = t.astype(np.float64)
    first = orc.quantize_rows(t, 4, True, 128, 1.0, 3)
    # tensor 1 of the first sweep is plain phi(T)
    assert np.array_equal(res.alpha[0], first.alpha) and np.array_equal(res.codes[0], first.codes)
    np.testing.assert_allclose(res.sse[0], first.sse, rtol=1e-12)
    # tensor 2 is phi of the fp32 residual T - alpha1*q1
    r1 = np.empty_like(t)
    for s in range(12):
        r1[s] = (t64[s] - np.float64(res.alpha[0, s]) * res.codes[0, s]).astype(np.float32)  # exact product, one rounding
    second = orc.quantize_rows(r1, 4, True, 128, 1.0, 3)
    assert np.array_equal(res.alpha[1], second.alpha) and np.array_equal(res.codes[1], second.codes)
    # the reported errors are the reconstruction errors of Section 3.5's objective
    rec1 = res.alpha[0][:, None].astype(np.float64) * res.codes[0]
    rec2 = rec1 + res.alpha[1][:, None].astype(np.float64) * res.codes[1]
    np.testing.assert_allclose(res.sse[0], np.sum((t64 - rec1) ** 2, axis=1), rtol=1e-9)
    np.testing.assert_allclose(res.sse[1], np.sum((t64 - rec2) ** 2, axis=1), rtol=1e-6)
    assert np.all(res.sse[1] < res.sse[0])                      # a second tensor shrinks the error
    assert res.sse[1].sum() < 0.1 * res.sse[0].sum()


def test_algorithm_1_second_sweep_uses_all_other_tensors():
    t = synth.student_t3(5 * 96, seed=21).reshape(5, 96)
    one = orc.residual_rows(t, (3, 3), True, 64, 1.0, 2, n_sweeps=1)
    two = orc.residual_rows(t, (3, 3), True, 64, 1.0, 2, n_sweeps=2)
    t64 = t.astype(np.float64)
    # second sweep, j = 1: phi(T - alpha2*q2) with the first sweep's second tensor
    for s in range(5):
        r = np.float32(t64[s] - np.float64(one.alpha[1, s]) * one.codes[1, s])
        p = orc.phi(r, 3, True, 64, 1.0, 2)
        assert p.alpha == two.alpha[0, s] and np.array_equal(p.codes, two.codes[0, s])
    rec = sum(two.alpha[j][:, None].astype(np.float64) * two.codes[j] for j in range(2))
    np.testing.assert_allclose(two.sse[1], np.sum((t64 - rec) ** 2, axis=1), rtol=1e-6)
    assert two.sse[1].sum() <= one.sse[1].sum() * 1.02


def test_three_tensors_keep_shrinking_the_error():
    t = synth.laplace(4 * 300, 0.01, seed=8).reshape(4, 300)
    res = orc.residual_rows(t, (2, 2, 2), True, 64, 1.0, 2, n_sweeps=1)
    assert np.all(res.sse[1] < res.sse[0]) and np.all(res.sse[2] < res.sse[1])
    assert res.codes.min() >= -2 and res.codes.max() <= 1


# ---------------------------------------------------------------- INT4 packing and compression ratio
def test_pack_layout_by_hand_and_round_trip_over_all_bytes():
    assert orc.pack_int4(np.array([1, -1, 7], np.int8)).tolist() == [0xF1, 0x07]
    assert orc.pack_int4(np.array([-8, 3, 0, -2], np.int8)).tolist() == [0x38, 0xE0]
    allbytes = np.arange(256, dtype=np.uint8)
    for signed in (True, False):
        q = orc.unpack_int4(allbytes, 512, signed)
        lo, hi = _bounds(4, signed)
        assert q.min() == lo and q.max() == hi
        assert np.array_equal(orc.pack_int4(q), allbytes)
        assert q[2 * 0x5A] == (0xA - 16 if signed else 0xA) and q[2 * 0x5A + 1] == 5


def test_compression_ratio_of_resnet50_shape_set_matches_the_paper():
    gold = dict(line.split() for line in open(os.path.join(GOLDEN, "compression_ratio.txt")) if line[0] != "#")
    shapes = synth.resnet50_shapes()
    n = sum(s * k for _, s, k in shapes)
    rows = sum(s for _, s, k in shapes)
    assert (len(shapes), n, rows) == (54, 25_502_912, 27_560)
    packed_bytes = sum(orc.pack_int4(np.zeros(s * k, np.int8)).size for _, s, k in shapes[:3]) \
        + sum((s * k + 1) // 2 for _, s, k in shapes[3:])
    cr = (packed_bytes + 4 * rows) / (4 * n)           # codes + one fp32 scale per kernel over the fp32 model
    assert float(gold["int4_non_dual_cr_approx"]) <= cr <= float(gold["resnet50_cr_with_dual_layers"]) + 5e-5
    assert cr == pytest.approx(0.12608, abs=1e-5)


# ---------------------------------------------------------------- Section 3.5: dual line search (n = 2)
def test_dual_per_element_enumeration_equals_joint_brute_force():
    """The third equation of Section 3.5: minimising over the first code with the second one rounded
    equals minimising over both codes jointly (brute force over all 16 x 16 pairs, float64)."""
    rng = np.random.default_rng(3)
    for trial in range(6):
        x = rng.laplace(0.0, 0.02, 40).astype(np.float32)
        a1 = np.float32(rng.uniform(0.004, 0.02))
        a2 = np.float32(a1 * rng.uniform(0.03, 0.3))
        t = np.arange(-8, 8)[:, None, None]
        q = np.arange(-8, 8)[None, :, None]
        err = (x.astype(np.float64)[None, None, :] - np.float64(a1) * t - np.float64(a2) * q) ** 2
        joint = err.reshape(256, -1).min(axis=0).sum()
        assert orc.dual_sse_at(x, a1, a2) == pytest.approx(joint, rel=1e-6)


def test_dual_recovers_inputs_on_the_joint_grid_exactly():
    a = 2.0 ** -4
    rng = np.random.default_rng(9)
    t = rng.integers(-8, 8, 50)
    q = rng.integers(-8, 8, 50)
    t[0], q[0] = -8, -8                              # max|x| = 8a + a/2 = 8.5a
    x = (t * a + q * (a / 16)).astype(np.float32)
    # one pair on the grid: alpha1 = hi_frac1*max = a, alpha2 = hi_frac2*alpha1 = a/16
    r = orc.dual(x, 4, 4, True, 1, 1, hi_frac1=1.0 / 8.5, hi_frac2=1.0 / 16)
    assert r.alpha[0] == pytest.approx(a, rel=1e-6) and r.alpha[1] == pytest.approx(a / 16, rel=1e-6)
    if r.alpha[0] == a and r.alpha[1] == a / 16:
        assert r.sse == 0.0 and np.array_equal(r.codes[0], t) and np.array_equal(r.codes[1], q)
    assert r.sse <= 1e-12


def test_dual_bookkeeping_argmin_and_invariants():
    x = synth.laplace(147, 0.05, seed=31)
    r = orc.dual(x, 4, 4, True, 12, 10, 1.0, 0.25, want_curve=True)
    assert r.best_idx == int(np.argmin(r.sse_curve)) and r.sse == pytest.approx(r.sse_curve[r.best_idx], rel=1e-12)
    c, d = divmod(r.best_idx, 10)
    a1, a2 = orc.dual_scales(float(np.max(np.abs(x))), 1.0, 0.25, 12, 10, c, d)
    assert (a1, a2) == (r.alpha[0], r.alpha[1])
    m = np.float32(np.max(np.abs(x)))
    assert a1 == np.float32(c + 1) * (m / np.float32(12)) and a2 == np.float32(d + 1) * (np.float32(0.25) * a1 / np.float32(10))
    rec = np.float64(a1) * r.codes[0] + np.float64(a2) * r.codes[1]
    assert r.sse == pytest.approx(np.sum((x.astype(np.float64) - rec) ** 2), rel=1e-12)
    assert r.codes.min() >= -8 and r.codes.max() <= 7
    again = orc.dual(x, 4, 4, True, 12, 10, 1.0, 0.25, start_idx=r.best_idx)
    assert again.sse == r.sse and np.array_equal(again.codes, r.codes)
    r8 = orc.dual(x * np.float32(4.0), 4, 4, True, 12, 10, 1.0, 0.25)
    assert np.array_equal(r8.codes, r.codes) and r8.alpha[0] == 4 * r.alpha[0] and r8.sse == pytest.approx(16 * r.sse, rel=1e-12)
    rows = orc.dual_rows(np.stack([x, -x, x[::-1]]), 4, 4, True, 12, 10, 1.0, 0.25)
    assert rows.sse[0] == r.sse and np.array_equal(rows.codes[:, 0], r.codes) and rows.alpha[0, 0] == r.alpha[0]
    z = orc.dual(np.zeros(5, np.float32), 4, 4, True, 4, 4)
    assert z.best_idx == -1 and z.sse == 0.0 and z.status & orc.STATUS_DEGENERATE


def test_dual_beats_the_residual_scheme_at_its_own_scales_and_on_average():
    """At the residual scheme's (alpha1, alpha2) its codes are one of the choices the enumeration sees,
    so the dual objective cannot be larger; over a grid it is smaller on average (Section 3.5)."""
    w = synth.conv_layer(seed=1)[:12]
    res = orc.residual_rows(w, (4, 4), True, 256, 1.0, 3, 1)
    gain = []
    for s in range(12):
        at = orc.dual_sse_at(w[s], res.alpha[0, s], res.alpha[1, s])
        assert at <= res.sse[1, s] * (1 + 1e-6)
        gain.append(res.sse[1, s] / orc.dual(w[s], 4, 4, True, 24, 24, 1.0, 0.25).sse)
    assert np.mean(gain) > 1.5


# ---------------------------------------------------------------- Section 3.5: key layers, compression ratio
def test_layer_mse_and_compression_ratio_by_hand():
    # two kernels of three weights with squared errors 0.03 and 0.09: MSE = 0.12 / 6 = 0.02
    assert orc.layer_mse(np.array([0.03, 0.09], np.float32), 3) == pytest.approx(0.02, rel=1e-6)
    # one layer of 10 kernels x 100 weights at 4 bits: (1000*4 + 10*32) / (1000*32) = 0.135
    assert orc.compression_ratio([10], [100], [4], [1]) == pytest.approx(0.135)
    # the same layer with two quantized tensors costs twice as much; mixed with a plain layer of equal size
    assert orc.compression_ratio([10, 10], [100, 100], [4, 4], [2, 1]) == pytest.approx(3 * 4320 / 64000)
    shapes = synth.resnet50_shapes()
    ks, ls = [s for _, s, k in shapes], [k for _, s, k in shapes]
    plain = orc.compression_ratio(ks, ls, [4] * 54, [1] * 54)
    assert plain == pytest.approx(0.12608, abs=1e-5)
    # Section 3.5, Table 3: ResNet-50 with its dual layers reads 0.1261; Table 6 reports 3.7 % dual layers = 2 of 54.
    # Doubling the two smallest layers moves the ratio by < 1e-4, doubling the two largest by ~0.02.
    order = np.argsort([s * k for _, s, k in shapes])
    nt = np.ones(54, int)
    nt[order[:2]] = 2
    assert orc.compression_ratio(ks, ls, [4] * 54, nt.tolist()) - plain < 1e-4
    nt = np.ones(54, int)
    nt[order[-2:]] = 2
    assert 0.01 < orc.compression_ratio(ks, ls, [4] * 54, nt.tolist()) - plain < 0.03


def test_algorithm_1_history_and_mixed_signedness():
    """The error after every update is non-increasing up to the grid resolution, ends at the reported error,
    and a non-negative tensor may take an unsigned first tensor with a signed residual tensor."""
    t = synth.student_t3(6 * 120, seed=77).reshape(6, 120)
    res, hist = orc.alg1_rows(t, (3, 3), (True, True), 64, 1.0, 2, n_sweeps=3)
    same = orc.residual_rows(t, (3, 3), True, 64, 1.0, 2, n_sweeps=3)
    assert np.array_equal(res.alpha, same.alpha) and np.array_equal(res.codes, same.codes)
    assert np.array_equal(hist[-1], res.sse)
    flat = hist.reshape(-1, 6)
    assert np.all(flat[1:] <= flat[:-1] * 1.05)                # each update re-solves one tensor with the rest fixed
    assert np.all(flat[-1] <= flat[1] * (1 + 1e-9))
    x = np.abs(t)
    mixed, _ = orc.alg1_rows(x, (4, 4), (False, True), 64, 1.0, 2, n_sweeps=1)
    assert mixed.codes[0].min() >= 0 and mixed.codes[0].max() <= 15 and mixed.codes[1].min() < 0
    uns, _ = orc.alg1_rows(x, (4, 4), (False, False), 64, 1.0, 2, n_sweeps=1)
    assert mixed.sse[1].sum() < uns.sse[1].sum()               # an unsigned residual tensor cannot fix negative rests
    first = orc.quantize_rows(x, 4, False, 64, 1.0, 2)
    assert np.array_equal(mixed.alpha[0], first.alpha) and np.array_equal(mixed.codes[0], first.codes)


# ---------------------------------------------------------------- Section 3.1: quantization with offset
def test_offset_quantizer_pins():
    x = synth.student_t3(4 * 150, seed=91).reshape(4, 150)
    # (a) one candidate at (max - min)/(2^p - 1) is the uniform scheme with offset of Section 3.1
    r = orc.offset_rows(x, 4, 1, 1.0 / 15, 0)
    for s in range(4):
        lo, hi = float(x[s].min()), float(x[s].max())
        assert r.delta[s] == np.float32(lo)
        assert r.alpha[s] == pytest.approx((hi - lo) / 15, rel=1e-6)
        rec = r.alpha[s].astype(np.float64) * (r.codes[s].astype(np.int64) & 0xFF) + np.float64(r.delta[s])
        assert np.max(np.abs(rec - x[s])) <= r.alpha[s] * 0.5 * (1 + 1e-5)
        assert r.codes[s].min() == 0 and r.codes[s].max() == 15
    # (b) non-negative data whose minimum is 0: the offset changes nothing
    a = np.abs(x)
    a[:, 0] = 0.0
    plain = orc.quantize_rows(a, 4, False, 128, 1.0, 3)
    off = orc.offset_rows(a, 4, 128, 1.0, 3)
    assert np.array_equal(off.alpha, plain.alpha) and np.array_equal(off.codes, plain.codes) and not off.delta.any()
    # (c) an exactly representable shift moves delta and nothing else
    g = (np.random.default_rng(4).integers(-40, 40, (3, 64)) * 2.0 ** -6).astype(np.float32)
    o1, o2 = orc.offset_rows(g, 4, 64, 1.0, 2), orc.offset_rows(g + np.float32(8.0), 4, 64, 1.0, 2)
    assert np.array_equal(o1.alpha, o2.alpha) and np.array_equal(o1.codes, o2.codes)
    assert np.array_equal(o2.delta, o1.delta + np.float32(8.0)) and np.array_equal(o1.sse, o2.sse)
    # (d) the reported error is the reconstruction error of alpha*q + delta
    o = orc.offset_rows(x, 4, 128, 1.0, 3)
    rec = o.alpha[:, None].astype(np.float64) * o.codes + o.delta[:, None].astype(np.float64)
    np.testing.assert_allclose(o.sse, np.sum((x.astype(np.float64) - rec) ** 2, axis=1), rtol=1e-5)
    # (e) for skewed data the offset beats the signed grid of the same width (the extra level of Section 3.1)
    skew = (np.abs(x) - np.float32(0.3)).astype(np.float32)
    assert orc.offset_rows(skew, 3, 128, 1.0, 3).sse.sum() < orc.quantize_rows(skew, 3, True, 128, 1.0, 3).sse.sum()


# ---------------------------------------------------------------- Section 3.4: the comparison solvers
def test_uniform_and_alternating_solvers_by_hand():
    """x = (1, 2, 3.5), signed 2-bit range {-2..1}, L = 1.  Uniform: alpha = 3.5, codes (0, 1, 1), error
    1 + 1.5^2 + 0 = 3.25.  One least-squares step: alpha = (2 + 3.5)/2 = 2.75, which re-quantizes to the
    same codes (1/2.75 = 0.36, 2/2.75 = 0.73, 3.5/2.75 = 1.27 saturates), so 2.75 is a fixed point with
    error 1 + 0.75^2 + 0.75^2 = 2.125."""
    x = np.array([[1.0, 2.0, 3.5]], np.float32)
    u = orc.solver_rows(x, orc.SOLVER_UNIFORM, bits=2)
    assert u.alpha[0] == np.float32(3.5) and u.codes.tolist() == [[0, 1, 1]] and u.sse[0] == pytest.approx(3.25)
    for n_iter in (1, 2, 9):
        a = orc.solver_rows(x, orc.SOLVER_ALTERNATING, bits=2, n_iter=n_iter)
        assert a.alpha[0] == np.float32(2.75) and a.sse[0] == pytest.approx(2.125) and a.codes.tolist() == [[0, 1, 1]]
    # unsigned 3-bit range: L = 7
    y = np.array([[0.0, 7.0, 3.0]], np.float32)
    assert orc.solver_rows(y, orc.SOLVER_UNIFORM, bits=3, is_signed=False).alpha[0] == np.float32(1.0)


def test_alternating_solver_is_monotone_and_ends_at_a_least_squares_fixed_point():
    w = synth.student_t3(8 * 200, seed=5).reshape(8, 200)
    prev = orc.solver_rows(w, orc.SOLVER_UNIFORM, bits=4).sse
    for n_iter in range(1, 30):
        cur = orc.solver_rows(w, orc.SOLVER_ALTERNATING, bits=4, n_iter=n_iter)
        assert np.all(cur.sse <= prev * (1 + 1e-12))      # each half-step solves its sub-problem exactly
        prev = cur.sse
    end, more = orc.solver_rows(w, orc.SOLVER_ALTERNATING, n_iter=200), orc.solver_rows(w, orc.SOLVER_ALTERNATING, n_iter=201)
    assert np.array_equal(end.alpha, more.alpha)
    q = end.codes.astype(np.float64)
    ls = (w.astype(np.float64) * q).sum(1) / (q * q).sum(1)
    np.testing.assert_allclose(end.alpha, ls, rtol=1e-6)   # the scale is the least-squares scale of its own codes
    # the same steps started from a grid candidate are phi's polish: one candidate at max/L, R polish steps
    one = orc.quantize_rows(w, 4, True, 1, 1.0 / 7, 5)
    alt = orc.solver_rows(w, orc.SOLVER_ALTERNATING, bits=4, n_iter=5)
    np.testing.assert_allclose(alt.alpha, one.alpha, rtol=1e-5)


def test_golden_section_first_steps_and_unimodal_case():
    rho = np.float32(0.618034)
    x = synth.laplace(300, 0.05, seed=12)
    m = np.float32(np.abs(x).max())
    # no shrink step: the two interior points of [0, m] are m - rho*m and rho*m; the better one is returned
    x1, x2 = np.float32(m - rho * m), np.float32(rho * m)
    f1, f2 = orc.sse_at(x, x1, 4, True), orc.sse_at(x, x2, 4, True)
    g0 = orc.solver_phi(x, orc.SOLVER_GOLDEN, n_iter=0)
    assert g0.alpha == (x1 if f1 <= f2 else x2) and g0.n_evals == 2
    # one shrink step keeps the half that holds the better point and adds one point inside it
    g1 = orc.solver_phi(x, orc.SOLVER_GOLDEN, n_iter=1)
    if f1 <= f2:      # bracket [0, x2]: new point x2 - rho*x2, old x1 stays
        new = np.float32(x2 - np.float32(rho * x2))
        cands = [(orc.sse_at(x, new, 4, True), new), (f1, x1)]
    else:             # bracket [x1, m]: new point x1 + rho*(m - x1), old x2 stays
        new = np.float32(x1 + np.float32(rho * np.float32(m - x1)))
        cands = [(f2, x2), (orc.sse_at(x, new, 4, True), new)]
    want = cands[0][1] if cands[0][0] <= cands[1][0] else cands[1][1]
    assert g1.alpha == want and g1.n_evals == 3
    # unimodal case with a known minimiser: every element equals v and the signed 2-bit range tops out at
    # code 1, so the error is K*(v - alpha)^2 on (0, 2v): minimum at alpha = v, inside the bracket [0, 1.5v]
    v = np.float32(0.8125)
    row = np.full(40, v, np.float32)
    for n_iter in (5, 10, 20, 30):
        g = orc.solver_phi(row, orc.SOLVER_GOLDEN, bits=2, n_iter=n_iter, hi_frac=1.5)
        width = 1.5 * float(v) * 0.618034 ** n_iter        # bracket length after n_iter steps
        assert abs(g.alpha - float(v)) <= width + 1e-6 and g.n_evals == n_iter + 2
        assert g.codes.tolist() == [1] * 40
    # never better than the exact optimum, and close to it on a smooth curve
    lo, hi = _bounds(4, True)
    for seed in range(6):
        t = synth.laplace(24, 1.0, seed=100 + seed)
        best = exact_optimum(t, lo, hi, a_max=float(np.abs(t).max()))[0]
        g = orc.solver_phi(t, orc.SOLVER_GOLDEN, n_iter=25)
        assert g.sse >= best * (1 - 1e-9)


def test_grid_search_is_the_best_of_the_four_solvers_on_average():
    """Ordering the paper's comparison reports for the MSE itself: the dense grid with polish reaches the lowest
    error; alternation from the uniform start improves on uniform but can stay in a local minimum."""
    w = np.concatenate([synth.laplace(64 * 288, 0.06, seed=3).reshape(64, 288),
                        synth.student_t3(64 * 288, seed=4).reshape(64, 288)])
    uni = orc.solver_rows(w, orc.SOLVER_UNIFORM).sse
    alt = orc.solver_rows(w, orc.SOLVER_ALTERNATING, n_iter=50).sse
    gold = orc.solver_rows(w, orc.SOLVER_GOLDEN, n_iter=25).sse
    grid = orc.quantize_rows(w, 4, True, 512, 1.0, 3).sse
    assert np.all(alt <= uni * (1 + 1e-12))
    assert grid.sum() < gold.sum() and grid.sum() < alt.sum() < uni.sum()
    assert np.mean(grid <= np.minimum(alt, gold) * (1 + 1e-3)) > 0.9
    assert np.any(grid < alt * 0.99)                      # alternation stuck in a local minimum somewhere


# ---------------------------------------------------------------- Section 3.1: offset and scale both searched
def test_affine_search_pins():
    x = synth.student_t3(5 * 96, seed=17).reshape(5, 96)
    # (a) a single offset on the grid is delta = min: the offset scheme
    one = orc.affine_rows(x, 4, 64, 1.0, n_delta=1, off_frac=0.25, refine_iters=2)
    off = orc.offset_rows(x, 4, 64, 1.0, 2)
    assert np.array_equal(one.alpha, off.alpha) and np.array_equal(one.codes, off.codes)
    assert np.array_equal(one.delta, off.delta) and np.array_equal(one.best_idx, off.best_idx)
    # (b) delta = min stays on the grid (d = 0), so more offsets can only lower the grid error
    g1 = orc.affine_rows(x, 4, 64, 1.0, n_delta=1, refine_iters=0)
    g8 = orc.affine_rows(x, 4, 64, 1.0, n_delta=8, off_frac=0.25, refine_iters=0)
    assert np.all(g8.sse <= g1.sse) and np.any(g8.sse < g1.sse * 0.9)     # heavy tails: clipping the low end pays
    assert np.all(g8.best_idx // 64 < 8) and np.all(g8.delta >= x.min(1))
    # (c) brute force over the whole (offset, scale) grid with shifted rows built here
    for s in range(5):
        lo, hi = np.float32(x[s].min()), np.float32(x[s].max())
        dstep = np.float32(np.float32(np.float32(0.25) * np.float32(hi - lo)) / np.float32(8))
        best = (np.inf, -1)
        for d in range(8):
            r = (x[s] - np.float32(lo + np.float32(np.float32(d) * dstep))).astype(np.float32)
            m = float(np.abs(r).max())
            for c in range(64):
                e = orc.sse_at(r, orc.candidate(m, 1.0, 64, c), 4, False)
                if e < best[0]:
                    best = (e, d * 64 + c)
        assert g8.best_idx[s] == best[1] and g8.sse[s] == pytest.approx(best[0], rel=1e-12)
        d = best[1] // 64
        assert g8.delta[s] == np.float32(lo + np.float32(np.float32(d) * dstep))
    a, dl, sse, idx, codes, curve = orc.affine_phi(x[0], 4, 64, 1.0, 8, 0.25, 0, want_curve=True)
    assert idx == int(np.argmin(curve.reshape(-1))) and sse == pytest.approx(curve.reshape(-1)[idx], rel=1e-12)
    # (d) an exactly representable shift moves delta and nothing else
    g = (np.random.default_rng(9).integers(-60, 60, (3, 80)) * 2.0 ** -6).astype(np.float32)
    o1 = orc.affine_rows(g, 4, 32, 1.0, 4, 0.25, 2)
    o2 = orc.affine_rows(g + np.float32(4.0), 4, 32, 1.0, 4, 0.25, 2)
    assert np.array_equal(o1.alpha, o2.alpha) and np.array_equal(o1.codes, o2.codes)
    assert np.array_equal(o2.delta, o1.delta + np.float32(4.0)) and np.array_equal(o1.best_idx, o2.best_idx)
    # (e) the reported error is the reconstruction error of alpha*q + delta, codes in the unsigned range
    full = orc.affine_rows(x, 4, 64, 1.0, 8, 0.25, 3)
    rec = full.alpha[:, None].astype(np.float64) * full.codes + full.delta[:, None].astype(np.float64)
    np.testing.assert_allclose(full.sse, np.sum((x.astype(np.float64) - rec) ** 2, axis=1), rtol=1e-4)
    assert full.codes.min() >= 0 and full.codes.max() <= 15
    # (f) per offset, the grid stays within the grid-resolution bound of the exact optimum for that offset
    lo4, hi4 = _bounds(4, False)
    t = synth.laplace(20, 1.0, seed=44)
    a, dl, sse, idx, codes, curve = orc.affine_phi(t, 4, 64, 1.0, 4, 0.25, 0, want_curve=True)
    tmin, tmax = np.float32(t.min()), np.float32(t.max())
    dstep = np.float32(np.float32(np.float32(0.25) * np.float32(tmax - tmin)) / np.float32(4))
    for d in range(4):
        r = (t - np.float32(tmin + np.float32(np.float32(d) * dstep))).astype(np.float32)
        m = float(np.abs(r).max())
        e_star, a_star, q_star = exact_optimum(r, lo4, hi4, a_max=m)
        step = m / 64
        assert curve[d].min() >= e_star * (1 - 1e-9)
        assert np.sqrt(curve[d].min()) <= np.sqrt(e_star) + 0.5 * step * np.linalg.norm(q_star) * (1 + 1e-6)


# ---------------------------------------------------------------- Section 3.5: Algorithm 1's while-condition
def test_algorithm_1_stops_when_the_error_stops_moving():
    t = synth.student_t3(10 * 160, seed=23).reshape(10, 160)
    fixed, hist_fixed = orc.alg1_rows(t, (3, 3), (True, True), 64, 1.0, 2, n_sweeps=6)
    # eps = -1 in the C function is the fixed count; a huge eps stops after the first sweep
    one, h1, d1 = orc.alg1_rows_eps(t, (3, 3), (True, True), 64, 1.0, 2, max_sweeps=6, eps=10.0)
    first, _ = orc.alg1_rows(t, (3, 3), (True, True), 64, 1.0, 2, n_sweeps=1)
    assert np.all(d1 == 1) and np.array_equal(one.alpha, first.alpha) and np.array_equal(one.codes, first.codes)
    assert np.array_equal(h1[0], first.sse) and np.array_equal(h1[5], first.sse)    # later entries repeat the last error
    # a moderate eps: every row stops exactly at the first sweep whose relative decrease is <= eps
    eps = 0.02
    res, hist, done = orc.alg1_rows_eps(t, (3, 3), (True, True), 64, 1.0, 2, max_sweeps=6, eps=eps)
    e0 = np.sum(t.astype(np.float64) ** 2, axis=1)
    assert done.min() >= 1 and done.max() <= 6 and len(set(done.tolist())) > 1
    for s in range(10):
        ends = np.concatenate([[e0[s]], hist_fixed[:, -1, s]])            # error after sweep 0 (nothing), 1, 2, ...
        rate = (ends[:-1] - ends[1:]) / ends[:-1]
        stop = next((i + 1 for i, r in enumerate(rate) if not r > eps), 6)
        assert done[s] == stop
        n = done[s]
        assert np.array_equal(hist[:n, :, s], hist_fixed[:n, :, s])       # the sweeps that ran are the fixed-count ones
        ref_n, _ = orc.alg1_rows(t[s:s + 1], (3, 3), (True, True), 64, 1.0, 2, n_sweeps=int(n))
        assert np.array_equal(res.alpha[:, s], ref_n.alpha[:, 0]) and np.array_equal(res.codes[:, s], ref_n.codes[:, 0])
    # eps = 0 runs until a sweep brings no decrease at all (or the cap)
    z, hz, dz = orc.alg1_rows_eps(t, (3, 3), (True, True), 64, 1.0, 2, max_sweeps=6, eps=0.0)
    assert np.all(dz >= done)


def test_key_layer_pipeline_marks_by_tau_and_counts_the_second_tensor():
    layers = [synth.laplace(16 * 72, 0.05, seed=1).reshape(16, 72), synth.student_t3(8 * 200, seed=2).reshape(8, 200),
              synth.laplace(32 * 27, 0.3, seed=3).reshape(32, 27)]
    probe = orc.key_layer_pipeline(layers, 4, True, 64, 1.0, 2, tau=0.0)
    assert probe.is_key.all() and set(probe.second) == {0, 1, 2}
    tau = float(np.sort(probe.mse)[1])                 # exactly one layer lies strictly above the middle MSE
    out = orc.key_layer_pipeline(layers, 4, True, 64, 1.0, 2, tau=tau)
    assert out.is_key.sum() == 1 and out.is_key[int(np.argmax(probe.mse))]
    l = int(np.argmax(probe.mse))
    assert np.array_equal(out.second[l].alpha[0], out.first[l].alpha)     # first tensor unchanged by the second pass
    assert np.all(out.second[l].sse[1] <= out.second[l].sse[0])
    n = [w.size for w in layers]
    s = [w.shape[0] for w in layers]
    want = sum((2 if i == l else 1) * (4 * n[i] + 32 * s[i]) for i in range(3)) / (32.0 * sum(n))
    assert out.compression_ratio == pytest.approx(want, rel=1e-12)


@pytest.mark.parametrize("lo1,hi1,lo2,hi2", [(-8, 7, -8, 7), (-4, 3, -8, 7), (0, 15, 0, 15), (-2, 1, -128, 127), (-8, 7, -2, 1)])
def test_dual_first_code_window_holds_the_minimum(lo1, hi1, lo2, hi2):
    """Section 3.5's dual objective min_t (x - a1*t - a2*[(x - a1*t)/a2]_Zp2)^2, enumerated over every first code,
    equals the minimum over the first codes within (max|Z_p2| + 1/2)*a2/a1 + 1/2 (at least 1) of round(x/a1), with
    codes beyond Z_p1 moved to its ends: the property the library's restricted enumeration relies on.  Brute force in
    fp64 over random values, scales from far narrower to wider than a step of the first grid, values in and out of range."""
    rng = np.random.default_rng(77)
    n = 60_000
    a1 = rng.uniform(0.05, 2.0, n)
    rho = np.exp(rng.uniform(np.log(0.004), np.log(3.0), n))
    a2 = a1 * rho
    x = rng.uniform(-1.6, 1.6, n) * a1 * max(hi1, -lo1)
    half = max(hi2, -lo2) + 0.5

    def err(t):
        r = x - a1 * t
        q = np.clip(np.rint(r / a2), lo2, hi2)
        return np.abs(r - a2 * q)

    full = np.min(np.stack([err(np.full(n, float(t))) for t in range(lo1, hi1 + 1)]), axis=0)
    w = np.maximum(1, np.floor(half * np.minimum(rho, 16.0) * 1.0001 + 0.501)).astype(int)
    t0 = np.rint(x / a1)
    win = np.full(n, np.inf)
    for s in range(-int(w.max()), int(w.max()) + 1):
        t = np.clip(t0 + s, lo1, hi1)
        e = np.where(np.abs(s) <= w, err(t), np.inf)
        win = np.minimum(win, e)
    assert np.all(win >= full)                       # a subset cannot do better
    assert np.allclose(win, full, rtol=0, atol=1e-12)
