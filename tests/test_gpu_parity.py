"""GPU parity: the CUDA library, called through its C interface, against the CPU oracle."""
import numpy as np
import pytest

from oracle import omse_oracle as orc
from paper_1902_06822_b200 import synth
from parity import RTOL, check_rows

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    import gpu_util
    return gpu_util


def _run_and_check(gpu, w, bits, signed, n_cand, refine, hi_frac=1.0, codes=True, packed=False, rows=None):
    alpha, sse, idx, q, pk = gpu.quantize_weights(w, bits, signed, n_cand, hi_frac, refine, codes, packed)
    stats = check_rows(w, alpha, sse, idx, q, pk, bits, signed, n_cand, hi_frac, refine, rows=rows)
    assert stats["idx_diff"] <= max(1, stats["rows"] // 100), stats
    assert stats["alpha_bitwise"] >= 0.99, stats
    return stats


# ---------------------------------------------------------------- configs[0]: one convolution layer
def test_single_conv_layer_config(gpu):
    w = synth.conv_layer(seed=1)
    _run_and_check(gpu, w, 4, True, 256, 3, codes=True, packed=True)
    _run_and_check(gpu, w, 4, True, 256, 0, codes=True, packed=False)


# ---------------------------------------------------------------- shapes: several tiles, ragged tails
@pytest.mark.parametrize("k", [1, 2, 3, 5, 27, 31, 32, 33, 64, 147, 255, 576, 1000, 4608])
def test_kernel_lengths_with_odd_row_counts(gpu, k):
    s = 37 if k < 2000 else 9
    w = synth.student_t3(s * k, seed=50 + k, tensor_id=k).reshape(s, k)
    _run_and_check(gpu, w, 4, True, 256, 3, codes=True, packed=True)


@pytest.mark.parametrize("n_cand", [1, 16, 50, 64, 100, 128, 500, 1024, 2048, 4096])
def test_candidate_counts(gpu, n_cand):
    w = synth.laplace(21 * 300, 0.05, seed=60, tensor_id=n_cand).reshape(21, 300)
    _run_and_check(gpu, w, 4, True, n_cand, 3, codes=True, packed=True)


@pytest.mark.parametrize("bits,signed", [(2, True), (3, True), (4, True), (8, True), (2, False), (4, False), (8, False)])
def test_bit_widths_and_signedness(gpu, bits, signed):
    w = synth.student_t3(33 * 576, seed=70, tensor_id=bits).reshape(33, 576)
    if not signed and bits != 4:
        w = np.abs(w)          # unsigned grid on non-negative data; bits == 4 keeps the negatives
    _run_and_check(gpu, w, bits, signed, 1024, 3, codes=True, packed=bits <= 4)


def test_hi_frac_other_than_one_and_packed_only(gpu):
    w = synth.laplace(40 * 147, 0.02, seed=80).reshape(40, 147)
    _run_and_check(gpu, w, 4, True, 256, 2, hi_frac=1.0 / 7, codes=True, packed=True)
    _run_and_check(gpu, w, 4, True, 256, 2, hi_frac=0.5, codes=False, packed=True)
    _run_and_check(gpu, w, 3, True, 64, 1, codes=False, packed=False)


def test_large_rows_span_element_groups(gpu):
    w = synth.sweep_tensor(25088, seed=5, n_kernels=6)
    _run_and_check(gpu, w, 4, True, 1024, 3, codes=True, packed=True)
    w = synth.sweep_tensor(28672, seed=6, n_kernels=3)
    _run_and_check(gpu, w, 2, True, 1024, 3, codes=True, packed=True)


# ---------------------------------------------------------------- degenerate and invalid inputs
def test_zero_rows_non_finite_values_and_status_word(gpu):
    w = synth.laplace(8 * 64, 0.02, seed=90).reshape(8, 64).copy()
    w[2] = 0.0
    w[5, 3] = np.nan
    w[6] = 1e-42          # every candidate below FLT_MIN
    gpu.ctx().omse_last_device_status()
    alpha, sse, idx, q, pk = gpu.quantize_weights(w, 4, True, 256, 1.0, 3, True, True)
    st = gpu.ctx().omse_last_device_status()
    assert st & 1 and st & 2
    for r in (2, 6):
        assert alpha[r] == 0.0 and idx[r] == -1 and not q.reshape(8, 64)[r].any()
    assert sse[2] == 0.0
    assert q.min() >= -8 and q.max() <= 7
    good = [0, 1, 3, 4, 7]
    check_rows(w, alpha, sse, idx, q, None, 4, True, 256, 1.0, 3, rows=good)
    assert gpu.ctx().omse_last_device_status() == 0


def test_invalid_arguments_are_rejected(gpu):
    import torch
    from paper_1902_06822_b200 import binding
    c = gpu.ctx()
    w = torch.zeros(64, device="cuda")
    a = torch.zeros(8, device="cuda")
    s = torch.zeros(8, device="cuda")
    pk = torch.zeros(32, dtype=torch.uint8, device="cuda")
    bad = [
        dict(bits=1), dict(bits=9), dict(n_cand=0), dict(n_cand=4097), dict(hi_frac=0.0), dict(refine_iters=-1),
        dict(kernel_len=0), dict(kernel_len=binding.MAX_KERNEL_LEN + 1), dict(n_kernels=-1), dict(bits=8, packed=pk),
    ]
    for kw in bad:
        args = dict(w=w, n_kernels=8, kernel_len=8, bits=4, is_signed=True, n_cand=16, hi_frac=1.0, refine_iters=1,
                    alpha=a, sse=s, packed=None)
        args.update(kw)
        with pytest.raises(binding.OmseError) as e:
            c.omse_quantize_weights(**args)
        assert e.value.code == binding.EINVAL, kw
    with pytest.raises(binding.OmseError):
        c.omse_residual_quantize(w, 8, 8, [4, 4], True, 16, 1.0, 1, 2, a, s, None, None)   # sweeps > 1 need codes
    with pytest.raises(binding.OmseError):
        c.omse_residual_quantize(w, 8, 8, [4] * 5, True, 16, 1.0, 1, 1, a, s, None, None)
    c.omse_quantize_weights(w, 0, 8, 4, True, 16, 1.0, 1, a, s)     # empty input: nothing to do
    torch.cuda.synchronize()


# ---------------------------------------------------------------- INT4 emission
@pytest.mark.parametrize("n", [0, 1, 2, 15, 16, 17, 4097, 1 << 20, (1 << 20) + 3])
def test_pack_int4_matches_oracle(gpu, n):
    import torch
    rng = np.random.default_rng(n)
    q = rng.integers(-8, 8, size=max(n, 1), dtype=np.int8)[:n]
    d_q = torch.from_numpy(q).cuda() if n else torch.zeros(1, dtype=torch.int8, device="cuda")
    d_p = torch.full(((n + 1) // 2 + 1,), 0xEE, dtype=torch.uint8, device="cuda")
    gpu.ctx().omse_pack_int4(d_q, n, True, d_p)
    torch.cuda.synchronize()
    out = d_p.cpu().numpy()
    assert out[-1] == 0xEE                                  # nothing written past the end
    assert np.array_equal(out[:-1], orc.pack_int4(q))
    if n > 16:                                              # unaligned views take the byte path
        gpu.ctx().omse_pack_int4(d_q[1:], n - 1, True, d_p[1:])
        torch.cuda.synchronize()
        assert np.array_equal(d_p.cpu().numpy()[1:1 + n // 2], orc.pack_int4(q[1:]))


# ---------------------------------------------------------------- Section 3.7: per-tensor scale
def _check_activation(gpu, x, bits, signed, n_cand, refine):
    alpha, sse, idx, curve = gpu.activation_scale(x, bits, signed, n_cand, 1.0, refine)
    ref = orc.activation_scale(x, bits, signed, n_cand, 1.0, refine)
    finite = np.isfinite(ref.sse_curve)
    assert np.array_equal(finite, np.isfinite(curve))
    np.testing.assert_allclose(curve[finite], ref.sse_curve[finite], rtol=2e-6)
    if idx != ref.best_idx:
        assert abs(ref.sse_curve[idx] - ref.sse_curve[ref.best_idx]) <= 1e-6 * ref.sse_curve[ref.best_idx]
        ref = orc.phi(x, bits, signed, n_cand, 1.0, refine, start_idx=idx, want_codes=False)
    assert alpha == pytest.approx(ref.alpha, rel=RTOL)
    assert sse == pytest.approx(ref.sse, rel=RTOL)
    return idx == ref.best_idx


@pytest.mark.parametrize("n", [1, 3, 4, 1000, 4096, 4097, 300_001, 2_000_000])
def test_activation_scale_sizes(gpu, n):
    x = synth.relu_activations(n, seed=3, tensor_id=n % 97)
    if n <= 4:
        x = x + np.float32(0.25)
    assert _check_activation(gpu, x, 4, False, 2048 if n > 1000 else 256, 3)


@pytest.mark.parametrize("bits,signed,n_cand", [(4, True, 50), (8, False, 500), (2, False, 64), (3, True, 4096),
                                                (4, False, 600), (4, True, 1100), (3, False, 1500), (4, False, 3000),
                                                (4, False, 33), (4, True, 129), (2, True, 700), (8, True, 2049)])
def test_activation_scale_grids(gpu, bits, signed, n_cand):
    """Every block shape of the per-tensor sweep: the thread count follows the candidate count (160 ... 512)."""
    x = synth.student_t3(250_000, seed=33, tensor_id=bits)
    if not signed:
        x = np.abs(x)
    _check_activation(gpu, x, bits, signed, n_cand, 2)


@pytest.mark.parametrize("neg_outlier", [False, True])
def test_activation_scale_unsigned_grid_on_signed_values(gpu, neg_outlier):
    """A grid that starts at 0 codes every negative value as 0 whatever the scale; values at the edge of the range of
    the smallest scales saturate.  With the outlier the negative side sets the grid's range."""
    x = synth.student_t3(300_001, seed=41, tensor_id=7)
    if neg_outlier:
        x[1234] = np.float32(-3.0) * np.abs(x).max()
    _check_activation(gpu, x, 4, False, 2048, 3)
    _check_activation(gpu, x, 3, False, 256, 1)


def test_activation_scale_degenerate(gpu):
    gpu.ctx().omse_last_device_status()
    alpha, sse, idx, curve = gpu.activation_scale(np.zeros(5000, np.float32), 4, False, 128, 1.0, 3)
    assert (alpha, sse, idx) == (0.0, 0.0, -1) and gpu.ctx().omse_last_device_status() & 2


# ---------------------------------------------------------------- Sections 3.5 / 3.7: residual, Algorithm 1
def _residual_step_by_step(gpu, t, bits, n_cand, refine, packed=False):
    alpha, sse, q, pk = gpu.residual_quantize(t, bits, True, n_cand, 1.0, refine, 1, True, packed)
    S, K = t.shape
    r = t.copy()
    for j, b in enumerate(bits):
        st = check_rows(r, alpha[j], sse[j], None, q[j], pk[j] if packed else None, b, True, n_cand, 1.0, refine)
        assert st["alpha_bitwise"] >= 0.99
        # next residual exactly as defined: one binary32 rounding of r - alpha*q per element
        r = (r.astype(np.float64) - alpha[j][:, None].astype(np.float64) * q[j].reshape(S, K)).astype(np.float32)
    assert np.all(sse[1] <= sse[0])
    return alpha, sse, q


def test_residual_two_tensors_small(gpu):
    t = synth.laplace_with_outliers(30 * 500, 0.005, seed=4, outlier_prob=0.01).reshape(30, 500)
    _residual_step_by_step(gpu, t, (4, 4), 256, 3, packed=True)
    t = synth.student_t3(15 * 147, seed=41).reshape(15, 147)
    _residual_step_by_step(gpu, t, (4, 2, 3), 128, 2, packed=True)


def test_algorithm_1_two_sweeps_matches_oracle(gpu):
    t = synth.student_t3(12 * 300, seed=21).reshape(12, 300)
    alpha, sse, q, _ = gpu.residual_quantize(t, (3, 3), True, 128, 1.0, 2, n_sweeps=2)
    ref = orc.residual_rows(t, (3, 3), True, 128, 1.0, 2, n_sweeps=2)
    np.testing.assert_allclose(alpha, ref.alpha, rtol=RTOL)
    np.testing.assert_allclose(sse, ref.sse, rtol=RTOL)
    same = np.all(alpha == ref.alpha, axis=0)
    assert same.mean() >= 0.9
    assert np.array_equal(q.reshape(2, 12, 300)[:, same], ref.codes[:, same])


# ---------------------------------------------------------------- several tensors in one launch
def test_batched_launch_matches_per_tensor_results(gpu):
    import torch
    shapes = [(7, 147), (33, 64), (5, 4608), (0, 32), (64, 576), (19, 27), (3, 1000)]
    hosts, descs = [], []
    for i, (s, k) in enumerate(shapes):
        w = synth.laplace(max(s * k, 1), 0.05, seed=300, tensor_id=i)[:s * k].reshape(s, k)
        hosts.append(w)
        descs.append(dict(w=torch.from_numpy(np.ascontiguousarray(w)).cuda() if s else torch.zeros(1, device="cuda"),
                          n_kernels=s, kernel_len=k,
                          alpha=torch.full((max(s, 1),), -1.0, device="cuda"),
                          sse=torch.full((max(s, 1),), -1.0, device="cuda"),
                          best_idx=torch.full((max(s, 1),), -7, dtype=torch.int32, device="cuda"),
                          codes=torch.full((max(s * k, 1),), 99, dtype=torch.int8, device="cuda"),
                          packed=torch.full(((s * k + 1) // 2 + 1,), 0xAB, dtype=torch.uint8, device="cuda")))
    gpu.ctx().omse_quantize_weights_batched(descs, 4, True, 1024, 1.0, 3)
    torch.cuda.synchronize()
    for w, d in zip(hosts, descs):
        s, k = w.shape
        if s == 0:
            continue
        pk = d["packed"].cpu().numpy()
        assert pk[-1] == 0xAB
        check_rows(w, d["alpha"].cpu().numpy(), d["sse"].cpu().numpy(), d["best_idx"].cpu().numpy(),
                   d["codes"].cpu().numpy(), pk[:-1], 4, True, 1024, 1.0, 3)
        one = gpu.quantize_weights(w, 4, True, 1024, 1.0, 3, True, True)   # same call, tensor by tensor
        assert np.array_equal(one[0], d["alpha"].cpu().numpy()) and np.array_equal(one[3], d["codes"].cpu().numpy())
    # the dispenser is back at zero: a second launch on the same context gives the same answer
    before = descs[2]["alpha"].clone()
    gpu.ctx().omse_quantize_weights_batched(descs, 4, True, 1024, 1.0, 3)
    torch.cuda.synchronize()
    assert torch.equal(before, descs[2]["alpha"])


# ---------------------------------------------------------------- magnitude-class regrouping (long and short rows)
@pytest.mark.parametrize("n_cand", [1, 16, 50, 100, 256, 500, 1024, 2048, 4096])
def test_long_rows_regrouped_for_every_candidate_layout(gpu, n_cand):
    """Rows of 1024+ elements are regrouped by magnitude class; every candidates-per-thread layout."""
    w = synth.student_t3(5 * 1500, seed=400, tensor_id=n_cand).reshape(5, 1500)
    _run_and_check(gpu, w, 4, True, n_cand, 3, codes=True, packed=True)
    w = synth.laplace(3 * 9000, 0.01, seed=401, tensor_id=n_cand).reshape(3, 9000)     # several element groups
    _run_and_check(gpu, w, 3, True, n_cand, 2, codes=True, packed=False)


@pytest.mark.parametrize("k", [1025, 1026, 1027, 2051, 8193, 8195, 14001])
def test_long_rows_of_ragged_length(gpu, k):
    """Block-per-row path on rows whose length is not a multiple of four: the per-element passes walk the row four
    elements at a time and rely on its zero padding; both block sizes (rows below and above 8192 elements)."""
    s = 7
    w = synth.student_t3(s * k, seed=410, tensor_id=k).reshape(s, k)
    _run_and_check(gpu, w, 4, True, 1024, 3, codes=True, packed=True)
    _run_and_check(gpu, np.abs(w), 3, False, 256, 1, codes=True, packed=True)


@pytest.mark.parametrize("k", [192, 193, 256, 500, 640])
def test_short_rows_regrouped_in_large_launches(gpu, k):
    """Enough short rows for the batched short-row path, with regrouping (192 <= K <= 640)."""
    s = 2500
    w = synth.laplace(s * k, 0.03, seed=410, tensor_id=k).reshape(s, k)
    _run_and_check(gpu, w, 4, True, 1024, 3, codes=True, packed=True, rows=np.arange(0, s, 7))
    _run_and_check(gpu, np.abs(w), 4, False, 1024, 1, codes=False, packed=False, rows=np.arange(3, s, 11))


def test_regrouping_corner_cases(gpu):
    k = 2048
    rng = np.random.default_rng(7)
    rows = [
        np.full(k, 0.37, np.float32),                                   # one magnitude: a single class
        np.where(np.arange(k) % 2 == 0, 1.0, -1.0).astype(np.float32),  # +-max only
        np.concatenate([[5.0], np.full(k - 1, 1e-6)]).astype(np.float32),   # one large element, rest below step/2
        np.concatenate([[5.0], np.zeros(k - 1)]).astype(np.float32),    # one element, exact zeros
        (rng.integers(-8, 8, k) * 0.125).astype(np.float32),            # already on a grid
        np.linspace(-1.0, 1.0, k).astype(np.float32),                   # every class populated
        (np.linspace(0.0, 1.0, k) ** 8).astype(np.float32),             # heavy concentration near zero
    ]
    w = np.stack(rows)
    for bits, signed in [(4, True), (2, True), (8, True), (4, False), (3, False)]:
        _run_and_check(gpu, w, bits, signed, 1024, 3, codes=True, packed=bits <= 4)
    _run_and_check(gpu, w, 4, True, 1024, 3, hi_frac=1.0 / 7, codes=True, packed=True)     # grid far below max|x|
    _run_and_check(gpu, w, 4, True, 1024, 3, hi_frac=2.0, codes=True, packed=True)         # grid beyond max|x|


def test_residual_on_regrouped_long_rows(gpu):
    t = synth.laplace_with_outliers(6 * 3000, 0.005, seed=420, outlier_prob=0.005).reshape(6, 3000)
    _residual_step_by_step(gpu, t, (4, 4), 1024, 3, packed=True)
    alpha, sse, q, _ = gpu.residual_quantize(t, (4, 3), True, 512, 1.0, 2, n_sweeps=2)
    ref = orc.residual_rows(t, (4, 3), True, 512, 1.0, 2, n_sweeps=2)
    np.testing.assert_allclose(alpha, ref.alpha, rtol=RTOL)
    np.testing.assert_allclose(sse, ref.sse, rtol=RTOL)


# ---------------------------------------------------------------- seeded random configurations
@pytest.mark.parametrize("seed", range(24))
def test_random_configurations(gpu, seed):
    """Random shapes, grids, bit widths and value distributions (seeded): every launch path gets hit."""
    rng = np.random.default_rng(1000 + seed)
    k = int(rng.choice([3, 17, 27, 64, 100, 147, 200, 333, 576, 640, 641, 1023, 1024, 2000, 4608, 9000]))
    max_rows = max(2, min(4000, 600_000 // k))
    s = int(rng.integers(1, max_rows))
    n_cand = int(rng.choice([7, 32, 50, 64, 128, 256, 500, 1024, 1024, 1024, 2048, 4096]))
    bits = int(rng.choice([2, 3, 4, 4, 8]))
    signed = bool(rng.integers(0, 2))
    refine = int(rng.integers(0, 4))
    hi_frac = float(rng.choice([1.0, 1.0, 0.5, 1.0 / 7, 1.5]))
    kind = int(rng.integers(0, 4))
    if kind == 0:
        w = synth.laplace(s * k, 0.02, seed=2000 + seed).reshape(s, k)
    elif kind == 1:
        w = synth.student_t3(s * k, seed=2000 + seed).reshape(s, k)
    elif kind == 2:
        w = synth.relu_activations(s * k, seed=2000 + seed, zero_prob=0.6).reshape(s, k)
    else:
        w = synth.laplace_with_outliers(s * k, 0.005, seed=2000 + seed, outlier_prob=0.01).reshape(s, k)
    if not signed and kind != 2 and seed % 2:
        w = np.abs(w)
    packed = bits <= 4
    rows = None if s * k * n_cand < 3e8 else np.unique(rng.integers(0, s, 300))
    alpha, sse, idx, q, pk = gpu.quantize_weights(w, bits, signed, n_cand, hi_frac, refine, True, packed)
    st = check_rows(w, alpha, sse, idx, q, pk if rows is None else None, bits, signed, n_cand, hi_frac, refine, rows=rows)
    assert st["idx_diff"] <= max(1, st["rows"] // 50) and st["alpha_bitwise"] >= 0.98, st
    if pk is not None:
        assert np.array_equal(pk, orc.pack_int4(q))


def test_algorithm_1_history_and_mixed_signedness_match_oracle(gpu):
    import torch
    t = np.abs(synth.student_t3(10 * 1200, seed=88)).reshape(10, 1200)
    S, K = t.shape
    d_t = torch.from_numpy(t).cuda()
    alpha = torch.empty(2, S, device="cuda")
    sse = torch.empty(2, S, device="cuda")
    hist = torch.full((3, 2, S), -1.0, device="cuda")
    codes = torch.empty(2, S * K, dtype=torch.int8, device="cuda")
    gpu.ctx().omse_alg1_quantize(d_t, S, K, [4, 3], [False, True], 256, 1.0, 2, 3, alpha, sse, hist, codes)
    torch.cuda.synchronize()
    ref, ref_hist = orc.alg1_rows(t, (4, 3), (False, True), 256, 1.0, 2, n_sweeps=3)
    np.testing.assert_allclose(alpha.cpu().numpy(), ref.alpha, rtol=RTOL)
    np.testing.assert_allclose(sse.cpu().numpy(), ref.sse, rtol=RTOL)
    np.testing.assert_allclose(hist.cpu().numpy(), ref_hist, rtol=RTOL)
    same = np.all(alpha.cpu().numpy() == ref.alpha, axis=0)
    assert same.mean() >= 0.8
    q = codes.cpu().numpy().reshape(2, S, K)
    assert np.array_equal(q[:, same], ref.codes[:, same])
    assert q[0].min() >= 0 and q[1].min() < 0
    assert torch.equal(hist[-1], sse)


# ---------------------------------------------------------------- very short rows in large numbers: a thread per row
@pytest.mark.parametrize("k,bits,signed", [(1, 4, True), (2, 4, True), (3, 2, True), (9, 4, False), (17, 3, True),
                                           (27, 4, True), (27, 2, True), (28, 8, True), (32, 4, True), (31, 4, False)])
def test_very_short_rows_thread_per_row_path(gpu, k, bits, signed):
    s = 9600 + 37                                  # at least 64 rows per SM; the last unit is ragged
    w = synth.student_t3(s * k, seed=900 + k, tensor_id=bits).reshape(s, k)
    if not signed and k != 31:
        w = np.abs(w)
    w[5] = 0.0                                     # a degenerate row inside a unit
    rows = np.unique(np.concatenate([np.arange(0, s, 13), [5, s - 1, s - 2, 127, 128, 129]]))
    alpha, sse, idx, q, pk = gpu.quantize_weights(w, bits, signed, 1024, 1.0, 3, True, bits <= 4)
    good = rows[rows != 5]
    st = check_rows(w, alpha, sse, idx, q, None, bits, signed, 1024, 1.0, 3, rows=good)
    assert st["idx_diff"] <= max(1, st["rows"] // 50) and st["alpha_bitwise"] >= 0.98, st
    assert alpha[5] == 0.0 and idx[5] == -1 and not q.reshape(s, k)[5].any()
    if pk is not None:
        assert np.array_equal(pk, orc.pack_int4(q))
    lo, hi = (-(1 << (bits - 1)), (1 << (bits - 1)) - 1) if signed else (0, (1 << bits) - 1)
    assert q.astype(np.int16).min() >= (lo if signed or bits < 8 else -128)


def test_non_finite_and_zero_rows_on_every_launch_path(gpu):
    """NaN / Inf / all-zero / denormal rows never fault and never disturb their neighbours, whichever path
    (long regrouped rows, batched short rows, thread-per-row) the launch takes."""
    for s, k in [(12, 3000), (2600, 256), (9700, 27)]:
        w = synth.laplace(s * k, 0.02, seed=950 + k).reshape(s, k).copy()
        w[1] = 0.0
        w[3, k // 2] = np.nan
        w[5, 0] = np.inf
        w[7] = 1e-42
        gpu.ctx().omse_last_device_status()
        alpha, sse, idx, q, pk = gpu.quantize_weights(w, 4, True, 1024, 1.0, 3, True, True)
        st = gpu.ctx().omse_last_device_status()
        assert st & 1 and st & 2
        for r in (1, 3, 5, 7):
            assert alpha[r] == 0.0 and idx[r] == -1 and not q.reshape(s, k)[r].any(), (k, r)
        assert sse[1] == 0.0
        assert q.min() >= -8 and q.max() <= 7
        good = np.array([0, 2, 4, 6, 8, 9, 10, 11, s - 1])
        check_rows(w, alpha, sse, idx, q, None, 4, True, 1024, 1.0, 3, rows=good)
        assert np.array_equal(pk, orc.pack_int4(q))
