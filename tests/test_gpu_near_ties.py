"""GPU parity where many candidate scales have (almost) the same error.

The library compares candidates by binary32 sums and then re-scores, in binary64 with the IEEE division,
every candidate whose sum lies within a narrow band of the smallest one; the winner must be the oracle's
(lowest index among equal errors) however many candidates fall into that band.  Two kinds of input:

* exact ties by construction: values in {0, +-a} with a = C * 2^-12, so that every scale a/j on the grid
  (j a divisor of C, j within the code range) reproduces the row exactly - dozens of candidates with error 0;
* near ties of natural data: sparse heavy-tailed rows on a grid so fine (hi_frac just above the optimum)
  that twenty-odd neighbouring candidates agree to a few parts per million.
"""
import numpy as np
import pytest

from oracle import omse_oracle as orc
from paper_1902_06822_b200 import synth
from parity import RTOL, check_rows

pytestmark = pytest.mark.gpu

C_TIES = 2520                      # 1..10 | 2520: 34 divisors up to 127, 39 up to 255
A_TIES = np.float32(C_TIES * 2.0 ** -12)   # step = 2^-12 exactly, every candidate exact in binary32


@pytest.fixture(scope="module")
def gpu():
    import gpu_util
    return gpu_util


def _tie_rows(s, k, seed, signed=True):
    rng = np.random.default_rng(seed)
    pick = rng.integers(-1 if signed else 0, 2, size=(s, k))
    w = (pick * A_TIES).astype(np.float32)
    w[:, 0] = A_TIES                       # the row maximum is a
    return w


def _divisors(limit):
    return [j for j in range(1, limit + 1) if C_TIES % j == 0]


@pytest.mark.parametrize("s,k", [(5, 2048), (3, 9000), (2500, 256), (2500, 64), (9700, 27), (6, 300)])
def test_exact_ties_beyond_any_list_on_every_row_path(gpu, s, k):
    """34 candidates with error exactly 0 on every row; long regrouped rows, element groups, batched short
    rows (with and without regrouping), thread-per-row and plain block-per-row paths."""
    assert len(_divisors(127)) == 34
    w = _tie_rows(s, k, seed=k)
    rows = None if s <= 10 else np.unique(np.concatenate([np.arange(0, s, 41), [s - 1]]))
    alpha, sse, idx, q, pk = gpu.quantize_weights(w, 8, True, C_TIES, 1.0, 3, True, False)
    sel = np.arange(s) if rows is None else rows
    # the oracle's lowest-index winner: scale a/126, all errors zero
    assert np.all(idx[sel] == C_TIES // 126 - 1)
    assert np.all(sse[sel] == 0.0)
    st = check_rows(w, alpha, sse, idx, q, None, 8, True, C_TIES, 1.0, 3, rows=rows)
    assert st["idx_diff"] == 0 and st["alpha_bitwise"] == 1.0


def test_exact_ties_per_tensor_and_offset(gpu):
    """39 candidates with error 0 for the per-tensor search (unsigned 8-bit) and its offset variant."""
    import torch
    assert len(_divisors(255)) == 39
    x = _tie_rows(1, 300_001, seed=11, signed=False).ravel()
    alpha, sse, idx, curve = gpu.activation_scale(x, 8, False, C_TIES, 1.0, 3)
    ref = orc.activation_scale(x, 8, False, C_TIES, 1.0, 3)
    assert int(np.sum(ref.sse_curve == 0.0)) == 39 and int(np.sum(curve == 0.0)) == 39
    assert idx == ref.best_idx == C_TIES // 252 - 1
    assert alpha == ref.alpha and sse == 0.0
    shifted = x + np.float32(1.0)          # exact in binary32: the offset scheme sees the same shifted tensor
    d_x = torch.from_numpy(shifted).cuda()
    a, d, e = (torch.empty(1, device="cuda") for _ in range(3))
    i = torch.empty(1, dtype=torch.int32, device="cuda")
    gpu.ctx().omse_activation_scale_offset(d_x, x.size, 8, C_TIES, 1.0, 3, a, d, e, i)
    torch.cuda.synchronize()
    assert d.item() == 1.0 and i.item() == ref.best_idx and a.item() == ref.alpha and e.item() == 0.0


def test_exact_ties_dual_search_beyond_the_pair_list(gpu):
    """Dual search: every alpha1 = a/j (j = 1..6) reproduces the row with any alpha2, and so do some pairs where
    the second tensor takes what the first leaves: about 400 pairs with error 0."""
    a = np.float32(60 * 2.0 ** -10)
    rng = np.random.default_rng(5)
    t = (rng.integers(-1, 2, size=(4, 500)) * a).astype(np.float32)
    t[:, 0] = a
    alpha, sse, idx, q, _ = gpu.dual_quantize(t, 4, 4, True, 60, 64, 1.0, 0.25)
    ref = orc.dual_rows(t, 4, 4, True, 60, 64, 1.0, 0.25)
    one = orc.dual(t[0], 4, 4, True, 60, 64, 1.0, 0.25, want_curve=True)
    assert int(np.sum(one.sse_curve == 0.0)) > 256 and one.best_idx == ref.best_idx[0]
    assert np.array_equal(idx, ref.best_idx)
    assert np.array_equal(alpha, ref.alpha) and np.all(sse == 0.0)
    assert np.array_equal(q.reshape(2, 4, 500), ref.codes)


NEAR_TIE_CASES = [(0.8, 4, 0.05315625), (0.5, 4, 0.05340234375), (0.5, 5, 0.0644765625), (0.9, 5, 0.06078515625)]


@pytest.mark.parametrize("zero_prob,seed,hi_frac", NEAR_TIE_CASES)
def test_natural_near_ties_rows_and_per_tensor(gpu, zero_prob, seed, hi_frac):
    """A sparse heavy-tailed row of 28,672 values on a 2-bit grid with 4096 candidates ending just above the
    optimum: more than twenty candidates within 4e-6 of the minimum, none of them equal."""
    x = synth.relu_activations(28672, seed, zero_prob=zero_prob)
    ref = orc.phi(x, 2, True, 4096, hi_frac, 3, want_curve=True)
    near = int(np.sum(ref.sse_curve <= ref.sse_curve.min() * (1 + 4e-6)))
    assert near >= 20
    w = np.stack([x, x[::-1].copy(), -x])
    alpha, sse, idx, q, _ = gpu.quantize_weights(w, 2, True, 4096, hi_frac, 3, True, False)
    check_rows(w, alpha, sse, idx, q, None, 2, True, 4096, hi_frac, 3)
    a1, s1, i1, curve = gpu.activation_scale(x, 2, True, 4096, hi_frac, 3)
    np.testing.assert_allclose(curve, ref.sse_curve, rtol=2e-6)
    if i1 != ref.best_idx:
        assert abs(ref.sse_curve[i1] - ref.sse_curve[ref.best_idx]) <= 1e-6 * ref.sse_curve[ref.best_idx]
        ref = orc.phi(x, 2, True, 4096, hi_frac, 3, start_idx=i1, want_codes=False)
    assert a1 == pytest.approx(ref.alpha, rel=RTOL) and s1 == pytest.approx(ref.sse, rel=RTOL)
