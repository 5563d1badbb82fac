"""GPU parity of the dual line search (Section 3.5, n = 2) against the CPU oracle."""
import numpy as np
import pytest

from oracle import omse_oracle as orc
from paper_1902_06822_b200 import synth
from parity import RTOL, TIE_RTOL

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    import gpu_util
    return gpu_util


def _check(gpu, t, bits1=4, bits2=4, signed=True, c1=16, c2=16, hf1=1.0, hf2=0.25, packed=False):
    S, K = t.shape
    alpha, sse, idx, q, pk = gpu.dual_quantize(t, bits1, bits2, signed, c1, c2, hf1, hf2, True, packed)
    ref = orc.dual_rows(t, bits1, bits2, signed, c1, c2, hf1, hf2)
    diff = np.nonzero(idx != ref.best_idx)[0]
    for s in diff:                                   # another pair only if the oracle itself calls it a tie
        m = float(np.max(np.abs(t[s])))
        a = orc.dual_scales(m, hf1, hf2, c1, c2, *divmod(int(idx[s]), c2))
        b = orc.dual_scales(m, hf1, hf2, c1, c2, *divmod(int(ref.best_idx[s]), c2))
        s_lib = orc.dual_sse_at(t[s], a[0], a[1], bits1, bits2, signed)
        s_ref = orc.dual_sse_at(t[s], b[0], b[1], bits1, bits2, signed)
        assert abs(s_lib - s_ref) <= TIE_RTOL * s_ref, (s, idx[s], ref.best_idx[s])
    if diff.size:
        redo = orc.dual_rows(np.ascontiguousarray(t[diff]), bits1, bits2, signed, c1, c2, hf1, hf2, start_idx=idx[diff])
        ref.alpha[:, diff], ref.sse[diff], ref.codes[:, diff] = redo.alpha, redo.sse, redo.codes
    assert diff.size <= max(1, S // 50)
    assert np.array_equal(alpha, ref.alpha)          # scales are grid points: bit-exact
    np.testing.assert_allclose(sse, ref.sse, rtol=RTOL, atol=1e-37)
    assert np.array_equal(q.reshape(2, S, K), ref.codes)
    if packed:
        for j in range(2):
            assert np.array_equal(pk[j], orc.pack_int4(ref.codes[j]))
    return alpha, sse


def test_dual_on_a_conv_layer(gpu):
    w = synth.conv_layer(seed=1)
    alpha, sse = _check(gpu, w, c1=24, c2=24, packed=True)
    res = orc.residual_rows(w, (4, 4), True, 256, 1.0, 3, 1)
    assert np.mean(res.sse[1] / sse) > 1.5            # the joint search beats the residual scheme (Section 3.5)


@pytest.mark.parametrize("k", [1, 2, 5, 27, 64, 147, 1000])
def test_dual_kernel_lengths_and_packing(gpu, k):
    t = synth.student_t3(9 * k, seed=600 + k, tensor_id=k).reshape(9, k)
    _check(gpu, t, c1=12, c2=10, packed=True)


@pytest.mark.parametrize("bits1,bits2,signed,hf2", [(2, 4, True, 0.5), (4, 2, True, 0.25), (3, 3, True, 1.0),
                                                    (4, 4, False, 0.25), (2, 8, True, 0.1), (8, 4, True, 0.02)])
def test_dual_bit_widths_signedness_and_second_grid_range(gpu, bits1, bits2, signed, hf2):
    t = synth.laplace(7 * 200, 0.03, seed=610, tensor_id=bits1 * 16 + bits2).reshape(7, 200)
    if not signed:
        t = np.abs(t)
    _check(gpu, t, bits1, bits2, signed, c1=9, c2=7, hf2=hf2, packed=bits1 <= 4 and bits2 <= 4)


@pytest.mark.parametrize("hf2", [0.03, 0.06, 0.12, 0.5, 1.0, 2.5])
def test_dual_first_code_window_over_second_grid_ranges(gpu, hf2):
    """The enumeration over first codes is cut to a window whose width follows alpha2/alpha1: from second grids so
    narrow that every rest saturates (the asymmetry of Z_p2 then decides between the two neighbours) to ones wider
    than a step of the first grid.  Evenly spread values reach every position between two first codes."""
    rng = np.random.default_rng(640)
    t = rng.uniform(-1.0, 1.0, size=(6, 384)).astype(np.float32)
    t[3] = np.abs(t[3])
    t[4] *= np.float32(1e-3)
    _check(gpu, t, c1=32, c2=32, hf2=hf2)
    _check(gpu, t, bits1=3, bits2=4, c1=8, c2=16, hf2=hf2)


@pytest.mark.parametrize("c1,c2", [(1, 1), (1, 33), (40, 3), (64, 64)])
def test_dual_grid_shapes(gpu, c1, c2):
    t = synth.laplace(5 * 96, 0.02, seed=620, tensor_id=c1).reshape(5, 96)
    _check(gpu, t, c1=c1, c2=c2)


def test_dual_degenerate_rows_and_invalid_arguments(gpu):
    import torch
    from paper_1902_06822_b200 import binding
    t = synth.laplace(4 * 50, 0.02, seed=630).reshape(4, 50).copy()
    t[1] = 0.0
    gpu.ctx().omse_last_device_status()
    alpha, sse, idx, q, _ = gpu.dual_quantize(t, 4, 4, True, 8, 8, 1.0, 0.25)
    assert gpu.ctx().omse_last_device_status() & 2
    assert alpha[0, 1] == 0.0 and alpha[1, 1] == 0.0 and idx[1] == -1 and sse[1] == 0.0
    assert not q.reshape(2, 4, 50)[:, 1].any()
    d = torch.zeros(64, device="cuda")
    a = torch.zeros(2, 8, device="cuda")
    s = torch.zeros(8, device="cuda")
    for kw in [dict(n_cand1=0), dict(n_cand2=2000), dict(bits1=1), dict(bits2=9), dict(hi_frac2=0.0)]:
        args = dict(t=d, n_kernels=8, kernel_len=8, bits1=4, bits2=4, is_signed=True, n_cand1=4, n_cand2=4,
                    hi_frac1=1.0, hi_frac2=0.25, alpha=a, sse=s)
        args.update(kw)
        with pytest.raises(binding.OmseError) as e:
            gpu.ctx().omse_dual_quantize(**args)
        assert e.value.code == binding.EINVAL
