"""GPU parity of the quantizer with offset (Section 3.1 scheme, MMSE scale) against the CPU oracle."""
import numpy as np
import pytest

from oracle import omse_oracle as orc
from paper_1902_06822_b200 import synth
from parity import RTOL, TIE_RTOL

pytestmark = pytest.mark.gpu


def _rows(w, bits, n_cand, refine, packed):
    import torch
    import gpu_util
    S, K = w.shape
    d_w = torch.from_numpy(np.ascontiguousarray(w)).cuda()
    alpha = torch.empty(S, device="cuda")
    delta = torch.full((S,), 123.0, device="cuda")
    sse = torch.empty(S, device="cuda")
    idx = torch.empty(S, dtype=torch.int32, device="cuda")
    codes = torch.empty(S * K, dtype=torch.int8, device="cuda")
    pk = torch.empty((S * K + 1) // 2, dtype=torch.uint8, device="cuda") if packed else None
    gpu_util.ctx().omse_quantize_weights_offset(d_w, S, K, bits, n_cand, 1.0, refine, alpha, delta, sse, idx, codes, pk)
    torch.cuda.synchronize()
    return (alpha.cpu().numpy(), delta.cpu().numpy(), sse.cpu().numpy(), idx.cpu().numpy(),
            codes.cpu().numpy().reshape(S, K), None if pk is None else pk.cpu().numpy())


@pytest.mark.parametrize("s,k,bits,n_cand", [(40, 147, 4, 256), (9, 2000, 4, 1024), (3000, 256, 3, 1024),
                                             (5, 9000, 8, 1024), (33, 27, 2, 64)])
def test_offset_rows_match_oracle(s, k, bits, n_cand):
    w = synth.student_t3(s * k, seed=800 + k, tensor_id=bits).reshape(s, k) + np.float32(0.7)
    alpha, delta, sse, idx, q, pk = _rows(w, bits, n_cand, 3, bits <= 4)
    ref = orc.offset_rows(w, bits, n_cand, 1.0, 3)
    assert np.array_equal(delta, ref.delta)
    diff = np.nonzero(idx != ref.best_idx)[0]
    assert diff.size <= max(1, s // 50)
    if diff.size:
        shifted = (w[diff] - ref.delta[diff, None]).astype(np.float32)
        for i, r in enumerate(diff):
            m = float(np.max(np.abs(shifted[i])))
            a = orc.sse_at(shifted[i], orc.candidate(m, 1.0, n_cand, int(idx[r])), bits, False)
            b = orc.sse_at(shifted[i], orc.candidate(m, 1.0, n_cand, int(ref.best_idx[r])), bits, False)
            assert abs(a - b) <= TIE_RTOL * b
        redo = orc.offset_rows(np.ascontiguousarray(w[diff]), bits, n_cand, 1.0, 3, start_idx=idx[diff])
        ref.alpha[diff], ref.sse[diff], ref.codes[diff] = redo.alpha, redo.sse, redo.codes
    np.testing.assert_allclose(alpha, ref.alpha, rtol=RTOL)
    np.testing.assert_allclose(sse, ref.sse, rtol=RTOL, atol=1e-37)
    same = alpha == ref.alpha
    assert same.mean() >= 0.98 and np.array_equal(q[same], ref.codes[same])
    if pk is not None:
        assert np.array_equal(pk, orc.pack_int4(q))


@pytest.mark.parametrize("n,n_cand", [(5, 512), (4097, 512), (1_000_000, 512), (250_000, 600), (250_000, 1100),
                                      (250_000, 1500), (250_000, 3000)])
def test_offset_activation_scale_matches_oracle(n, n_cand):
    import torch
    import gpu_util
    x = synth.student_t3(n, seed=810, tensor_id=n % 89) * np.float32(0.5) + np.float32(2.0)
    d_x = torch.from_numpy(x).cuda()
    alpha, delta, sse = (torch.empty(1, device="cuda") for _ in range(3))
    idx = torch.empty(1, dtype=torch.int32, device="cuda")
    curve = torch.empty(n_cand, dtype=torch.float64, device="cuda")
    gpu_util.ctx().omse_activation_scale_offset(d_x, n, 4, n_cand, 1.0, 3, alpha, delta, sse, idx, curve)
    torch.cuda.synchronize()
    ref = orc.offset_rows(x.reshape(1, -1), 4, n_cand, 1.0, 3)
    assert delta.item() == ref.delta[0] == x.min()
    shifted = (x - ref.delta[0]).astype(np.float32)
    ref_curve = orc.phi(shifted, 4, False, n_cand, 1.0, 0, want_codes=False, want_curve=True).sse_curve
    np.testing.assert_allclose(curve.cpu().numpy(), ref_curve, rtol=2e-6)
    if idx.item() != ref.best_idx[0]:
        assert abs(ref_curve[idx.item()] - ref_curve[ref.best_idx[0]]) <= TIE_RTOL * ref_curve[ref.best_idx[0]]
        ref = orc.offset_rows(x.reshape(1, -1), 4, n_cand, 1.0, 3, start_idx=np.array([idx.item()], np.int32))
    assert alpha.item() == pytest.approx(ref.alpha[0], rel=RTOL)
    assert sse.item() == pytest.approx(ref.sse[0], rel=RTOL)
    # the plain call afterwards is unaffected by the offset state
    a2, s2, i2, _ = gpu_util.activation_scale(np.abs(x), 4, False, 512, 1.0, 3, want_curve=False)
    r2 = orc.activation_scale(np.abs(x), 4, False, 512, 1.0, 3, want_curve=False)
    assert a2 == pytest.approx(r2.alpha, rel=RTOL) and s2 == pytest.approx(r2.sse, rel=RTOL)
