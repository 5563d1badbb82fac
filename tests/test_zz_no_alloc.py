"""The allocation-free per-tensor entry point against the ordinary one, through the C interface.

Some callers may not allocate device memory at the moment they need a scale (a plugin inside an
application whose pool owns the GPU's memory, a loop that forbids allocation after start-up), so
they can use neither a context nor anything that calls cudaMalloc.  omse_activation_scale_static
keeps its scratch in a fixed array inside the library; here it must reproduce
omse_activation_scale on the same inputs, on two calls in a row (the array keeps the first call's
contents, so the second call checks that everything that must start from zero is cleared).

Collected last on purpose: a run that stops at the first failure has then run every other test.
"""
import numpy as np
import pytest

from paper_1902_06822_b200 import synth

pytestmark = pytest.mark.gpu


def _both(x, bits, signed, n_cand, refine):
    import torch
    from paper_1902_06822_b200 import binding
    d_x = torch.from_numpy(np.ascontiguousarray(x)).cuda()
    n = d_x.numel()

    def outputs():
        return (torch.full((1,), -1.0, device="cuda"), torch.full((1,), -1.0, device="cuda"),
                torch.full((1,), -7, dtype=torch.int32, device="cuda"),
                torch.full((n_cand,), -1.0, dtype=torch.float64, device="cuda"))

    ctx = binding.Context(0)
    a0, s0, i0, c0 = outputs()
    ctx.omse_activation_scale(d_x, n, bits, signed, n_cand, 1.0, refine, a0, s0, i0, c0)
    torch.cuda.synchronize()
    ref = (a0.item(), s0.item(), i0.item(), c0.cpu().numpy())
    ctx.close()
    got = []
    for _ in range(2):                                   # two calls in a row share the scratch
        a1, s1, i1, c1 = outputs()
        st = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        binding.omse_activation_scale_static(d_x, n, bits, signed, n_cand, 1.0, refine, a1, s1, i1, c1, st)
        torch.cuda.synchronize()
        got.append((a1.item(), s1.item(), i1.item(), c1.cpu().numpy(), st.item()))
    return ref, got


@pytest.mark.parametrize("n,bits,signed,n_cand", [(300_001, 4, False, 2048), (70_000, 3, True, 256), (5, 4, False, 50),
                                                  (200_000, 4, False, 600), (200_000, 4, True, 1100),
                                                  (200_000, 2, False, 1500)])
def test_static_entry_point_matches_the_context_one_twice(n, bits, signed, n_cand):
    x = synth.relu_activations(n, seed=3, tensor_id=7) if not signed else synth.student_t3(n, seed=9)
    if n <= 8:
        x = x + np.float32(0.5)
    ref, got = _both(x, bits, signed, n_cand, 3)
    for alpha, sse, idx, curve, status in got:
        assert idx == ref[2]
        assert alpha == pytest.approx(ref[0], rel=1e-5)
        assert sse == pytest.approx(ref[1], rel=1e-5)
        np.testing.assert_allclose(curve, ref[3], rtol=2e-6)
        assert status == 0
    assert got[0][:3] == got[1][:3] and np.array_equal(got[0][3], got[1][3])   # second call starts clean
    # ... and both entry points agree with the CPU oracle, not only with each other
    from oracle import omse_oracle as orc
    want = orc.activation_scale(x, bits, signed, n_cand, 1.0, 3)
    alpha, sse, idx, curve, _ = got[1]
    np.testing.assert_allclose(curve, want.sse_curve, rtol=2e-6)
    if idx != want.best_idx:
        assert abs(want.sse_curve[idx] - want.sse_curve[want.best_idx]) <= 1e-6 * want.sse_curve[want.best_idx]
        want = orc.phi(x, bits, signed, n_cand, 1.0, 3, start_idx=idx, want_codes=False)
    assert alpha == pytest.approx(want.alpha, rel=1e-5) and sse == pytest.approx(want.sse, rel=1e-5)


def test_static_entry_point_clears_the_status_of_the_previous_call_and_rejects_oversize():
    import torch
    from paper_1902_06822_b200 import binding
    out = [torch.zeros(1, device="cuda"), torch.zeros(1, device="cuda")]
    st = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    zeros = torch.zeros(4096, device="cuda")
    binding.omse_activation_scale_static(zeros, 4096, 4, False, 128, 1.0, 1, out[0], out[1], None, None, st)
    torch.cuda.synchronize()
    assert st.item() & binding.DEV_DEGENERATE and out[0].item() == 0.0
    ones = torch.rand(4096, device="cuda") + 0.1
    binding.omse_activation_scale_static(ones, 4096, 4, False, 128, 1.0, 1, out[0], out[1], None, None, st)
    torch.cuda.synchronize()
    assert st.item() == 0 and out[0].item() > 0.0
    with pytest.raises(binding.OmseError) as e:
        binding.omse_activation_scale_static(ones, 4096, 4, False, binding.STATIC_MAX_CANDIDATES + 1, 1.0, 1,
                                             out[0], out[1])
    assert e.value.code == binding.ELIMIT
