"""GPU parity of the comparison solvers of Section 3.4 (uniform, alternating, golden-section), of the
offset scheme with the offset searched (Section 3.1), of Algorithm 1's loop condition and of the
one-call key-layer procedure (Section 3.5), each against the CPU oracle through the C interface."""
import numpy as np
import pytest

from oracle import omse_oracle as orc
from paper_1902_06822_b200 import synth
from parity import RTOL, TIE_RTOL

pytestmark = pytest.mark.gpu

ORACLE_SOLVER = {1: orc.SOLVER_UNIFORM, 2: orc.SOLVER_ALTERNATING, 3: orc.SOLVER_GOLDEN}


def _solver(w, bits, signed, solver, n_iter, hi_frac, refine, packed):
    import torch
    import gpu_util
    S, K = w.shape
    d_w = torch.from_numpy(np.ascontiguousarray(w)).cuda()
    alpha = torch.full((S,), -1.0, device="cuda")
    sse = torch.full((S,), -1.0, device="cuda")
    idx = torch.full((S,), -7, dtype=torch.int32, device="cuda")
    codes = torch.full((S * K,), 99, dtype=torch.int8, device="cuda")
    pk = torch.empty((S * K + 1) // 2, dtype=torch.uint8, device="cuda") if packed else None
    gpu_util.ctx().omse_quantize_weights_solver(d_w, S, K, bits, signed, solver, n_iter, 64, hi_frac, refine, alpha, sse,
                                                idx, codes, pk)
    torch.cuda.synchronize()
    return (alpha.cpu().numpy(), sse.cpu().numpy(), idx.cpu().numpy(), codes.cpu().numpy().reshape(S, K),
            None if pk is None else pk.cpu().numpy())


@pytest.mark.parametrize("solver,n_iter", [(1, 0), (2, 1), (2, 12), (3, 0), (3, 1), (3, 20), (3, 40)])
@pytest.mark.parametrize("s,k,bits,signed", [(37, 147, 4, True), (300, 576, 4, True), (6, 9000, 3, True),
                                              (11, 64, 8, True), (50, 27, 2, True), (20, 300, 4, False)])
def test_solver_rows_match_oracle(solver, n_iter, s, k, bits, signed):
    w = synth.student_t3(s * k, seed=900 + k, tensor_id=bits).reshape(s, k)
    if not signed:
        w = np.abs(w)
    alpha, sse, idx, q, pk = _solver(w, bits, signed, solver, n_iter, 1.0, 0, bits <= 4)
    ref = orc.solver_rows(w, ORACLE_SOLVER[solver], bits, signed, n_iter, 1.0, 0)
    # Once the golden-section bracket is down to a few binary32 steps, the two interior errors agree to the last
    # bits of their binary64 sums and the order of summation may decide a branch: the scales then differ by a few
    # ulp.  Everything else is bit-equal.
    same = alpha == ref.alpha
    assert same.all() if not (solver == 3 and n_iter > 20) else same.mean() >= 0.9
    np.testing.assert_allclose(alpha, ref.alpha, rtol=RTOL)
    np.testing.assert_allclose(sse, ref.sse, rtol=RTOL)
    assert np.array_equal(q[same], ref.codes[same]) and np.all(idx == 0)
    for r in np.nonzero(~same)[0]:
        assert np.array_equal(q[r], orc.codes(w[r], alpha[r], bits, signed))
    if pk is not None:
        assert np.array_equal(pk, orc.pack_int4(q))


def test_solver_edge_cases_and_polish():
    w = synth.laplace(40 * 200, 0.1, seed=77).reshape(40, 200)
    w[3] = 0.0                                   # degenerate row
    w[5, 7] = np.inf                             # non-finite value
    for solver in (1, 2, 3):
        alpha, sse, idx, q, _ = _solver(w, 4, True, solver, 10, 1.5, 2, False)
        ref = orc.solver_rows(w, ORACLE_SOLVER[solver], 4, True, 10, 1.5, 2)
        ok = np.ones(40, bool)
        ok[5] = False
        assert np.array_equal(alpha[ok], ref.alpha[ok]) and np.array_equal(q[ok], ref.codes[ok])
        assert alpha[3] == 0.0 and idx[3] == -1 and not q[3].any()
    # the grid solver through the same entry point is omse_quantize_weights
    import gpu_util
    a0, s0, i0, q0, _ = gpu_util.quantize_weights(w[:3], 4, True, 64, 1.0, 3)
    a1, s1, i1, q1, _ = _solver(w[:3], 4, True, 0, 0, 1.0, 3, False)
    assert np.array_equal(a0, a1) and np.array_equal(i0, i1) and np.array_equal(q0.reshape(3, -1), q1)


def test_four_solvers_ordering_on_conv_shaped_rows():
    """Same inputs, four ways to the scale (the comparison of Section 3.4 for the error itself)."""
    import gpu_util
    w = synth.laplace(256 * 1152, 1.0 / np.sqrt(1152.0), seed=31).reshape(256, 1152)
    uni = _solver(w, 4, True, 1, 0, 1.0, 0, False)[1].astype(np.float64)
    alt = _solver(w, 4, True, 2, 50, 1.0, 0, False)[1].astype(np.float64)
    gold = _solver(w, 4, True, 3, 25, 1.0, 0, False)[1].astype(np.float64)
    grid = gpu_util.quantize_weights(w, 4, True, 1024, 1.0, 3, want_codes=False)[1].astype(np.float64)
    assert np.all(alt <= uni * (1 + 1e-6))
    assert grid.sum() <= gold.sum() * (1 + 1e-6) and grid.sum() < alt.sum() < uni.sum()


def _affine(w, bits, n_cand, refine, n_delta, off_frac, packed):
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
    gpu_util.ctx().omse_quantize_weights_affine(d_w, S, K, bits, n_cand, 1.0, refine, n_delta, off_frac, alpha, delta,
                                                sse, idx, codes, pk)
    torch.cuda.synchronize()
    return (alpha.cpu().numpy(), delta.cpu().numpy(), sse.cpu().numpy(), idx.cpu().numpy(),
            codes.cpu().numpy().reshape(S, K), None if pk is None else pk.cpu().numpy())


@pytest.mark.parametrize("s,k,bits,n_cand,n_delta", [(40, 147, 4, 256, 8), (7, 2000, 4, 1024, 4), (200, 256, 3, 512, 6),
                                                      (3, 20000, 4, 1024, 3), (33, 27, 2, 64, 16), (12, 576, 8, 256, 5)])
def test_affine_rows_match_oracle(s, k, bits, n_cand, n_delta):
    w = synth.student_t3(s * k, seed=950 + k, tensor_id=bits).reshape(s, k) + np.float32(0.4)
    alpha, delta, sse, idx, q, pk = _affine(w, bits, n_cand, 3, n_delta, 0.25, bits <= 4)
    ref = orc.affine_rows(w, bits, n_cand, 1.0, n_delta, 0.25, 3)
    diff = np.nonzero(idx != ref.best_idx)[0]
    assert diff.size <= max(1, s // 20)
    for r in diff:                                   # another pair only when the oracle's own errors tie
        a, dl, e, fi, _, curve = orc.affine_phi(w[r], bits, n_cand, 1.0, n_delta, 0.25, 0, want_curve=True)
        flat = curve.reshape(-1)
        assert abs(flat[idx[r]] - flat[ref.best_idx[r]]) <= TIE_RTOL * flat[ref.best_idx[r]]
    if diff.size:
        redo = orc.affine_rows(np.ascontiguousarray(w[diff]), bits, n_cand, 1.0, n_delta, 0.25, 3, start_flat=idx[diff])
        ref.alpha[diff], ref.sse[diff], ref.codes[diff], ref.delta[diff] = redo.alpha, redo.sse, redo.codes, redo.delta
    assert np.array_equal(delta, ref.delta)
    np.testing.assert_allclose(alpha, ref.alpha, rtol=RTOL)
    np.testing.assert_allclose(sse, ref.sse, rtol=RTOL, atol=1e-37)
    same = alpha == ref.alpha
    assert same.mean() >= 0.95 and np.array_equal(q[same], ref.codes[same])
    if pk is not None:
        assert np.array_equal(pk, orc.pack_int4(q))
    # one offset on the grid is the offset call
    if k <= 2000:
        import torch
        import gpu_util
        a1, d1, s1, i1, q1, _ = _affine(w, bits, n_cand, 3, 1, 0.25, False)
        o = orc.offset_rows(w, bits, n_cand, 1.0, 3)
        assert np.array_equal(d1, o.delta)
        np.testing.assert_allclose(a1, o.alpha, rtol=RTOL)


def test_affine_rejects_bad_arguments():
    import torch
    import gpu_util
    from paper_1902_06822_b200 import binding
    t = torch.zeros(8, device="cuda")
    for n_delta, off in ((0, 0.2), (65, 0.2), (4, -0.1), (4, 1.5)):
        with pytest.raises(binding.OmseError):
            gpu_util.ctx().omse_quantize_weights_affine(t, 1, 8, 4, 16, 1.0, 0, n_delta, off, t[:1], t[1:2], t[2:3])
    with pytest.raises(binding.OmseError):
        gpu_util.ctx().omse_quantize_weights_solver(t, 1, 8, 4, True, 7, 3, 16, 1.0, 0, t[:1], t[1:2])
    assert binding.Context.workspace_bytes(10, 576, 1024, 2) > 16 << 20
    assert binding.Context.workspace_bytes(10, 0, 1024, 2) == 0


@pytest.mark.parametrize("s,k,bits,eps", [(24, 160, (3, 3), 0.02), (6, 3000, (4, 4), 0.005), (40, 64, (2, 2, 2), 0.05),
                                          (10, 160, (3, 3), 0.0), (10, 160, (3, 3), 10.0)])
def test_algorithm_1_loop_condition_matches_oracle(s, k, bits, eps):
    import torch
    import gpu_util
    t = synth.student_t3(s * k, seed=23 + k).reshape(s, k)
    n, max_sweeps = len(bits), 6
    d_t = torch.from_numpy(t).cuda()
    alpha = torch.empty(n, s, device="cuda")
    sse = torch.empty(n, s, device="cuda")
    hist = torch.full((max_sweeps, n, s), -1.0, device="cuda")
    done = torch.full((s,), -1, dtype=torch.int32, device="cuda")
    codes = torch.empty(n, s * k, dtype=torch.int8, device="cuda")
    gpu_util.ctx().omse_alg1_quantize_converge(d_t, s, k, list(bits), [True] * n, 64, 1.0, 2, max_sweeps, eps, alpha, sse,
                                               hist, done, codes)
    torch.cuda.synchronize()
    ref, rhist, rdone = orc.alg1_rows_eps(t, bits, (True,) * n, 64, 1.0, 2, max_sweeps, eps)
    assert np.array_equal(done.cpu().numpy(), rdone)
    np.testing.assert_allclose(alpha.cpu().numpy(), ref.alpha, rtol=RTOL)
    np.testing.assert_allclose(sse.cpu().numpy(), ref.sse, rtol=RTOL)
    np.testing.assert_allclose(hist.cpu().numpy(), rhist, rtol=RTOL)
    same = alpha.cpu().numpy() == ref.alpha
    q = codes.cpu().numpy().reshape(n, s, k)
    assert same.mean() > 0.95 and np.array_equal(q[same], ref.codes[same])
    if eps == 10.0:
        assert np.all(rdone == 1)


@pytest.mark.parametrize("packed", [False, True])
def test_key_layer_procedure_in_one_call_matches_oracle(packed):
    import torch
    import gpu_util
    shapes = [(16, 27), (32, 144), (8, 1152), (10, 64), (1, 500), (300, 64), (40, 2304)]
    scales = [0.2, 0.05, 0.01, 0.3, 0.02, 0.25, 0.004]
    ws = [synth.laplace(s * k, b, seed=720, tensor_id=i).reshape(s, k) for i, ((s, k), b) in enumerate(zip(shapes, scales))]
    tau = 8e-5
    descs = []
    for w in ws:
        s, k = w.shape
        d = dict(w=torch.from_numpy(w).cuda(), n_kernels=s, kernel_len=k, alpha=torch.empty(s, device="cuda"),
                 sse=torch.empty(s, device="cuda"), alpha2=torch.full((s,), -5.0, device="cuda"),
                 sse2=torch.full((s,), -5.0, device="cuda"))
        if packed:
            d["packed"] = torch.empty((s * k + 1) // 2, dtype=torch.uint8, device="cuda")
            d["packed2"] = torch.full(((s * k + 1) // 2,), 0xEE, dtype=torch.uint8, device="cuda")
        else:
            d["codes"] = torch.empty(s * k, dtype=torch.int8, device="cuda")
            d["codes2"] = torch.full((s * k,), 77, dtype=torch.int8, device="cuda")
        descs.append(d)
    L = len(ws)
    mse = torch.empty(L, dtype=torch.float64, device="cuda")
    key = torch.full((L,), -3, dtype=torch.int32, device="cuda")
    cr = torch.empty(1, dtype=torch.float64, device="cuda")
    gpu_util.ctx().omse_last_device_status()             # clear what earlier tests left in the status word
    gpu_util.ctx().omse_quantize_key_layers(descs, 4, True, 256, 1.0, 3, tau, mse, key, cr)
    torch.cuda.synchronize()
    ref = orc.key_layer_pipeline(ws, 4, True, 256, 1.0, 3, tau)
    key_h = key.cpu().numpy()
    assert np.array_equal(key_h.astype(bool), ref.is_key) and 0 < key_h.sum() < L
    np.testing.assert_allclose(mse.cpu().numpy(), ref.mse, rtol=RTOL)
    assert cr.item() == pytest.approx(ref.compression_ratio, rel=1e-12)
    for l, (w, d) in enumerate(zip(ws, descs)):
        np.testing.assert_allclose(d["alpha"].cpu().numpy(), ref.first[l].alpha, rtol=RTOL)
        if key_h[l]:
            r2 = ref.second[l]
            a2, s2 = d["alpha2"].cpu().numpy(), d["sse2"].cpu().numpy()
            np.testing.assert_allclose(a2, r2.alpha[1], rtol=RTOL)
            np.testing.assert_allclose(s2, r2.sse[1], rtol=RTOL, atol=1e-37)
            same = (a2 == r2.alpha[1]) & (d["alpha"].cpu().numpy() == r2.alpha[0])
            assert same.mean() > 0.9
            if packed:
                if same.all():
                    assert np.array_equal(d["packed2"].cpu().numpy(), orc.pack_int4(r2.codes[1]))
            else:
                q2 = d["codes2"].cpu().numpy().reshape(w.shape)
                assert np.array_equal(q2[same], r2.codes[1][same])
        else:                                            # untouched: not a key layer
            assert torch.all(d["alpha2"] == -5.0) and torch.all(d["sse2"] == -5.0)
            if packed:
                assert torch.all(d["packed2"] == 0xEE)
            else:
                assert torch.all(d["codes2"] == 77)
    assert gpu_util.ctx().omse_last_device_status() == 0


def test_launch_counter_counts_one_launch_per_row_path():
    """A batched weight call is issued as one launch per row path present; the counter is what bench.py reports."""
    import torch
    import gpu_util
    ctx = gpu_util.ctx()
    ctx.omse_read_launches()
    shapes = [(3000, 64), (2500, 576), (40, 2304), (16, 4608)]            # short rows in numbers + long rows
    descs = [dict(w=torch.from_numpy(synth.laplace(s * k, 0.05, seed=5, tensor_id=i).reshape(s, k)).cuda(), n_kernels=s,
                  kernel_len=k, alpha=torch.empty(s, device="cuda"), sse=torch.empty(s, device="cuda"))
             for i, (s, k) in enumerate(shapes)]
    ctx.omse_quantize_weights_batched(descs, 4, True, 1024, 1.0, 3)
    assert ctx.omse_read_launches() == 2
    ctx.omse_quantize_weights_batched(descs[2:], 4, True, 1024, 1.0, 3)
    assert ctx.omse_read_launches() == 1 and ctx.omse_read_launches() == 0
    x = torch.from_numpy(synth.relu_activations(100_000, seed=3)).cuda()
    a, e = torch.empty(1, device="cuda"), torch.empty(1, device="cuda")
    ctx.omse_activation_scale(x, x.numel(), 4, False, 2048, 1.0, 3, a, e)
    assert ctx.omse_read_launches() == 11          # init, maxima, two sweeps, curve, argmin, re-score, 3 polish steps, final
    torch.cuda.synchronize()


def test_back_to_back_batched_calls_with_two_row_paths_stay_ordered_and_reproducible():
    """A list with long and short rows runs its two launches beside each other (second stream inside the call).  Many
    such calls queued without a synchronisation in between, interleaved with per-tensor searches and single-path calls
    on the same context, must give the same bits every time, and the values of the oracle."""
    import torch
    import gpu_util
    ctx = gpu_util.ctx()
    shapes = [(700, 64), (900, 147), (600, 576), (50, 1152), (24, 4608), (12000, 27)]   # short, long and very short rows
    ws = [synth.student_t3(s * k, seed=9, tensor_id=i).reshape(s, k) for i, (s, k) in enumerate(shapes)]
    x = torch.from_numpy(synth.relu_activations(300_000, seed=5)).cuda()
    a_x, e_x = torch.empty(1, device="cuda"), torch.empty(1, device="cuda")
    ctx.omse_last_device_status()                    # clears the sticky status word
    rounds = []
    for it in range(12):
        descs = [dict(w=torch.from_numpy(w).cuda(), n_kernels=w.shape[0], kernel_len=w.shape[1],
                      alpha=torch.empty(w.shape[0], device="cuda"), sse=torch.empty(w.shape[0], device="cuda"),
                      packed=torch.empty((w.size + 1) // 2, dtype=torch.uint8, device="cuda")) for w in ws]
        ctx.omse_quantize_weights_batched(descs, 4, True, 1024, 1.0, 3)
        if it % 3 == 0:
            ctx.omse_activation_scale(x, x.numel(), 4, False, 2048, 1.0, 3, a_x, e_x)
        if it % 4 == 1:
            ctx.omse_quantize_weights_batched(descs[3:5], 4, True, 1024, 1.0, 3)     # long rows only: one launch
        rounds.append(descs)
    torch.cuda.synchronize()
    assert ctx.omse_last_device_status() == 0
    for descs in rounds[1:]:
        for d, d0 in zip(descs, rounds[0]):
            assert torch.equal(d["alpha"], d0["alpha"]) and torch.equal(d["sse"], d0["sse"])
            assert torch.equal(d["packed"], d0["packed"])
    for w, d in zip(ws, rounds[-1]):
        rows = np.arange(0, w.shape[0], max(1, w.shape[0] // 40))
        ref = orc.quantize_rows(np.ascontiguousarray(w[rows]), 4, True, 1024, 1.0, 3)
        np.testing.assert_allclose(d["alpha"].cpu().numpy()[rows], ref.alpha, rtol=1e-5)
        np.testing.assert_allclose(d["sse"].cpu().numpy()[rows], ref.sse, rtol=1e-5)
