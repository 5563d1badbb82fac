"""Acceptance rule shared by the GPU parity tests.

Codes and packed bytes must be bit-exact given the same scale; the chosen grid index must be the
oracle's unless the oracle's own errors at the two indices agree to 1e-6 relative (then the oracle
is re-run from the library's index and compared from there); scales and errors agree to 1e-5.
"""
import numpy as np

from oracle import omse_oracle as orc

RTOL = 1e-5        # scales and squared errors
TIE_RTOL = 1e-6    # two candidates count as tied when their oracle errors agree to this


def check_rows(w, alpha, sse, best_idx, codes, packed, bits, signed, n_cand, hi_frac, refine_iters, rows=None):
    """Compare library outputs for the selected rows of w [S, K] with the oracle; returns statistics."""
    S, K = w.shape
    rows = np.arange(S) if rows is None else np.asarray(rows)
    sub = np.ascontiguousarray(w[rows])
    ref = orc.quantize_rows(sub, bits, signed, n_cand, hi_frac, refine_iters)
    g_alpha, g_sse = alpha[rows], sse[rows]
    n_idx_diff = 0
    if best_idx is not None:
        g_idx = best_idx[rows]
        diff = np.nonzero(g_idx != ref.best_idx)[0]
        n_idx_diff = diff.size
        for i in diff:
            assert g_idx[i] >= 0 and ref.best_idx[i] >= 0, f"row {rows[i]}: degenerate mismatch"
            m = float(np.max(np.abs(sub[i])))
            s_lib = orc.sse_at(sub[i], orc.candidate(m, hi_frac, n_cand, int(g_idx[i])), bits, signed)
            s_ref = orc.sse_at(sub[i], orc.candidate(m, hi_frac, n_cand, int(ref.best_idx[i])), bits, signed)
            assert abs(s_lib - s_ref) <= TIE_RTOL * s_ref, \
                f"row {rows[i]}: index {g_idx[i]} vs {ref.best_idx[i]} is not a tie ({s_lib} vs {s_ref})"
        if diff.size:
            redo = orc.quantize_rows(np.ascontiguousarray(sub[diff]), bits, signed, n_cand, hi_frac, refine_iters,
                                     start_idx=g_idx[diff])
            ref.alpha[diff], ref.sse[diff], ref.codes[diff] = redo.alpha, redo.sse, redo.codes
    np.testing.assert_allclose(g_alpha, ref.alpha, rtol=RTOL, atol=0)
    np.testing.assert_allclose(g_sse, ref.sse, rtol=RTOL, atol=1e-37)
    same_alpha = g_alpha == ref.alpha
    if codes is not None:
        g_codes = codes.reshape(S, K)[rows]
        assert np.array_equal(g_codes[same_alpha], ref.codes[same_alpha])
        for i in np.nonzero(~same_alpha)[0]:       # scale off by an ulp: codes must be the oracle's for THAT scale
            assert np.array_equal(g_codes[i], orc.codes(sub[i], g_alpha[i], bits, signed)), f"row {rows[i]}"
    if packed is not None:
        flat_ref = np.zeros(S * K, np.int8)
        full = codes.reshape(S, K) if codes is not None else None
        if full is None:
            assert rows.size == S, "packed-only comparison needs every row"
            full = ref.codes.copy()
            for i in np.nonzero(~same_alpha)[0]:
                full[i] = orc.codes(sub[i], g_alpha[i], bits, signed)
        flat_ref = np.ascontiguousarray(full).reshape(-1)
        assert np.array_equal(packed, orc.pack_int4(flat_ref))
    return {"rows": int(rows.size), "idx_diff": int(n_idx_diff), "alpha_bitwise": float(np.mean(same_alpha))}
