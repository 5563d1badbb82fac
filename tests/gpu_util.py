"""Helpers for the GPU tests: run the library through its C interface on numpy inputs."""
import numpy as np
import torch

from paper_1902_06822_b200 import binding

_ctx = None


def ctx():
    global _ctx
    if _ctx is None:
        _ctx = binding.Context(0)
    return _ctx


def quantize_weights(w, bits=4, signed=True, n_cand=256, hi_frac=1.0, refine_iters=3, want_codes=True,
                     want_packed=False):
    S, K = w.shape
    d_w = torch.from_numpy(np.ascontiguousarray(w)).cuda()
    alpha = torch.full((S,), -1.0, dtype=torch.float32, device="cuda")
    sse = torch.full((S,), -1.0, dtype=torch.float32, device="cuda")
    idx = torch.full((S,), -7, dtype=torch.int32, device="cuda")
    codes = torch.full((S * K,), 99, dtype=torch.int8, device="cuda") if want_codes else None
    packed = torch.full(((S * K + 1) // 2,), 0xAB, dtype=torch.uint8, device="cuda") if want_packed else None
    ctx().omse_quantize_weights(d_w, S, K, bits, signed, n_cand, hi_frac, refine_iters, alpha, sse, idx, codes, packed)
    torch.cuda.synchronize()
    return (alpha.cpu().numpy(), sse.cpu().numpy(), idx.cpu().numpy(),
            None if codes is None else codes.cpu().numpy(), None if packed is None else packed.cpu().numpy())


def activation_scale(x, bits=4, signed=False, n_cand=2048, hi_frac=1.0, refine_iters=3, want_curve=True):
    d_x = torch.from_numpy(np.ascontiguousarray(x)).cuda()
    alpha = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
    sse = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
    idx = torch.full((1,), -7, dtype=torch.int32, device="cuda")
    curve = torch.full((n_cand,), -1.0, dtype=torch.float64, device="cuda") if want_curve else None
    ctx().omse_activation_scale(d_x, d_x.numel(), bits, signed, n_cand, hi_frac, refine_iters, alpha, sse, idx, curve)
    torch.cuda.synchronize()
    return float(alpha.item()), float(sse.item()), int(idx.item()), None if curve is None else curve.cpu().numpy()


def residual_quantize(t, bits=(4, 4), signed=True, n_cand=1024, hi_frac=1.0, refine_iters=3, n_sweeps=1,
                      want_codes=True, want_packed=False):
    S, K = t.shape
    n = len(bits)
    d_t = torch.from_numpy(np.ascontiguousarray(t)).cuda()
    alpha = torch.full((n, S), -1.0, dtype=torch.float32, device="cuda")
    sse = torch.full((n, S), -1.0, dtype=torch.float32, device="cuda")
    codes = torch.full((n, S * K), 99, dtype=torch.int8, device="cuda") if want_codes else None
    packed = torch.full((n, (S * K + 1) // 2), 0xAB, dtype=torch.uint8, device="cuda") if want_packed else None
    ctx().omse_residual_quantize(d_t, S, K, list(bits), signed, n_cand, hi_frac, refine_iters, n_sweeps, alpha, sse,
                                 codes, packed)
    torch.cuda.synchronize()
    return (alpha.cpu().numpy(), sse.cpu().numpy(), None if codes is None else codes.cpu().numpy(),
            None if packed is None else packed.cpu().numpy())


def dual_quantize(t, bits1=4, bits2=4, signed=True, n_cand1=32, n_cand2=32, hi_frac1=1.0, hi_frac2=0.25,
                  want_codes=True, want_packed=False):
    S, K = t.shape
    d_t = torch.from_numpy(np.ascontiguousarray(t)).cuda()
    alpha = torch.full((2, S), -1.0, dtype=torch.float32, device="cuda")
    sse = torch.full((S,), -1.0, dtype=torch.float32, device="cuda")
    idx = torch.full((S,), -7, dtype=torch.int32, device="cuda")
    codes = torch.full((2, S * K), 99, dtype=torch.int8, device="cuda") if want_codes else None
    packed = torch.full((2, (S * K + 1) // 2), 0xAB, dtype=torch.uint8, device="cuda") if want_packed else None
    ctx().omse_dual_quantize(d_t, S, K, bits1, bits2, signed, n_cand1, n_cand2, hi_frac1, hi_frac2, alpha, sse, idx,
                             codes, packed)
    torch.cuda.synchronize()
    return (alpha.cpu().numpy(), sse.cpu().numpy(), idx.cpu().numpy(),
            None if codes is None else codes.cpu().numpy(), None if packed is None else packed.cpu().numpy())
