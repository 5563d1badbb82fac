"""Section 3.5 pipeline on a small synthetic network: quantize every layer, find the key layers
(MSE > tau), give them a second tensor, report the compression ratio."""
import numpy as np
import pytest

from oracle import omse_oracle as orc
from paper_1902_06822_b200 import synth

pytestmark = pytest.mark.gpu


def test_key_layer_selection_and_compression_ratio():
    import torch
    import gpu_util
    from paper_1902_06822_b200 import binding
    ctx = gpu_util.ctx()
    shapes = [(16, 27), (32, 144), (8, 1152), (10, 64), (1, 500)]
    scales = [0.2, 0.05, 0.01, 0.3, 0.02]                  # layers with larger weights have larger MSE
    ws = [synth.laplace(s * k, b, seed=700, tensor_id=i).reshape(s, k) for i, ((s, k), b) in enumerate(zip(shapes, scales))]
    descs = [dict(w=torch.from_numpy(w).cuda(), n_kernels=w.shape[0], kernel_len=w.shape[1],
                  alpha=torch.empty(w.shape[0], device="cuda"), sse=torch.empty(w.shape[0], device="cuda"))
             for w in ws]
    ctx.omse_quantize_weights_batched(descs, 4, True, 256, 1.0, 3)
    mse = torch.full((len(ws),), -1.0, dtype=torch.float64, device="cuda")
    key = torch.full((len(ws),), -7, dtype=torch.int32, device="cuda")
    tau = 8e-5                                             # the threshold the paper uses for INT4 (Table 3 caption)
    ctx.omse_select_key_layers([(d["sse"], d["n_kernels"], d["kernel_len"]) for d in descs], tau, mse, key)
    torch.cuda.synchronize()
    mse_h, key_h = mse.cpu().numpy(), key.cpu().numpy()
    for i, (w, d) in enumerate(zip(ws, descs)):
        ref = orc.layer_mse(d["sse"].cpu().numpy(), w.shape[1])
        assert mse_h[i] == pytest.approx(ref, rel=1e-12)
        full = orc.quantize_rows(w, 4, True, 256, 1.0, 3)
        assert mse_h[i] == pytest.approx(full.sse.sum() / w.size, rel=1e-5)
        assert key_h[i] == int(ref > tau)
    assert 0 < key_h.sum() < len(ws)                       # the threshold separates the layers
    # key layers get a second tensor (Section 3.5): their error drops, the others stay as they are
    n_t = []
    for w, d, k in zip(ws, descs, key_h):
        n_t.append(2 if k else 1)
        if k:
            a2, s2, _, _ = gpu_util.residual_quantize(w, (4, 4), True, 256, 1.0, 3, 1, want_codes=False)
            assert s2[1].sum() < d["sse"].cpu().numpy().sum()
    ks, ls = [s for s, _ in shapes], [k for _, k in shapes]
    cr = binding.omse_compression_ratio(ks, ls, [4] * len(ws), n_t)
    assert cr == pytest.approx(orc.compression_ratio(ks, ls, [4] * len(ws), n_t), rel=1e-12)
    assert cr > binding.omse_compression_ratio(ks, ls, [4] * len(ws), [1] * len(ws)) > 0.125
    with pytest.raises(binding.OmseError):
        ctx.omse_select_key_layers([(descs[0]["sse"], 0, 5)], tau, mse, key)
    assert binding.omse_compression_ratio([1], [0], [4], [1]) == -1.0
