"""Seeded synthetic tensors with the shapes and value distributions of the paper's workloads.

The paper quantizes ImageNet-trained CNN weights and calibration activations (Section 4);
neither is available offline, so these generators stand in for them: heavy-tailed,
zero-centred weights at the public ResNet-50 / VGG-16 shapes, and sparse non-negative
post-ReLU activations.  This module holds no arithmetic of the quantization method: it only
produces fp32 arrays, and the same bytes are handed to the CUDA library and to its checker.

Random numbers are counter-based: element i of stream (seed, tensor_id, lane) is
SplitMix64's output function applied to key + (i+1)*golden, so any slice can be
regenerated independently and results do not depend on chunking.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_CHUNK = 1 << 22


def _mix(z: np.ndarray) -> np.ndarray:
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def _key(seed: int, tensor_id: int, lane: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = np.array([seed], dtype=np.uint64) * _GOLDEN
        k = _mix(k + np.uint64(tensor_id) * _M1 + np.uint64(lane) * _M2 + np.uint64(1))
    return k[0]


def uniform01(seed: int, tensor_id: int, lane: int, start: int, count: int) -> np.ndarray:
    """float64 uniforms in the open interval (0, 1) for counters start..start+count-1."""
    with np.errstate(over="ignore"):
        ctr = (np.arange(start + 1, start + count + 1, dtype=np.uint64)) * _GOLDEN + _key(seed, tensor_id, lane)
        bits = _mix(ctr)
    return ((bits >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / (1 << 53))


def _normal(seed, tensor_id, lane, start, count):
    u1 = uniform01(seed, tensor_id, 2 * lane, start, count)
    u2 = uniform01(seed, tensor_id, 2 * lane + 1, start, count)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def _chunks(n):
    for s in range(0, n, _CHUNK):
        yield s, min(_CHUNK, n - s)


def _for_chunks(n, work):
    """work(start, count) for every chunk; chunks are independent (counter-based), so they run on host threads."""
    chunks = list(_chunks(n))
    if len(chunks) <= 1:
        for s, c in chunks:
            work(s, c)
        return
    with ThreadPoolExecutor(max_workers=min(len(chunks), os.cpu_count() or 1)) as ex:
        list(ex.map(lambda sc: work(*sc), chunks))


def laplace(n: int, b: float, seed: int, tensor_id: int = 0) -> np.ndarray:
    """Laplace(0, b) by inverse CDF."""
    out = np.empty(n, np.float32)

    def work(s, c):
        u = uniform01(seed, tensor_id, 0, s, c) - 0.5
        out[s:s + c] = (-b * np.sign(u) * np.log1p(-2.0 * np.abs(u))).astype(np.float32)
    _for_chunks(n, work)
    return out


def student_t3(n: int, seed: int, tensor_id: int = 0) -> np.ndarray:
    """Student-t with 3 degrees of freedom, unit scale: Z / sqrt((Z1^2+Z2^2+Z3^2)/3)."""
    out = np.empty(n, np.float32)

    def work(s, c):
        z = _normal(seed, tensor_id, 0, s, c)
        chi = sum(_normal(seed, tensor_id, l, s, c) ** 2 for l in (1, 2, 3))
        out[s:s + c] = (z / np.sqrt(chi / 3.0)).astype(np.float32)
    _for_chunks(n, work)
    return out


def relu_activations(n: int, seed: int, zero_prob: float = 0.4, tensor_id: int = 0) -> np.ndarray:
    """Post-ReLU stand-in: |t_3| magnitudes, each element exactly zero with probability zero_prob."""
    out = np.abs(student_t3(n, seed, tensor_id))

    def work(s, c):
        out[s:s + c][uniform01(seed, tensor_id, 15, s, c) < zero_prob] = 0.0
    _for_chunks(n, work)
    return out


def laplace_with_outliers(n: int, b: float, seed: int, outlier_prob: float = 1e-3, n_sigma: float = 20.0,
                          tensor_id: int = 0) -> np.ndarray:
    """Laplace(0, b); with probability outlier_prob an element becomes +-n_sigma*sigma, sigma = b*sqrt(2)."""
    out = laplace(n, b, seed, tensor_id)
    mag = np.float32(n_sigma * b * np.sqrt(2.0))

    def work(s, c):
        hit = uniform01(seed, tensor_id, 14, s, c) < outlier_prob
        sign = np.where(uniform01(seed, tensor_id, 13, s, c) < 0.5, np.float32(-1), np.float32(1))
        out[s:s + c] = np.where(hit, sign * mag, out[s:s + c])
    _for_chunks(n, work)
    return out


def resnet50_shapes() -> list[tuple[str, int, int]]:
    """(name, n_kernels, kernel_len) for the 53 convolutions and the FC layer of ResNet-50.

    kernel_len = in_channels * k_h * k_w: one row per output kernel (Section 3.1, W_lk).
    """
    shapes = [("conv1", 64, 3 * 7 * 7)]
    inplanes = 64
    for stage, (blocks, width) in enumerate(zip((3, 4, 6, 3), (64, 128, 256, 512)), start=1):
        for b in range(blocks):
            p = f"layer{stage}.{b}"
            shapes.append((f"{p}.conv1", width, inplanes))
            shapes.append((f"{p}.conv2", width, width * 9))
            shapes.append((f"{p}.conv3", width * 4, width))
            if b == 0:
                shapes.append((f"{p}.downsample", width * 4, inplanes))
            inplanes = width * 4
    shapes.append(("fc", 1000, 2048))
    return shapes


def resnet50_weights(seed: int = 2) -> list[tuple[str, np.ndarray]]:
    """He-scaled Laplace weights (std sqrt(2/fan_in), i.e. b = 1/sqrt(kernel_len)) at ResNet-50 shapes."""
    out = []
    for tid, (name, s, k) in enumerate(resnet50_shapes()):
        out.append((name, laplace(s * k, 1.0 / np.sqrt(k), seed, tid).reshape(s, k)))
    return out


def conv_layer(seed: int = 1) -> np.ndarray:
    """One 64x64x3x3 convolution as 64 kernels of 576 values, Laplace(0, 0.02)."""
    return laplace(64 * 576, 0.02, seed).reshape(64, 576)


def activation_tensor(seed: int = 3, n: int = 64 * 256 * 56 * 56) -> np.ndarray:
    return relu_activations(n, seed)


def fc6_weights(seed: int = 4, n_kernels: int = 4096, kernel_len: int = 25088) -> np.ndarray:
    """VGG-16 fc6-shaped matrix: Laplace(0, 0.005) with 0.1% outliers at 20 sigma."""
    return laplace_with_outliers(n_kernels * kernel_len, 0.005, seed).reshape(n_kernels, kernel_len)


def sweep_tensor(kernel_len: int, seed: int = 5, total: int = 1 << 26, n_kernels: int | None = None) -> np.ndarray:
    """Student-t(3) rows of length kernel_len filling about `total` elements."""
    s = n_kernels if n_kernels is not None else total // kernel_len
    return student_t3(s * kernel_len, seed, tensor_id=kernel_len).reshape(s, kernel_len)
