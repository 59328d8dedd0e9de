"""Helpers shared by the GPU parity tests: move a synthetic layer to the device, pack it, run the library."""

from __future__ import annotations

import numpy as np
import torch

import paper_2510_19482_b200 as elutq


def to_dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def pack_layer(layer):
    """Device blob of a workloads.HlqLayer via elutq_pack."""
    planes = to_dev(layer.planes)
    scales = to_dev(layer.scales.view(np.int16)).view(torch.float16)
    offsets = to_dev(layer.offsets.view(np.int16)).view(torch.float16)
    packed = elutq.elutq_pack(planes, scales, offsets, layer.q, layer.G, layer.N, layer.K)
    torch.cuda.synchronize()
    return packed


def x_dev(X: np.ndarray) -> torch.Tensor:
    return to_dev(X.view(np.int16)).view(torch.float16)


def gemm_f32(X: np.ndarray, packed, N: int, K: int, flags: int = 0) -> np.ndarray:
    M = X.shape[0]
    Y = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    elutq.elutq_lut_gemm_f32(x_dev(X), packed, Y, M, N, K, flags)
    torch.cuda.synchronize()
    return Y.cpu().numpy()


def gemm_f16(X: np.ndarray, packed, N: int, K: int) -> np.ndarray:
    M = X.shape[0]
    Y = torch.full((M, N), float("nan"), dtype=torch.float16, device="cuda")
    elutq.elutq_lut_gemm(x_dev(X), packed, Y, M, N, K)
    torch.cuda.synchronize()
    return Y.cpu().numpy()
