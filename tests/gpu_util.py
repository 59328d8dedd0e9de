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


def assert_elementwise(y, ref, A, q: int, K: int, tensor_path: bool, out_f16: bool, where="") -> None:
    """Element-wise bound over ALL outputs (a norm can hide one wrong element in a large result).

    A = oracle.hlq.magnitude_bound(X, scales, offsets, G) bounds |X| |W_hat|^T and every intermediate of the +-1
    form.  Roundings of the paths, each at most its unit roundoff times A (worst case, all errors aligned):
      look-up kernels   fp32 table entries and fp32 accumulation over K terms      K * 2^-24 * A
      tensor-core path  W_hat rebuilt in fp16: z^ rounded once, one rounding per plane add   (q + 1) * 2^-11 * A
                        then fp32 accumulation in tensor memory                    K * 2^-23 * A
      fp16 output       one more rounding of the result                            2^-11 * |y|
    """
    import numpy as np
    y64 = np.asarray(y, dtype=np.float64)
    tol = (K * 2.0 ** -23 + (q + 1) * 2.0 ** -11) * A if tensor_path else K * 2.0 ** -24 * A
    if out_f16:
        tol = tol + 2.0 ** -11 * np.abs(ref) * 1.001 + 2.0 ** -24      # (+ fp16 subnormal spacing)
    bad = np.abs(y64 - ref) > tol
    if bad.any():
        i = np.argwhere(bad)[0]
        raise AssertionError(f"{where}: {int(bad.sum())} of {bad.size} elements outside the bound, first at {tuple(i)}: "
                             f"got {y64[tuple(i)]!r}, want {ref[tuple(i)]!r}, tolerance {tol[tuple(i)]!r}")
