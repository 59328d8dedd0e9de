"""The definition of the HLQ product, in fp64 (test infrastructure).

Hierarchical Linear Quantization (Section 4.1, Eq. 3; dequantisation Eq. 6)
writes a group of weights as

    W_hat = sum_{j=0}^{q-1} s_j * b_j + z,     b_j in {0,1}^n, s_j, z real.

Algorithm 1 gives the parameter shapes for a matrix W in R^{N x K}: weights are
grouped along K in contiguous groups of G (its line "reshape W into groups"),
scales are s in R^{N x K/G x q} and zero-points z in R^{N x K/G}.  Scales and
zero-points are stored in fp16 (caption of the C4 perplexity table).

The linear layer is Y = X W_hat^T with fp16 activations X in R^{M x K}.
"""

from __future__ import annotations

import numpy as np


def split_bit_planes(w_int: np.ndarray, q: int) -> np.ndarray:
    """Split q-bit integers into q one-bit matrices (Appendix B).

    Plane j holds bit j of every integer, plane 0 being the lowest bit: the
    paper's example maps (9, 7, 6, 3) to lowest plane (1,1,0,1) and highest
    plane (1,0,0,0).  Returns uint8 [q, *w_int.shape].
    """
    w = np.asarray(w_int).astype(np.int64)
    if np.any(w < 0) or np.any(w >= (1 << q)):
        raise ValueError("integer weights must lie in [0, 2^q)")
    return np.stack([((w >> j) & 1).astype(np.uint8) for j in range(q)])


def reconstruct(planes: np.ndarray, scales: np.ndarray, offsets: np.ndarray, G: int) -> np.ndarray:
    """W_hat[n,k] = sum_j s[n, k div G, j] * b_j[n,k] + z[n, k div G]   (Eq. 3 / Eq. 6).

    planes uint8 [q,N,K] (non-zero = 1), scales [N,K/G,q], offsets [N,K/G];
    everything is promoted to fp64.  Returns fp64 [N,K].
    """
    q, N, K = planes.shape
    if K % G != 0:
        raise ValueError("K must be a multiple of G")
    s = np.asarray(scales, dtype=np.float64)
    z = np.asarray(offsets, dtype=np.float64)
    if s.shape != (N, K // G, q) or z.shape != (N, K // G):
        raise ValueError("scale / offset shapes do not match (N, K/G, q) / (N, K/G)")
    w = np.repeat(z, G, axis=1)                       # z[n, k div G]
    for j in range(q):
        bj = (planes[j] != 0).astype(np.float64)
        w += np.repeat(s[:, :, j], G, axis=1) * bj    # + s_j * b_j
    return w


def matmul(X: np.ndarray, planes: np.ndarray, scales: np.ndarray, offsets: np.ndarray,
           G: int, row_block: int = 1024) -> np.ndarray:
    """Y[m,n] = sum_k X[m,k] * W_hat[n,k] in fp64.

    W_hat is rebuilt a block of output rows at a time (so a 70B-sized layer
    never needs the whole fp64 matrix) and multiplied with the library fp64
    matmul.  Returns fp64 [M,N].
    """
    X64 = np.asarray(X, dtype=np.float64)
    q, N, K = planes.shape
    Y = np.empty((X64.shape[0], N), dtype=np.float64)
    for n0 in range(0, N, row_block):
        n1 = min(N, n0 + row_block)
        w = reconstruct(planes[:, n0:n1], scales[n0:n1], offsets[n0:n1], G)
        Y[:, n0:n1] = X64 @ w.T
    return Y


def matmul_loops(X, planes, scales, offsets, G) -> np.ndarray:
    """Same as `matmul`, as the plain triple loop (k ascending); tiny shapes only."""
    q, N, K = planes.shape
    M = len(X)
    Y = np.zeros((M, N), dtype=np.float64)
    for m in range(M):
        for n in range(N):
            acc = 0.0
            for k in range(K):
                w = float(offsets[n][k // G])
                for j in range(q):
                    if planes[j][n][k]:
                        w += float(scales[n][k // G][j])
                acc += float(X[m][k]) * w
            Y[m, n] = acc
    return Y


def offset_term(X: np.ndarray, offsets: np.ndarray, G: int) -> np.ndarray:
    """Y_bias[m,n] = sum_Gi z[n,Gi] * sum_{k in Gi} X[m,k]  (the z part of Eq. 3 under Y = X W_hat^T)."""
    X64 = np.asarray(X, dtype=np.float64)
    M, K = X64.shape
    S = X64.reshape(M, K // G, G).sum(axis=2)          # group sums of the activations
    return S @ np.asarray(offsets, dtype=np.float64).T


def scale_term(X, planes, scales, G, row_block: int = 1024) -> np.ndarray:
    """Y_scale = Y - Y_bias: the product with the offsets set to zero."""
    zero = np.zeros(np.asarray(scales).shape[:2], dtype=np.float64)
    return matmul(X, planes, scales, zero, G, row_block)


def magnitude_bound(X: np.ndarray, scales: np.ndarray, offsets: np.ndarray, G: int) -> np.ndarray:
    """A[m,n] = sum_Gi a[n,Gi] * sum_{k in Gi} |X[m,k]|  with  a = |z + (1/2) sum_j s_j| + (1/2) sum_j |s_j|.

    In the +-1 form of Appendix D every weight of a group is  z^ + sum_j (+-) s_j / 2  with z^ = z + (1/2) sum_j s_j,
    so a[n,Gi] bounds the magnitude of every weight of the group AND of every intermediate sum met when the terms
    are added one by one, whatever the bit-planes are: A >= |X| |W_hat|^T element-wise.  The parity tests use A as
    the scale of element-wise error bounds (each rounding of a path costs at most its unit roundoff times A).
    Independent of the planes, cost O(M N K / G).  Returns fp64 [M,N].
    """
    X64 = np.abs(np.asarray(X, dtype=np.float64))
    M, K = X64.shape
    s = np.asarray(scales, dtype=np.float64)
    z = np.asarray(offsets, dtype=np.float64)
    a = np.abs(z + 0.5 * s.sum(axis=2)) + 0.5 * np.abs(s).sum(axis=2)      # [N, K/G]
    S = X64.reshape(M, K // G, G).sum(axis=2)                              # [M, K/G]
    return S @ a.T


def to_fp16(Y: np.ndarray) -> np.ndarray:
    """Round an fp64 result once to fp16 (round-to-nearest-even), as the library's output does."""
    return np.asarray(Y, dtype=np.float64).astype(np.float16)


def rel_fro_error(Y_test: np.ndarray, Y_ref: np.ndarray) -> float:
    """||Y_test - Y_ref||_F / ||Y_ref||_F in fp64."""
    a = np.asarray(Y_test, dtype=np.float64)
    b = np.asarray(Y_ref, dtype=np.float64)
    den = float(np.linalg.norm(b))
    num = float(np.linalg.norm(a - b))
    return num / den if den > 0 else num
