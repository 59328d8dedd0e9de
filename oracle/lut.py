"""The bit-serial look-up-table procedure, in fp64 (test infrastructure).

Appendix B describes the computation in three steps:

 1. offline, the q-bit weights are split into q one-bit matrices;
 2. at run time, for every slice of g consecutive activations, the dot
    products of that slice with all 2^g single-bit weight patterns are
    precomputed and stored in a table;
 3. the product is then "table look-ups followed by summation": each one-bit
    weight row selects, per slice, the table entry addressed by its g bits.

With HLQ (Eq. 3) every quantisation group has its own scale per bit-plane and
its own offset, so the per-plane sums are kept per group, multiplied by
s[n,Gi,j], and the offset contributes z[n,Gi] times the group's activation sum,
which is the all-ones table entry summed over the group's slices.

Appendix D ("mirror storage") rewrites the same weights with +-1 bits:
s^ = s/2, b^ = 2b-1, z^ = z + (1/2) sum_j s_j; the +-1 table is antisymmetric
under complementing the index, so only half of it needs storing.

Bit order inside an index (the paper shows it only in a figure): bit i of the
index pairs with activation g*t + i of slice t (little-endian).
"""

from __future__ import annotations

import numpy as np


def patterns(g: int) -> np.ndarray:
    """All single-bit weight patterns of a g-wide slice: P[p,i] = bit i of p, fp64 [2^g, g]."""
    p = np.arange(1 << g)
    return np.stack([(p >> i) & 1 for i in range(g)], axis=1).astype(np.float64)


def build_lut(x_row: np.ndarray, g: int) -> np.ndarray:
    """LUT[t,p] = sum_i bit_i(p) * x[g*t+i]  (step 2), by the definition, fp64 [K/g, 2^g]."""
    x = np.asarray(x_row, dtype=np.float64)
    if x.size % g != 0:
        raise ValueError("K must be a multiple of the LUT width g")
    return x.reshape(-1, g) @ patterns(g).T


def plane_indices(planes: np.ndarray, g: int) -> np.ndarray:
    """idx[j,n,t] = sum_i b_j[n, g*t+i] * 2^i : the table address of each slice (int64 [q,N,K/g])."""
    q, N, K = planes.shape
    b = (planes != 0).astype(np.int64).reshape(q, N, K // g, g)
    w = (1 << np.arange(g, dtype=np.int64))
    return (b * w).sum(axis=3)


def lut_matmul(X, planes, scales, offsets, G: int, g: int = 4) -> np.ndarray:
    """Y = X W_hat^T by table look-ups, per-group scale multiply and offset term (fp64 [M,N])."""
    X64 = np.asarray(X, dtype=np.float64)
    M, K = X64.shape
    q, N, _ = planes.shape
    if G % g != 0 or K % G != 0:
        raise ValueError("need g | G | K")
    s = np.asarray(scales, dtype=np.float64)
    z = np.asarray(offsets, dtype=np.float64)
    idx = plane_indices(planes, g)                      # [q,N,T]
    T = K // g
    t_ar = np.arange(T)[None, :]
    Y = np.zeros((M, N), dtype=np.float64)
    for m in range(M):
        lut = build_lut(X64[m], g)                      # [T, 2^g]
        for j in range(q):
            looked = lut[t_ar, idx[j]]                  # [N,T]  one look-up per slice
            acc = looked.reshape(N, K // G, G // g).sum(axis=2)   # summation inside each group
            Y[m] += (s[:, :, j] * acc).sum(axis=1)      # per-plane, per-group scale
        S = lut[:, (1 << g) - 1].reshape(K // G, G // g).sum(axis=1)  # group sums = all-ones entries
        Y[m] += z @ S
    return Y


def table_f16_lut_matmul(X, planes, scales, offsets, G: int, g: int = 8) -> np.ndarray:
    """Table quantisation, first form (Appendix D): the tables hold fp16 values.

    Every table entry (an exact sum of g activations) is rounded once to fp16 before it is looked up;
    look-ups, per-group scale multiply and the offset term are as in lut_matmul, in fp64.  The offset
    term uses the unrounded group sums.  Returns fp64 [M,N]."""
    X64 = np.asarray(X, dtype=np.float64)
    M, K = X64.shape
    q, N, _ = planes.shape
    if G % g != 0 or K % G != 0:
        raise ValueError("need g | G | K")
    s = np.asarray(scales, dtype=np.float64)
    z = np.asarray(offsets, dtype=np.float64)
    idx = plane_indices(planes, g)
    T = K // g
    t_ar = np.arange(T)[None, :]
    Y = np.zeros((M, N), dtype=np.float64)
    for m in range(M):
        lut = build_lut(X64[m], g)
        lut16 = lut.astype(np.float16).astype(np.float64)          # one rounding per entry
        for j in range(q):
            looked = lut16[t_ar, idx[j]]
            acc = looked.reshape(N, K // G, G // g).sum(axis=2)
            Y[m] += (s[:, :, j] * acc).sum(axis=1)
        S = lut[:, (1 << g) - 1].reshape(K // G, G // g).sum(axis=1)
        Y[m] += z @ S
    return Y


def table_i8_lut_matmul(X, planes, scales, offsets, G: int, g: int = 8) -> np.ndarray:
    """Table quantisation, second form (Appendix D): the table values are mapped to int8.

    The paper fixes no scale; the reading taken here (and by the CUDA variant): one scale per activation
    row and quantisation group, scale = A / 127 with A the largest magnitude an entry of the group can
    take (the maximum over the group's slices of sum_i |x_i|), code = round-to-nearest-even(entry / scale)
    in [-127, 127], looked-up value = code * scale.  Look-ups of a group are summed as integers, then
    scaled; plane scales and the offset term (from the unquantised group sums) as in lut_matmul.  fp64."""
    X64 = np.asarray(X, dtype=np.float64)
    M, K = X64.shape
    q, N, _ = planes.shape
    if G % g != 0 or K % G != 0:
        raise ValueError("need g | G | K")
    s = np.asarray(scales, dtype=np.float64)
    z = np.asarray(offsets, dtype=np.float64)
    idx = plane_indices(planes, g)
    T = K // g
    t_ar = np.arange(T)[None, :]
    Y = np.zeros((M, N), dtype=np.float64)
    for m in range(M):
        lut = build_lut(X64[m], g)                                             # [T, 2^g]
        amax = np.abs(X64[m]).reshape(K // G, G // g, g).sum(axis=2).max(axis=1)   # [groups]
        sc = amax / 127.0
        inv = np.where(amax > 0, 127.0 / np.where(amax > 0, amax, 1.0), 0.0)
        codes = np.rint(lut * np.repeat(inv, G // g)[:, None]).astype(np.int64)     # [T, 2^g]
        for j in range(q):
            looked = codes[t_ar, idx[j]]                                        # [N, T] integers
            acc = looked.reshape(N, K // G, G // g).sum(axis=2)                 # integer sums per group
            Y[m] += (s[:, :, j] * (acc * sc[None, :])).sum(axis=1)
        S = lut[:, (1 << g) - 1].reshape(K // G, G // g).sum(axis=1)
        Y[m] += z @ S
    return Y


def mirror_transform(scales, offsets):
    """(s, z) -> (s^, z^) of Appendix D: s^ = s/2, z^ = z + (1/2) sum_j s_j, in fp64."""
    s = np.asarray(scales, dtype=np.float64)
    z = np.asarray(offsets, dtype=np.float64)
    return s / 2.0, z + 0.5 * s.sum(axis=2)


def reconstruct_mirror(planes, scales, offsets, G: int) -> np.ndarray:
    """W_hat = sum_j s^_j * b^_j + z^ with b^ = 2b-1 in {-1,+1} (Appendix D), fp64 [N,K]."""
    q, N, K = planes.shape
    sh, zh = mirror_transform(scales, offsets)
    w = np.repeat(zh, G, axis=1)
    for j in range(q):
        bh = 2.0 * (planes[j] != 0).astype(np.float64) - 1.0
        w += np.repeat(sh[:, :, j], G, axis=1) * bh
    return w


def build_mirror_half_lut(x_row: np.ndarray, g: int) -> np.ndarray:
    """Stored half of the +-1 table: entries whose top index bit is 0, fp64 [K/g, 2^(g-1)]."""
    x = np.asarray(x_row, dtype=np.float64)
    signs = 2.0 * patterns(g)[: 1 << (g - 1)] - 1.0     # top bit (i = g-1) is 0 -> -1
    return x.reshape(-1, g) @ signs.T


def mirror_lookup(half_lut: np.ndarray, t, p, g: int):
    """Entry p of slice t of the full +-1 table, recovered from the stored half by negation."""
    full = (1 << g) - 1
    top = (p >> (g - 1)) & 1
    p_half = np.where(top == 1, full ^ p, p)            # complement lands in the stored half
    val = half_lut[t, p_half]
    return np.where(top == 1, -val, val)


def mirror_lut_matmul(X, planes, scales, offsets, G: int, g: int = 4) -> np.ndarray:
    """Y through the half-size +-1 tables of Appendix D (fp64 [M,N])."""
    X64 = np.asarray(X, dtype=np.float64)
    M, K = X64.shape
    q, N, _ = planes.shape
    sh, zh = mirror_transform(scales, offsets)
    idx = plane_indices(planes, g)
    t_ar = np.arange(K // g)[None, :]
    Y = np.zeros((M, N), dtype=np.float64)
    for m in range(M):
        half = build_mirror_half_lut(X64[m], g)
        for j in range(q):
            looked = mirror_lookup(half, t_ar, idx[j], g)
            acc = looked.reshape(N, K // G, G // g).sum(axis=2)
            Y[m] += (sh[:, :, j] * acc).sum(axis=1)
        S = X64[m].reshape(K // G, G).sum(axis=1)
        Y[m] += zh @ S
    return Y
