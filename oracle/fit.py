"""Algorithm 1: alternating optimisation of the HLQ parameters, in fp64 (test infrastructure).

For every group of G consecutive weights of a row (Algorithm 1, "reshape W into groups"):

    Delta = (max - min) / (2^q - 1);  s^(0) = [Delta, 2 Delta, ..., 2^(q-1) Delta];  z^(0) = min
    for t = 1 .. T_max:
        W' = W - z^(t-1)                                   (shifted weights)
        V  = s^(t-1) x C^T                                 (the 2^q candidate values)
        k* = argmin_k |W' - V_k| per weight;  B^(t) = C_k*  (bit-pattern selection, Eq. 5)
        (s^(t), z^(t)) = LSE(W, B^(t))                      (least squares on [B 1], Section 4.2)

and the result is B^(T), s^(T), z^(T), with s and z stored in fp16.

Readings where the paper is silent (the CUDA side takes the same ones):
* codebook order: row k of C holds the binary digits of k, digit j (value 2^j) being b_j;
* ties of the argmin go to the smallest k;
* the least-squares problem is solved from its normal equations [B 1]^T [B 1] x = [B 1]^T W; when
  that matrix is singular (a plane that is constant over the group, two equal planes, ...) the
  least-squares solution is not unique and the step keeps s^(t-1), z^(t-1): the error still does
  not increase.  Singularity is decided exactly, in integer arithmetic (the matrix holds bit counts);
* arithmetic is fp64; candidate values are accumulated as ((0 + s_0 c_0) + s_1 c_1) + ...; the
  right-hand side sums are exact (fp16 inputs are integers in units of 2^-24); the normal equations
  are solved by elimination without pivoting (the matrix is symmetric positive definite when it is
  not singular), one rounding per operation, no fused multiply-add.

Everything is vectorised over groups; per group the order of operations is the one listed above.
"""

from __future__ import annotations

import numpy as np

_FIX = float(1 << 24)      # every finite fp16 value is an integer multiple of 2^-24


def _groups(W: np.ndarray, G: int) -> np.ndarray:
    W = np.asarray(W)
    if W.dtype != np.float16:
        raise ValueError("W must be fp16")
    N, K = W.shape
    if K % G != 0:
        raise ValueError("K must be a multiple of G")
    return W.astype(np.float64).reshape(N * (K // G), G)


def candidates(s: np.ndarray, q: int) -> np.ndarray:
    """V[..., k] = sum_j s[..., j] * digit_j(k), accumulated from j = 0 upwards (Eq. 4 without z)."""
    out = np.zeros(s.shape[:-1] + (1 << q,), dtype=np.float64)
    for k in range(1 << q):
        v = np.zeros(s.shape[:-1], dtype=np.float64)
        for j in range(q):
            if (k >> j) & 1:
                v = v + s[..., j]
        out[..., k] = v
    return out


def select_bits(w: np.ndarray, s: np.ndarray, z: np.ndarray, q: int) -> np.ndarray:
    """Bit-pattern selection (Eq. 5): index of the nearest candidate per weight, first minimum on ties.

    w [g, G] fp64, s [g, q], z [g]; returns int64 codes [g, G] (bit j of a code is b_j)."""
    shifted = w - z[:, None]
    V = candidates(s, q)
    best = np.zeros(w.shape, dtype=np.int64)
    best_d = np.abs(shifted - V[:, 0][:, None])
    for k in range(1, 1 << q):
        d = np.abs(shifted - V[:, k][:, None])
        better = d < best_d
        best = np.where(better, k, best)
        best_d = np.where(better, d, best_d)
    return best


def normal_equations(w: np.ndarray, codes: np.ndarray, q: int):
    """A = [B 1]^T [B 1] (exact integers) and r = [B 1]^T w (exact, via 2^-24 fixed point)."""
    g, G = w.shape
    n = q + 1
    cols = [((codes >> j) & 1).astype(np.int64) for j in range(q)] + [np.ones_like(codes, dtype=np.int64)]
    A = np.zeros((g, n, n), dtype=np.int64)
    for i in range(n):
        for j in range(n):
            A[:, i, j] = np.sum(cols[i] * cols[j], axis=1)
    wi = np.rint(w * _FIX).astype(np.int64)
    if not np.array_equal(wi.astype(np.float64) / _FIX, w):
        raise ValueError("weights are not fp16 values")
    r = np.zeros((g, n), dtype=np.float64)
    for i in range(n):
        r[:, i] = np.sum(cols[i] * wi, axis=1).astype(np.float64) / _FIX
    return A, r


def is_singular(A: np.ndarray) -> np.ndarray:
    """Exact test: fraction-free elimination without pivoting on the integer matrix; a zero pivot
    (a vanishing leading principal minor) means the positive semi-definite matrix is singular."""
    g, n, _ = A.shape
    m = A.astype(object)                       # Python integers: no overflow
    sing = np.zeros(g, dtype=bool)
    prev = np.ones(g, dtype=object)
    for c in range(n):
        sing |= (m[:, c, c] == 0)
        piv = np.where(sing, 1, m[:, c, c])    # groups already known singular carry on with dummy pivots
        for i in range(c + 1, n):
            for j in range(c + 1, n):
                m[:, i, j] = (m[:, i, j] * piv - m[:, i, c] * m[:, c, j]) // prev
        prev = piv
    return sing


def solve_spd(A: np.ndarray, r: np.ndarray) -> np.ndarray:
    """Elimination without pivoting, then back substitution, vectorised over groups (fp64, one
    rounding per operation).  Singular systems must be masked out by the caller."""
    g, n, _ = A.shape
    a = A.astype(np.float64).copy()
    b = r.copy()
    with np.errstate(divide="ignore", invalid="ignore"):
        for c in range(n):
            for i in range(c + 1, n):
                f = a[:, i, c] / a[:, c, c]
                for j in range(c + 1, n):
                    a[:, i, j] = a[:, i, j] - f * a[:, c, j]
                b[:, i] = b[:, i] - f * b[:, c]
        x = np.zeros((g, n), dtype=np.float64)
        for i in range(n - 1, -1, -1):
            acc = b[:, i].copy()
            for j in range(i + 1, n):
                acc = acc - a[:, i, j] * x[:, j]
            x[:, i] = acc / a[:, i, i]
    return x


def sse(w: np.ndarray, codes: np.ndarray, s: np.ndarray, z: np.ndarray, q: int) -> np.ndarray:
    """Squared reconstruction error per group for given bits and parameters (Eq. 7)."""
    rec = np.repeat(z[:, None], w.shape[1], axis=1)
    for j in range(q):
        rec = rec + s[:, j][:, None] * ((codes >> j) & 1)
    return np.sum((w - rec) ** 2, axis=1)


def fit(W: np.ndarray, q: int, G: int, t_max: int = 10, trace: bool = False):
    """Algorithm 1 on an fp16 matrix W [N, K].

    Returns (planes uint8 [q, N, K], scales fp16 [N, K/G, q], offsets fp16 [N, K/G]) and, with
    trace=True, also the per-group squared error [t_max + 1, N*K/G]: row 0 for the uniform
    initialisation with its own nearest codes, row t after iteration t (fp64 parameters)."""
    if t_max < 1:
        raise ValueError("t_max must be at least 1")
    w = _groups(W, G)
    N, K = W.shape
    g = w.shape[0]
    wmax = np.max(w, axis=1)
    wmin = np.min(w, axis=1)
    delta = (wmax - wmin) / float((1 << q) - 1)
    s = np.stack([delta * float(1 << j) for j in range(q)], axis=1)
    z = wmin.copy()
    errs = []
    if trace:
        errs.append(sse(w, select_bits(w, s, z, q), s, z, q))
    codes = np.zeros(w.shape, dtype=np.int64)
    for _ in range(t_max):
        codes = select_bits(w, s, z, q)
        A, r = normal_equations(w, codes, q)
        sing = is_singular(A)
        x = solve_spd(A, r)
        keep = sing[:, None]
        s = np.where(keep, s, x[:, :q])
        z = np.where(sing, z, x[:, q])
        if trace:
            errs.append(sse(w, codes, s, z, q))
    planes = np.stack([((codes >> j) & 1).astype(np.uint8).reshape(N, K) for j in range(q)])
    scales = s.astype(np.float16).reshape(N, K // G, q)
    offsets = z.astype(np.float16).reshape(N, K // G)
    if trace:
        return planes, scales, offsets, np.stack(errs)
    return planes, scales, offsets
