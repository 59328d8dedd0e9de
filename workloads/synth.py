"""Counter-based seeded generators for HLQ layers and activations.

Every tensor is a pure function of (seed, tag, element index): a splitmix64
hash of a 64-bit counter gives the raw bits, so any row range of any tensor
can be drawn on its own and the result does not depend on the numpy or torch
version.  Value distributions follow the synthetic recipe of the benchmark
configurations:

* activations  X[M,K]      fp16( N(0,1) ), optionally with ceil(1 % of K)
                            seeded "outlier" columns scaled by 20
* bit-planes   b_j[n,k]    iid Bernoulli(0.5), stored as uint8 {0,1}, [q,N,K]
* scales       s[n,Gi,j]   fp16( |N(0, 0.02)| ),               [N,K/G,q]
* offsets      z[n,Gi]     fp16( N(0, 0.01) ),                 [N,K/G]

Nothing here computes anything the method computes.
"""

from __future__ import annotations

import math
import zlib
from dataclasses import dataclass

import numpy as np

_U64 = np.uint64
_GOLDEN = _U64(0x9E3779B97F4A7C15)
_M1 = _U64(0xBF58476D1CE4E5B9)
_M2 = _U64(0x94D049BB133111EB)


def _splitmix64(x: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser applied element-wise to uint64 counters."""
    with np.errstate(over="ignore"):
        z = (x + _GOLDEN).astype(_U64)
        z = (z ^ (z >> _U64(30))) * _M1
        z = (z ^ (z >> _U64(27))) * _M2
        z = z ^ (z >> _U64(31))
    return z


def _key(seed: int, tag: str) -> np.uint64:
    """64-bit stream key from the integer seed and a tensor tag."""
    t = zlib.crc32(tag.encode("utf-8")) & 0xFFFFFFFF
    base = np.array([(int(seed) & 0xFFFFFFFF) << 32 | t], dtype=_U64)
    return _splitmix64(_splitmix64(base))[0]


def _raw(seed: int, tag: str, start: int, count: int) -> np.ndarray:
    """`count` raw 64-bit words of stream (seed, tag) starting at counter `start`."""
    ctr = np.arange(start, start + count, dtype=_U64)
    with np.errstate(over="ignore"):
        return _splitmix64(ctr * _U64(0xD1342543DE82EF95) + _key(seed, tag))


def _normal(seed: int, tag: str, start: int, count: int) -> np.ndarray:
    """`count` standard normals (fp64) by Box-Muller; element i uses counters 2i, 2i+1."""
    r = _raw(seed, tag, 2 * start, 2 * count)
    u1 = ((r[0::2] >> _U64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)
    u2 = ((r[1::2] >> _U64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2)


def bit_planes(seed: int, tag: str, q: int, N: int, K: int,
               rows: np.ndarray | None = None) -> np.ndarray:
    """Bernoulli(0.5) bit-planes as uint8 {0,1}.

    Returns [q, N, K], or [q, len(rows), K] when `rows` selects output rows.
    Bit (j, n, k) is bit (idx mod 64) of raw word idx // 64, idx = (j*N+n)*K+k,
    so K must be a multiple of 64 for row-wise generation.
    """
    if K % 64 != 0:
        # small test shapes: draw everything, one word per bit
        r = _raw(seed, tag + "/bits1", 0, q * N * K)
        full = (r >> _U64(63)).astype(np.uint8).reshape(q, N, K)
        return full if rows is None else full[:, np.asarray(rows), :]
    wpr = K // 64
    if rows is None:
        words = _raw(seed, tag + "/bits", 0, q * N * wpr)
        by = words.view(np.uint8)  # little-endian bytes
        bits = np.unpackbits(by, bitorder="little")
        return bits.reshape(q, N, K)
    rows = np.asarray(rows, dtype=np.int64)
    out = np.empty((q, len(rows), K), dtype=np.uint8)
    for j in range(q):
        for i, n in enumerate(rows):
            words = _raw(seed, tag + "/bits", (j * N + int(n)) * wpr, wpr)
            out[j, i] = np.unpackbits(words.view(np.uint8), bitorder="little")
    return out


def scales(seed: int, tag: str, N: int, Gn: int, q: int, std: float = 0.02,
           rows: np.ndarray | None = None, signed: bool = False) -> np.ndarray:
    """Per-group per-plane scales fp16 [N, Gn, q] = |N(0,std)| (signed=True keeps the sign)."""
    per_row = Gn * q
    if rows is None:
        v = _normal(seed, tag + "/scales", 0, N * per_row).reshape(N, Gn, q)
    else:
        rows = np.asarray(rows, dtype=np.int64)
        v = np.stack([_normal(seed, tag + "/scales", int(n) * per_row, per_row).reshape(Gn, q)
                      for n in rows]) if len(rows) else np.zeros((0, Gn, q))
    v = v * std
    if not signed:
        v = np.abs(v)
    return v.astype(np.float16)


def offsets(seed: int, tag: str, N: int, Gn: int, std: float = 0.01,
            rows: np.ndarray | None = None) -> np.ndarray:
    """Per-group offsets fp16 [N, Gn] = N(0,std)."""
    if rows is None:
        v = _normal(seed, tag + "/offsets", 0, N * Gn).reshape(N, Gn)
    else:
        rows = np.asarray(rows, dtype=np.int64)
        v = np.stack([_normal(seed, tag + "/offsets", int(n) * Gn, Gn) for n in rows]) \
            if len(rows) else np.zeros((0, Gn))
    return (v * std).astype(np.float16)


def outlier_columns(seed: int, tag: str, K: int, frac: float = 0.01) -> np.ndarray:
    """ceil(frac*K) distinct column indices chosen by a seeded permutation (sorted)."""
    n_out = int(math.ceil(frac * K))
    keys = _raw(seed, tag + "/outlier_perm", 0, K)
    return np.sort(np.argsort(keys, kind="stable")[:n_out])


def activations(seed: int, tag: str, M: int, K: int, outliers: bool = False) -> np.ndarray:
    """X fp16 [M, K] ~ N(0,1); with outliers=True, 1 % of the columns are scaled by 20."""
    x = _normal(seed, tag + "/x", 0, M * K).reshape(M, K)
    if outliers:
        cols = outlier_columns(seed, tag, K)
        x[:, cols] *= 20.0
    return x.astype(np.float16)


def dense_weights(seed: int, tag: str, N: int, K: int, std: float = 0.02, heavy_frac: float = 0.002) -> np.ndarray:
    """Unquantised weights fp16 [N, K] for the parameter fitter: N(0, std) with a fraction of entries
    scaled by 6 (the heavy tails of trained linear layers, which make uniform grids wasteful)."""
    w = _normal(seed, tag + "/w", 0, N * K) * std
    u = _raw(seed, tag + "/w_heavy", 0, N * K)
    heavy = (u >> np.uint64(40)).astype(np.float64) / float(1 << 24) < heavy_frac
    w = np.where(heavy, w * 6.0, w)
    return w.reshape(N, K).astype(np.float16)


@dataclass
class HlqLayer:
    """One synthetic HLQ linear layer (host numpy tensors)."""
    q: int
    G: int
    N: int
    K: int
    planes: np.ndarray   # uint8 [q, N, K]
    scales: np.ndarray   # fp16  [N, K/G, q]
    offsets: np.ndarray  # fp16  [N, K/G]
    tag: str = ""
    seed: int = 0


def hlq_layer(seed: int, tag: str, q: int, G: int, N: int, K: int,
              signed_scales: bool = False) -> HlqLayer:
    """Draw a whole layer: planes Bernoulli(0.5), scales |N(0,.02)|, offsets N(0,.01)."""
    if K % G != 0:
        raise ValueError("K must be a multiple of the quantisation group G")
    Gn = K // G
    return HlqLayer(q=q, G=G, N=N, K=K,
                    planes=bit_planes(seed, tag, q, N, K),
                    scales=scales(seed, tag, N, Gn, q, signed=signed_scales),
                    offsets=offsets(seed, tag, N, Gn),
                    tag=tag, seed=seed)
