"""Reference packer for the library's device layout "v1" (test infrastructure).

The paper rearranges the one-bit matrices offline so that the kernel's loads
are contiguous and decoding needs only AND and shift (Appendix D,
"Weight-Rearrange"); the concrete arrangement there is specific to 128-bit NEON
registers and shown only in a figure.  The device layout below is therefore
this library's own choice ("parity unpinned" by the paper).  It is a pure
function of (q, G, N, K), written here in scatter form - for every logical
element, where it lands - independently of the CUDA packer.

Geometry
    tile        = 16 output rows x 512 input columns (one "row block" rb = n div 16,
                  one "K chunk" kc = k div 512); tiles are stored kc-major:
                  tile index = kc * n_rb + rb, n_rb = ceil(N/16), n_kc = ceil(K/512)
    column      = 8 consecutive k (one byte of one bit-plane): c = (k mod 512) div 8, 0..63;
                  bit (k mod 8) of that byte, little-endian, is b_j[n,k]
    super-group = 16 columns (128 k): sigma = c div 16, tau = c mod 16
    lane        = 16*h + l,  l = n mod 16,  h = sigma mod 2;  u = sigma div 2
                  (a lane owns one output row and super-groups h and h+2 of the chunk)
    sub-group   = one quantisation group inside a super-group: w = G/8 columns,
                  nsg = 128/G of them per super-group
    step        a lane visits the 16 columns of a super-group in a rotated order so
                  that the 16 lanes of a half-warp touch 16 different columns at every
                  step.  With a = l div w, r = l mod w, step i = v*w + ii (ii < w):
                      tau(l, i) = w * ((a + v) mod nsg) + (r + ii) mod w
    tile bytes  = 32 * (32*q + 2*gl*(q+1)),  gl = 2*nsg groups per lane

Inside a tile
    plane vectors  V[vec][lane][16 bytes], vec = u*q + j; byte i is the byte of
                   plane j, row n, column 16*(h+2u) + tau(l, i)
    parameters     P[word][lane] 32-bit words after the plane vectors; a lane's record is
                   gl*(q+1) fp16 values: for u in 0..1, for v in 0..nsg-1: the group
                   gamma = nsg*(h+2u) + (a+v) mod nsg of the chunk, as [s_0 .. s_{q-1}, z];
                   fp16 value e sits in word e div 2, low half first
    rows >= N and columns >= K hold zero bits and +0.0 parameters

A 128-byte header precedes the tiles (little-endian uint32 words):
    magic 'ELTQ', version 1, q, G, N, K, n_rb, n_kc, tile_bytes, 0...
"""

from __future__ import annotations

import numpy as np

HEADER_BYTES = 128
MAGIC = 0x51544C45
VERSION = 1
TILE_ROWS = 16
CHUNK_K = 512


def geometry(q: int, G: int, N: int, K: int) -> dict:
    if G not in (32, 64, 128):
        raise ValueError("G must be 32, 64 or 128")
    if K % G != 0:
        raise ValueError("K must be a multiple of G")
    nsg = 128 // G
    gl = 2 * nsg
    n_rb = -(-N // TILE_ROWS)
    n_kc = -(-K // CHUNK_K)
    tile_bytes = 32 * (32 * q + 2 * gl * (q + 1))
    return dict(q=q, G=G, N=N, K=K, w=G // 8, nsg=nsg, gl=gl, n_rb=n_rb, n_kc=n_kc,
                tile_bytes=tile_bytes, plane_bytes=32 * 32 * q,
                total=HEADER_BYTES + n_kc * n_rb * tile_bytes)


def packed_bytes(q: int, G: int, N: int, K: int) -> int:
    return geometry(q, G, N, K)["total"]


def _plane_byte_offsets(geo: dict, j: int, n: np.ndarray, cg: np.ndarray) -> np.ndarray:
    """Byte offset of the byte of plane j holding row n, global column cg = k div 8."""
    q, w, nsg = geo["q"], geo["w"], geo["nsg"]
    rb, l = n // TILE_ROWS, n % TILE_ROWS
    kc, c = cg // 64, cg % 64
    sigma, tau = c // 16, c % 16
    h, u = sigma % 2, sigma // 2
    a, r = l // w, l % w
    sg, rr = tau // w, tau % w
    v = (sg - a) % nsg
    ii = (rr - r) % w
    i = v * w + ii
    lane = 16 * h + l
    tile = kc * geo["n_rb"] + rb
    return HEADER_BYTES + tile * geo["tile_bytes"] + ((u * q + j) * 32 + lane) * 16 + i


def _param_offsets(geo: dict, n: np.ndarray, gi: np.ndarray, comp: int) -> np.ndarray:
    """Byte offset of fp16 parameter `comp` (0..q-1 scale of plane comp, q = offset) of (row n, group gi)."""
    q, G, w, nsg = geo["q"], geo["G"], geo["w"], geo["nsg"]
    rb, l = n // TILE_ROWS, n % TILE_ROWS
    gpc = CHUNK_K // G                       # groups per chunk
    kc, gamma = gi // gpc, gi % gpc
    sigma, sg = gamma // nsg, gamma % nsg
    h, u = sigma % 2, sigma // 2
    a = l // w
    v = (sg - a) % nsg
    e = (u * nsg + v) * (q + 1) + comp
    lane = 16 * h + l
    tile = kc * geo["n_rb"] + rb
    return (HEADER_BYTES + tile * geo["tile_bytes"] + geo["plane_bytes"]
            + ((e // 2) * 32 + lane) * 4 + 2 * (e % 2))


def header(geo: dict) -> np.ndarray:
    hdr = np.zeros(HEADER_BYTES // 4, dtype="<u4")
    hdr[:9] = [MAGIC, VERSION, geo["q"], geo["G"], geo["N"], geo["K"],
               geo["n_rb"], geo["n_kc"], geo["tile_bytes"]]
    return hdr.view(np.uint8)


def pack_reference(planes: np.ndarray, scales: np.ndarray, offsets: np.ndarray, G: int) -> np.ndarray:
    """The device blob (uint8) for a layer, built by scattering every logical element."""
    q, N, K = planes.shape
    geo = geometry(q, G, N, K)
    blob = np.zeros(geo["total"], dtype=np.uint8)
    blob[:HEADER_BYTES] = header(geo)
    n = np.arange(N, dtype=np.int64)[:, None]
    cg = np.arange(K // 8, dtype=np.int64)[None, :]
    for j in range(q):
        by = np.packbits(planes[j] != 0, axis=1, bitorder="little")      # [N, K/8]
        blob[_plane_byte_offsets(geo, j, n, cg)] = by
    gi = np.arange(K // G, dtype=np.int64)[None, :]
    s16 = np.ascontiguousarray(np.asarray(scales, dtype=np.float16))
    z16 = np.ascontiguousarray(np.asarray(offsets, dtype=np.float16))
    for comp in range(q + 1):
        val = s16[:, :, comp] if comp < q else z16
        raw = np.ascontiguousarray(val).view(np.uint16)
        off = _param_offsets(geo, n, gi, comp)
        blob[off] = (raw & 0xFF).astype(np.uint8)
        blob[off + 1] = (raw >> 8).astype(np.uint8)
    return blob


def parse_header(blob: np.ndarray) -> dict:
    hdr = np.ascontiguousarray(blob[:HEADER_BYTES]).view("<u4")
    if int(hdr[0]) != MAGIC or int(hdr[1]) != VERSION:
        raise ValueError("not a v1 ELTQ blob")
    return dict(q=int(hdr[2]), G=int(hdr[3]), N=int(hdr[4]), K=int(hdr[5]),
                n_rb=int(hdr[6]), n_kc=int(hdr[7]), tile_bytes=int(hdr[8]))


def unpack_reference(blob: np.ndarray):
    """Inverse of `pack_reference`: (planes uint8 [q,N,K], scales fp16 [N,K/G,q], offsets fp16 [N,K/G])."""
    h = parse_header(blob)
    q, G, N, K = h["q"], h["G"], h["N"], h["K"]
    geo = geometry(q, G, N, K)
    n = np.arange(N, dtype=np.int64)[:, None]
    cg = np.arange(K // 8, dtype=np.int64)[None, :]
    planes = np.empty((q, N, K), dtype=np.uint8)
    for j in range(q):
        by = blob[_plane_byte_offsets(geo, j, n, cg)]
        planes[j] = np.unpackbits(by, axis=1, bitorder="little")
    gi = np.arange(K // G, dtype=np.int64)[None, :]
    s = np.empty((N, K // G, q), dtype=np.float16)
    z = np.empty((N, K // G), dtype=np.float16)
    for comp in range(q + 1):
        off = _param_offsets(geo, n, gi, comp)
        raw = blob[off].astype(np.uint16) | (blob[off + 1].astype(np.uint16) << 8)
        if comp < q:
            s[:, :, comp] = raw.view(np.float16)
        else:
            z[:] = raw.view(np.float16)
    return planes, s, z


def index_map(planes: np.ndarray) -> np.ndarray:
    """idx_j(n, c): the 8-bit table address of plane j, row n, column c (uint8 [q,N,K/8])."""
    return np.stack([np.packbits(p != 0, axis=1, bitorder="little") for p in planes])


def consumer_walk(blob: np.ndarray, X: np.ndarray) -> np.ndarray:
    """Y = X W_hat^T computed by reading the blob the way a lane of the kernel is documented to.

    For every tile and lane, in program order (u, v, plane j, step ii) the walk
    fetches byte i of plane vector u*q+j, takes it as the 8-bit address of the
    column 16*(h+2u)+tau(l,i), sums the addressed activations per sub-group,
    multiplies by the lane record's scale and adds offset * group activation sum.
    Plain Python loops: tiny shapes only.  Returns fp64 [M,N].
    """
    hd = parse_header(blob)
    q, G, N, K = hd["q"], hd["G"], hd["N"], hd["K"]
    geo = geometry(q, G, N, K)
    w, nsg, tb = geo["w"], geo["nsg"], geo["tile_bytes"]
    X64 = np.asarray(X, dtype=np.float64)
    M = X64.shape[0]
    Xp = np.zeros((M, geo["n_kc"] * CHUNK_K), dtype=np.float64)
    Xp[:, :K] = X64
    Y = np.zeros((M, geo["n_rb"] * TILE_ROWS), dtype=np.float64)
    for kc in range(geo["n_kc"]):
        for rb in range(geo["n_rb"]):
            base = HEADER_BYTES + (kc * geo["n_rb"] + rb) * tb
            pbase = base + geo["plane_bytes"]
            for lane in range(32):
                h, l = lane // 16, lane % 16
                a, r = l // w, l % w
                rec = []
                for e in range(geo["gl"] * (q + 1)):
                    o = pbase + ((e // 2) * 32 + lane) * 4 + 2 * (e % 2)
                    rec.append(float(np.ascontiguousarray(blob[o:o + 2]).view(np.float16)[0]))
                for u in range(2):
                    sigma = h + 2 * u
                    for v in range(nsg):
                        prm = rec[(u * nsg + v) * (q + 1):(u * nsg + v + 1) * (q + 1)]
                        sub = (a + v) % nsg
                        k_sub = kc * CHUNK_K + (16 * sigma + w * sub) * 8
                        xsum = Xp[:, k_sub:k_sub + G].sum(axis=1)
                        for j in range(q):
                            acc = np.zeros(M)
                            for ii in range(w):
                                i = v * w + ii
                                tau = w * sub + (r + ii) % w
                                byte = int(blob[base + ((u * q + j) * 32 + lane) * 16 + i])
                                k0 = kc * CHUNK_K + (16 * sigma + tau) * 8
                                for bit in range(8):
                                    if (byte >> bit) & 1:
                                        acc += Xp[:, k0 + bit]
                            Y[:, rb * TILE_ROWS + l] += prm[j] * acc
                        Y[:, rb * TILE_ROWS + l] += prm[q] * xsum
    return Y[:, :N]
