// Offline packing of HLQ bit-planes, scales and offsets into the device layout, and its inverse.
//
// Packing runs in gather form: every thread owns one 16-byte plane vector (or one 32-bit
// parameter word) of the output and collects the logical elements that belong there.
// Unpacking runs per logical element.  Neither is on the per-token path.
#include "common.cuh"

namespace elutq {

namespace {

__global__ void write_header_kernel(uint32_t* hdr, Geo g) {
    const int i = threadIdx.x;
    if (i >= ELUTQ_HEADER_BYTES / 4) return;
    uint32_t v = 0;
    switch (i) {
        case 0: v = (uint32_t)kMagic; break;
        case 1: v = (uint32_t)kVersion; break;
        case 2: v = (uint32_t)g.q; break;
        case 3: v = (uint32_t)g.G; break;
        case 4: v = (uint32_t)g.N; break;
        case 5: v = (uint32_t)g.K; break;
        case 6: v = (uint32_t)g.n_rb; break;
        case 7: v = (uint32_t)g.n_kc; break;
        case 8: v = (uint32_t)g.tile_bytes; break;
        default: break;
    }
    hdr[i] = v;
}

// One thread per plane vector: (tile, vec = u*q + j, lane) -> 16 bytes, byte i = column tau(l,i).
__global__ void pack_planes_kernel(const uint8_t* __restrict__ planes, uint8_t* __restrict__ tiles, Geo g) {
    const long long nvec = (long long)g.n_kc * g.n_rb * 2 * g.q * 32;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= nvec) return;
    const int lane = (int)(idx & 31);
    const int vec = (int)((idx >> 5) % (2 * g.q));
    const long long tile = idx / (64LL * g.q);
    const int kc = (int)(tile / g.n_rb), rb = (int)(tile % g.n_rb);
    const int u = vec / g.q, j = vec % g.q;
    const int h = lane >> 4, l = lane & 15;
    const int n = rb * kTileRows + l;
    const int sigma = h + 2 * u;
    uint32_t out[4] = {0u, 0u, 0u, 0u};
    if (n < g.N) {
        const uint8_t* row = planes + ((size_t)j * g.N + n) * g.K;
        for (int i = 0; i < 16; ++i) {
            const int k0 = kc * kChunkK + (16 * sigma + tau_of(l, i, g.w, g.nsg)) * 8;
            uint32_t byte = 0;
            if (k0 < g.K) {
                const uint64_t x = *reinterpret_cast<const uint64_t*>(row + k0);
#pragma unroll
                for (int b = 0; b < 8; ++b) byte |= (((x >> (8 * b)) & 0xffull) != 0ull ? 1u : 0u) << b;
            }
            out[i >> 2] |= byte << (8 * (i & 3));
        }
    }
    uint4* dst = reinterpret_cast<uint4*>(tiles + (size_t)tile * g.tile_bytes) + vec * 32 + lane;
    *dst = make_uint4(out[0], out[1], out[2], out[3]);
}

// One thread per parameter word: (tile, word, lane) -> two fp16 values of the lane's record.
__global__ void pack_params_kernel(const uint16_t* __restrict__ scales, const uint16_t* __restrict__ offsets,
                                   uint8_t* __restrict__ tiles, Geo g) {
    const int words = g.gl * (g.q + 1) / 2;
    const long long total = (long long)g.n_kc * g.n_rb * words * 32;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int lane = (int)(idx & 31);
    const int word = (int)((idx >> 5) % words);
    const long long tile = idx / (32LL * words);
    const int kc = (int)(tile / g.n_rb), rb = (int)(tile % g.n_rb);
    const int h = lane >> 4, l = lane & 15;
    const int n = rb * kTileRows + l;
    const int Gn = g.K / g.G;
    const int a = l / g.w;
    uint32_t packed = 0;
    for (int half = 0; half < 2; ++half) {
        const int e = 2 * word + half;
        const int comp = e % (g.q + 1);
        const int uv = e / (g.q + 1);
        const int u = uv / g.nsg, v = uv % g.nsg;
        const int gamma = g.nsg * (h + 2 * u) + (a + v) % g.nsg;    // group inside the chunk
        const int gi = kc * (kChunkK / g.G) + gamma;
        uint32_t bits = 0;
        if (n < g.N && gi < Gn)
            bits = comp < g.q ? scales[((size_t)n * Gn + gi) * g.q + comp] : offsets[(size_t)n * Gn + gi];
        packed |= bits << (16 * half);
    }
    uint32_t* dst = reinterpret_cast<uint32_t*>(tiles + (size_t)tile * g.tile_bytes + g.plane_bytes) + word * 32 + lane;
    *dst = packed;
}

// One thread per (plane j, row n, byte-column cg): expands a packed byte to 8 uint8 {0,1}.
__global__ void unpack_planes_kernel(const uint8_t* __restrict__ tiles, uint8_t* __restrict__ planes, Geo g) {
    if (!blob_header_matches(tiles, g.q, g.G, g.N, g.K, nullptr)) return;   // before any tile is read
    const int cols = g.K / 8;
    const long long total = (long long)g.q * g.N * cols;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int cg = (int)(idx % cols);
    const int n = (int)((idx / cols) % g.N);
    const int j = (int)(idx / ((long long)cols * g.N));
    const int rb = n / kTileRows, l = n % kTileRows;
    const int kc = cg / 64, c = cg % 64;
    const int sigma = c / 16, tau = c % 16;
    const int h = sigma & 1, u = sigma >> 1;
    const int sg = tau / g.w, rr = tau % g.w;
    const int a = l / g.w, r = l % g.w;
    const int v = (sg - a + g.nsg) % g.nsg;
    const int ii = (rr - r + g.w) % g.w;
    const int i = v * g.w + ii;
    const size_t off = ((size_t)kc * g.n_rb + rb) * g.tile_bytes + ((size_t)(u * g.q + j) * 32 + 16 * h + l) * 16 + i;
    const uint32_t byte = tiles[off];
    uint64_t x = 0;
#pragma unroll
    for (int b = 0; b < 8; ++b) x |= (uint64_t)((byte >> b) & 1u) << (8 * b);
    *reinterpret_cast<uint64_t*>(planes + ((size_t)j * g.N + n) * g.K + (size_t)cg * 8) = x;
}

// One thread per (row n, group gi, component): copies one fp16 parameter back.
__global__ void unpack_params_kernel(const uint8_t* __restrict__ tiles, uint16_t* __restrict__ scales,
                                     uint16_t* __restrict__ offsets, Geo g) {
    if (!blob_header_matches(tiles, g.q, g.G, g.N, g.K, nullptr)) return;   // before any tile is read
    const int Gn = g.K / g.G;
    const long long total = (long long)g.N * Gn * (g.q + 1);
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= total) return;
    const int comp = (int)(idx % (g.q + 1));
    const int gi = (int)((idx / (g.q + 1)) % Gn);
    const int n = (int)(idx / ((long long)(g.q + 1) * Gn));
    const int rb = n / kTileRows, l = n % kTileRows;
    const int gpc = kChunkK / g.G;
    const int kc = gi / gpc, gamma = gi % gpc;
    const int sigma = gamma / g.nsg, sg = gamma % g.nsg;
    const int h = sigma & 1, u = sigma >> 1;
    const int a = l / g.w;
    const int v = (sg - a + g.nsg) % g.nsg;
    const int e = (u * g.nsg + v) * (g.q + 1) + comp;
    const size_t off = ((size_t)kc * g.n_rb + rb) * g.tile_bytes + g.plane_bytes + ((size_t)(e / 2) * 32 + 16 * h + l) * 4 + 2 * (e % 2);
    const uint16_t bits = *reinterpret_cast<const uint16_t*>(tiles + off);
    if (comp < g.q) scales[((size_t)n * Gn + gi) * g.q + comp] = bits;
    else offsets[(size_t)n * Gn + gi] = bits;
}

inline unsigned blocks_for(long long total, int threads) { return (unsigned)((total + threads - 1) / threads); }

}  // namespace

int launch_pack(const uint8_t* planes, const __half* scales, const __half* offsets, const Geo& g,
                uint8_t* packed, cudaStream_t stream) {
    uint8_t* tiles = packed + ELUTQ_HEADER_BYTES;
    write_header_kernel<<<1, 32, 0, stream>>>(reinterpret_cast<uint32_t*>(packed), g);
    const long long nvec = (long long)g.n_kc * g.n_rb * 2 * g.q * 32;
    pack_planes_kernel<<<blocks_for(nvec, 256), 256, 0, stream>>>(planes, tiles, g);
    const long long nwords = (long long)g.n_kc * g.n_rb * (g.gl * (g.q + 1) / 2) * 32;
    pack_params_kernel<<<blocks_for(nwords, 256), 256, 0, stream>>>(
        reinterpret_cast<const uint16_t*>(scales), reinterpret_cast<const uint16_t*>(offsets), tiles, g);
    count_launch(3);
    return (int)cudaGetLastError();
}

int launch_unpack(const uint8_t* packed, const Geo& g, uint8_t* planes, __half* scales, __half* offsets,
                  cudaStream_t stream) {
    const uint8_t* tiles = packed + ELUTQ_HEADER_BYTES;
    const long long nb = (long long)g.q * g.N * (g.K / 8);
    unpack_planes_kernel<<<blocks_for(nb, 256), 256, 0, stream>>>(tiles, planes, g);
    const long long np = (long long)g.N * (g.K / g.G) * (g.q + 1);
    unpack_params_kernel<<<blocks_for(np, 256), 256, 0, stream>>>(
        tiles, reinterpret_cast<uint16_t*>(scales), reinterpret_cast<uint16_t*>(offsets), g);
    count_launch(2);
    return (int)cudaGetLastError();
}

}  // namespace elutq
