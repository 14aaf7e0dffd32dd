// Offline weight packer and its inverse (Sec. 3.4: weights are quantised to 4 bits offline).
// A pure permutation of codes, scales and zero points into the blob layout described in
// w4a8_internal.cuh; one CTA per blob (128 output channels x one group of 128 k).
#include "w4a8_internal.cuh"

namespace w4a8 {
namespace {

constexpr int PACK_THREADS = 256;

__global__ void __launch_bounds__(PACK_THREADS)
pack_weights_kernel(const uint8_t* __restrict__ qw, const uint16_t* __restrict__ scales,
                    const uint8_t* __restrict__ zeros, int N, int K, uint8_t* __restrict__ packed) {
    const int G = K / GROUP;
    const int ntile = blockIdx.x / G, g = blockIdx.x % G;
    uint8_t* blob = packed + (size_t)blockIdx.x * BLOB_BYTES;
    uint32_t* words = reinterpret_cast<uint32_t*>(blob);
    // 2048 words: word w = row r (w/16), word-in-row kk (w%16) <- four codes in its low nibbles, four in its high ones
    for (int w = threadIdx.x; w < TILE_N * 16; w += PACK_THREADS) {
        int r = w >> 4, kk = w & 15;
        const uint8_t* src = qw + (size_t)(ntile * TILE_N + r) * K + g * GROUP + blob_word_k(kk);
        const uint32_t lo = *reinterpret_cast<const uint32_t*>(src), hi = *reinterpret_cast<const uint32_t*>(src + 8);
        words[r * 16 + blob_chunk_pos(r, kk >> 2) * 4 + (kk & 3)] = (lo & 0x0F0F0F0Fu) | ((hi & 0x0F0F0F0Fu) << 4);
    }
    if (threadIdx.x < TILE_N) {
        int r = threadIdx.x;
        reinterpret_cast<uint16_t*>(blob + BLOB_SCALE_OFF)[r] = scales[(size_t)g * N + ntile * TILE_N + r];
    }
    if (threadIdx.x < TILE_N / 2) {
        int r = 2 * threadIdx.x;
        const uint8_t* zr = zeros + (size_t)g * N + ntile * TILE_N + r;
        blob[BLOB_ZERO_OFF + threadIdx.x] = (uint8_t)((zr[0] & 0xF) | ((zr[1] & 0xF) << 4));
    }
}

__global__ void __launch_bounds__(PACK_THREADS)
unpack_weights_kernel(const uint8_t* __restrict__ packed, int N, int K, uint8_t* __restrict__ qw,
                      uint16_t* __restrict__ scales, uint8_t* __restrict__ zeros) {
    const int G = K / GROUP;
    const int ntile = blockIdx.x / G, g = blockIdx.x % G;
    const uint8_t* blob = packed + (size_t)blockIdx.x * BLOB_BYTES;
    const uint32_t* words = reinterpret_cast<const uint32_t*>(blob);
    if (qw) {
        for (int w = threadIdx.x; w < TILE_N * 16; w += PACK_THREADS) {
            int r = w >> 4, kk = w & 15;
            uint32_t v = words[r * 16 + blob_chunk_pos(r, kk >> 2) * 4 + (kk & 3)];
            uint8_t* dst = qw + (size_t)(ntile * TILE_N + r) * K + g * GROUP + blob_word_k(kk);
            *reinterpret_cast<uint32_t*>(dst) = v & 0x0F0F0F0Fu;
            *reinterpret_cast<uint32_t*>(dst + 8) = (v >> 4) & 0x0F0F0F0Fu;
        }
    }
    if (threadIdx.x < TILE_N) {
        int r = threadIdx.x;
        if (scales)
            scales[(size_t)g * N + ntile * TILE_N + r] = reinterpret_cast<const uint16_t*>(blob + BLOB_SCALE_OFF)[r];
        if (zeros)
            zeros[(size_t)g * N + ntile * TILE_N + r] = (blob[BLOB_ZERO_OFF + (r >> 1)] >> ((r & 1) * 4)) & 0xF;
    }
}

}  // namespace

cudaError_t launch_pack_weights(const uint8_t* qw, const uint16_t* scales, const uint8_t* zeros,
                                int N, int K, void* packed, cudaStream_t stream) {
    int blobs = (N / TILE_N) * (K / GROUP);
    pack_weights_kernel<<<blobs, PACK_THREADS, 0, stream>>>(qw, scales, zeros, N, K, static_cast<uint8_t*>(packed));
    return cudaGetLastError();
}

cudaError_t launch_unpack_weights(const void* packed, int N, int K, uint8_t* qw, uint16_t* scales,
                                  uint8_t* zeros, cudaStream_t stream) {
    int blobs = (N / TILE_N) * (K / GROUP);
    unpack_weights_kernel<<<blobs, PACK_THREADS, 0, stream>>>(static_cast<const uint8_t*>(packed), N, K, qw, scales, zeros);
    return cudaGetLastError();
}

}  // namespace w4a8
