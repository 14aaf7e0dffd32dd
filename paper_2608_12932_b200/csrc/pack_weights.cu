// Offline weight packer and its inverse (Sec. 3.4: weights are quantised to 4 bits offline).
// A pure permutation of codes, scales and zero points into the blob layout described in
// w4a8_internal.cuh; one CTA per blob (128 output channels x one group of 128 k).
#include <cuda_bf16.h>
#include <cuda_fp16.h>
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

// Dequantised weights for the weight-only (W4A16) form of a large-M product: W[n,k] = bf16(s_w (q_w - z)), row-major
// [N,K].  One CTA per blob, one thread per row: 64 packed bytes -> 128 bf16 (the product of an fp16 scale and an
// integer of magnitude <= 15 is exact in fp32, so there is one rounding).
__global__ void __launch_bounds__(TILE_N)
dequantize_weights_kernel(const uint8_t* __restrict__ packed, int N, int K, __nv_bfloat16* __restrict__ W) {
    const int G = K / GROUP;
    const int ntile = blockIdx.x / G, g = blockIdx.x % G;
    const uint8_t* blob = packed + (size_t)blockIdx.x * BLOB_BYTES;
    const int r = threadIdx.x;
    const float s = __half2float(reinterpret_cast<const __half*>(blob + BLOB_SCALE_OFF)[r]);
    const int z = (blob[BLOB_ZERO_OFF + (r >> 1)] >> ((r & 1) * 4)) & 0xF;
    __nv_bfloat16* dst = W + (size_t)(ntile * TILE_N + r) * K + g * GROUP;
    for (int p = 0; p < 4; ++p) {
        const uint4 c = *reinterpret_cast<const uint4*>(blob + r * 64 + blob_chunk_pos(r, p) * 16);
        const uint32_t w[4] = {c.x, c.y, c.z, c.w};
        __align__(16) __nv_bfloat16 out[32];
        for (int q = 0; q < 4; ++q) {
            const int k0 = blob_word_k(q);                          // inside the chunk: 0, 4, 16, 20
            for (int b = 0; b < 4; ++b) {
                out[k0 + b] = __float2bfloat16_rn(s * (float)((int)((w[q] >> (8 * b)) & 0xF) - z));
                out[k0 + 8 + b] = __float2bfloat16_rn(s * (float)((int)((w[q] >> (8 * b + 4)) & 0xF) - z));
            }
        }
        uint4* d4 = reinterpret_cast<uint4*>(dst + 32 * p);
        const uint4* o4 = reinterpret_cast<const uint4*>(out);
        d4[0] = o4[0]; d4[1] = o4[1]; d4[2] = o4[2]; d4[3] = o4[3];
    }
}

}  // namespace

cudaError_t launch_dequantize_weights(const void* packed, int N, int K, void* W_bf16, cudaStream_t stream) {
    int blobs = (N / TILE_N) * (K / GROUP);
    dequantize_weights_kernel<<<blobs, TILE_N, 0, stream>>>(static_cast<const uint8_t*>(packed), N, K,
                                                            static_cast<__nv_bfloat16*>(W_bf16));
    return cudaGetLastError();
}

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
