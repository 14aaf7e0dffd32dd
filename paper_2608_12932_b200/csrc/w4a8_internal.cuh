// Internal declarations shared by the translation units of libw4a8: packed layout
// constants, the workspace layout, kernel launchers.  Not part of the public ABI.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include "w4a8.h"

namespace w4a8 {

// ---- packed weight layout -----------------------------------------------------------------
// The [N,K] layer is cut into blobs of 128 output channels x one group of 128 k.  Blob
// (ntile, g) sits at byte offset (ntile * G + g) * BLOB_BYTES and holds
//   [0, 8192)     128 rows x 64 B of nibbles.  Row r, 32-bit word kk (0..15) belongs to the 16-byte chunk
//                 kk / 4, which covers 32 consecutive k.  Call the chunk's k range eight runs of four,
//                 a0..a7.  Word q = kk % 4 of the chunk has, byte by byte, run a(4 (q / 2) + q % 2) in its
//                 low nibbles and the run two further on in its high nibbles: words 0..3 hold
//                 (a0, a2), (a1, a3), (a4, a6), (a5, a7).   w & 0x0F0F0F0F  and  (w >> 4) & 0x0F0F0F0F
//                 are four consecutive-k bytes each, and the low nibbles of two neighbouring words go
//                 with two neighbouring 4-byte words of an activation row (so do the high ones): a
//                 warp-level MMA takes its two activation registers as they were loaded (blob_word_k).
//                 The four 16-byte chunks of a row are stored XOR-swizzled: chunk p of row r sits at
//                 position p ^ ((r >> 1) & 3) of the row (blob_chunk_pos).  A thread-per-row reader
//                 (16-byte loads at a 64-byte stride) then takes its four chunks without shared-memory
//                 bank conflicts: eight consecutive rows touch all eight 16-byte bank groups; a
//                 reader of two rows x four chunks per quarter-warp is conflict-free either way.
//   [8192, 8448)  128 fp16 scales, row order
//   [8448, 8512)  128 zero points, two per byte (row 2i low nibble, row 2i+1 high nibble)
// A blob is exactly the algorithmic 4.15625 bits per weight: no padding.
constexpr int TILE_N = 128;
__host__ __device__ constexpr int blob_chunk_pos(int r, int p) { return p ^ ((r >> 1) & 3); }
// first k (inside the group) of the four codes in the low nibbles of word kk of a row; the high nibbles start 8 later
__host__ __device__ constexpr int blob_word_k(int kk) { return 32 * (kk >> 2) + 16 * ((kk & 3) >> 1) + 4 * (kk & 1); }
constexpr int GROUP = 128;
constexpr int BLOB_NIBBLE_BYTES = TILE_N * GROUP / 2;        // 8192
constexpr int BLOB_SCALE_OFF = BLOB_NIBBLE_BYTES;             // 8192
constexpr int BLOB_ZERO_OFF = BLOB_SCALE_OFF + TILE_N * 2;    // 8448
constexpr int BLOB_BYTES = BLOB_ZERO_OFF + TILE_N / 2;        // 8512

// ---- workspace layout -----------------------------------------------------------------------
//   [0, 4)                    status word (0 = fine, else a w4a8_status written by a kernel)
//   [256, 256 + 4*n_tiles)    split-K arrival counters, one per 128-channel tile (zero between calls)
//   [HEADER, SHARED)          hand-over slots of the strip kernel: one per CTA, each word a float and a tag
//                             (all zero between calls: the tag is what says that a word has been written)
//   [SHARED, ...)             split-K fp32 slices  [S][M][N], or the tensor-core kernel's hand-over tiles
constexpr int WS_STATUS_OFF = 0;
constexpr int WS_FUSE_SYNC_OFF = 64;    // fused gate+up form: 16 per-token maxima, arrivals, departures (18 words)
constexpr int WS_COUNTER_OFF = 256;
constexpr int WS_HEADER_BYTES = W4A8_WORKSPACE_HEADER_BYTES;
constexpr int MAX_N_TILES = (WS_HEADER_BYTES - WS_COUNTER_OFF) / 4;   // 960 tiles = N up to 122880
constexpr int WS_SHARED_OFF = W4A8_WORKSPACE_ZEROED_BYTES;
// Hand-over area of the tcgen05 kernel's balanced walk (after the header, sharing the space of the split-K
// slices: the two are never in use at once): one fp32 tile of 208 x 128 per CTA; flags in the counter words.
constexpr int HANDOVER_SLOTS = 192;
inline size_t handover_bytes(int M, int N, int /*K*/) {
    // needed where the tcgen05 kernel can run (more than 16 tokens) with more tiles, at its shortest
    // tiling, than a small sm_100 part has SMs
    const long tiles = (long)((M + 63) / 64) * (N / TILE_N);
    return (M > 16 && tiles > 128) ? (size_t)HANDOVER_SLOTS * 208 * TILE_N * sizeof(float) : 0;
}

// ---- split-K path -----------------------------------------------------------------------------
constexpr int SPLITK_MAX_M = 64;          // tokens the streaming kernel handles (8 blocks of 8)
constexpr int SPLITK_MAX_GROUPS = 8;      // groups one CTA keeps in shared memory at once
int splitk_num_slices(int M, int N, int K);
int32_t* withhold_marker();

cudaError_t make_qa_tensor_map(CUtensorMap* out, const int8_t* qa, int M, int K, int box_rows);
cudaError_t make_y_tensor_map(CUtensorMap* out, void* y, int M, int N);
cudaError_t make_strip_weight_maps(CUtensorMap* nib, CUtensorMap* scale, CUtensorMap* zero, const void* packed,
                                   int N, int K, int R, int GS);
cudaError_t make_qa_group_map(CUtensorMap* out, const int8_t* qa, int M, int K, int box_rows, int box_groups);
cudaError_t launch_quantize_act(const void* x, int M, int K, int8_t* qa, uint16_t* sa, int32_t* asum,
                                cudaStream_t stream);
// h = bf16(SiLU(gate) * up) of a chunk-interleaved gate+up output y [M, 2 I], quantised like an activation row;
// h_out (bf16 [M, I]) may be null
cudaError_t launch_silu_mul_quantize(const void* y_gate_up, int M, int I, void* h_out, int8_t* qa, uint16_t* sa,
                                     int32_t* asum, cudaStream_t stream);
cudaError_t launch_pack_weights(const uint8_t* qw, const uint16_t* scales, const uint8_t* zeros,
                                int N, int K, void* packed, cudaStream_t stream);
cudaError_t launch_unpack_weights(const void* packed, int N, int K, uint8_t* qw, uint16_t* scales,
                                  uint8_t* zeros, cudaStream_t stream);
// `header` = the workspace's first WS_HEADER_BYTES (status word, counters), `slices` = room for the split-K slices
cudaError_t launch_gemm_splitk(const int8_t* qa, const uint16_t* sa, const int32_t* asum, const void* packed,
                               void* y, int M, int N, int K, void* header, float* slices, int32_t* debug_partials,
                               cudaStream_t stream);
void* static_scratch_address();              // device address of the static-scratch array on the current device, or NULL
// ---- strip path (up to 16 tokens) ---------------------------------------------------------------
constexpr int STRIP_MAX_M = 16;
constexpr int STRIP_MAX_CTAS = 192;                       // hand-over slots and flags in the workspace
constexpr int STRIP_SLOT_BYTES = TILE_N * STRIP_MAX_M * 8;  // one strip's fp32 sums, at most 128 channels x 16 tokens, 8 bytes each
static_assert(WS_HEADER_BYTES + STRIP_MAX_CTAS * STRIP_SLOT_BYTES == W4A8_WORKSPACE_ZEROED_BYTES, "strip slots fill the zeroed part");
bool strip_supported(int M, int N, int K);
void strip_plan(int M, int N, int K, int* strip_rows, int* ctas);
cudaError_t launch_gemm_strip(const int8_t* qa, const uint16_t* sa, const int32_t* asum, const void* packed,
                              void* y, const void* residual, int M, int N, int K, void* workspace, int32_t* debug_partials,
                              cudaStream_t stream);
// streaming prefill: rotary embedding of pre-rotation cached keys at shifted positions; the streaming attention mask
cudaError_t launch_rope_shifted_keys(const void* k_pre, const int32_t* pos, int delta, int T, int H, int D, double base,
                                     void* k_rot, cudaStream_t stream);
cudaError_t launch_streaming_mask(int V, int F, int n, uint8_t* mask, cudaStream_t stream);
// W4A16 (bf16 activations against the same packed weights), up to STRIP_MAX_M tokens
bool a16_supported(int M, int N, int K);
void a16_plan(int M, int N, int K, int* strip_rows, int* ctas);
cudaError_t launch_gemm_strip_a16(const void* x, const void* packed, void* y, int M, int N, int K, void* workspace,
                                  cudaStream_t stream);
cudaError_t launch_dequantize_weights(const void* packed, int N, int K, void* W_bf16, cudaStream_t stream);
cudaError_t make_x_half_group_map(CUtensorMap* out, const void* x, int M, int K, int box_rows, int box_halves);
// the strip kernel with the SiLU * up epilogue, then the requantisation of h: by a second small kernel, or
// (one_kernel) by the CTAs that arrive last (needs strip_supported and I % 128 == 0)
cudaError_t launch_gemm_strip_gate_up(const int8_t* qa, const uint16_t* sa, const int32_t* asum, const void* packed,
                                      int M, int N, int K, void* h, int8_t* qa_h, uint16_t* sa_h, int32_t* asum_h,
                                      bool one_kernel, void* workspace, cudaStream_t stream);
int device_sm_count();                       // SMs of the current device (cached per device)
int cluster_num_slices(int M, int N, int K);
// residual: null, or bf16 [M,N] added to the projection before the one rounding (may be y itself)
cudaError_t launch_gemm_cluster(const int8_t* qa, const uint16_t* sa, const int32_t* asum, const void* packed,
                                void* y, const void* residual, int M, int N, int K, void* workspace, int32_t* debug_partials,
                                cudaStream_t stream);
cudaError_t launch_gemm_tcgen05(const int8_t* qa, const uint16_t* sa, const void* packed, void* y, const void* residual,
                                int M, int N, int K, void* workspace, int32_t* debug_partials,
                                cudaStream_t stream);
cudaError_t launch_gemm_tcgen05_per_channel(const int8_t* qa, const uint16_t* sa, const void* packed, void* y,
                                            int M, int N, int K, void* workspace, int32_t* debug_sums,
                                            cudaStream_t stream);
// tile height, K split (at most max_split slices) and, if asked for, whether the balanced walk is taken, as the
// tcgen05 launcher picks them; returns its time estimate (ns)
long tcgen05_plan(int M, int N, int K, int sms, int* tile_m, int* split, int max_split = 4, int* balanced = nullptr);
bool small_m_prefers_tcgen05(int M, int N, int K, int sms);

}  // namespace w4a8
