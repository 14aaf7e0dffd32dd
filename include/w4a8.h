/*
 * w4a8.h - C ABI of the B200 (sm_100a) W4A8 quantized linear layer.
 *
 * The operation is the paper's W4A8 scheme (Sec. 3.4, "Quantization": 4-bit weights,
 * 8-bit activations, INT8 matrix multiply).  The paper fixes no bit layout, group
 * size or rounding; this library uses:
 *
 *   weights      q_w[n,k] in 0..15; per (group of 128 consecutive k, output channel n)
 *                one fp16 scale s_w[g,n] and one zero point z[g,n] in 0..15
 *                (dequantised weight = s_w * (q_w - z))
 *   activations  per token m: s_a[m] = fp16_rne(max_k |x[m,k]| / 127), saturating at 65504;
 *                q_a[m,k] = clamp(round_half_even(x[m,k] / s_a[m]), -127, 127);
 *                a token whose scale is 0 has all codes 0
 *   partials     D[m,g,n] = sum_{k in g} q_w[n,k] q_a[m,k] - z[g,n] sum_{k in g} q_a[m,k]   (int32, exact)
 *   output       y[m,n]   = bf16_rne( s_a[m] * sum_g s_w[g,n] * D[m,g,n] )   (fp32 accumulation over g)
 *
 * M tokens, K in-features, N out-features, G = K / group.  y = x W^T with W stored [N,K].
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers owned by the caller (w4a8_linear_host marks its two
 *     HOST arguments).  Inputs are only read,
 *     outputs are fully overwritten.  Nothing is allocated or freed by the library.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  Work is
 *     enqueued on it; the host is never synchronised (w4a8_check_status excepted).
 *   - Errors are reported by return value only.  After W4A8_ERR_CUDA the CUDA error is
 *     left in place for cudaGetLastError().
 *   - Shapes: group must be 128, K a multiple of 128, N a multiple of 128, M >= 0
 *     (M == 0 returns W4A8_OK and enqueues nothing), otherwise W4A8_ERR_SHAPE.
 *   - The device must be compute capability 10.x, otherwise W4A8_ERR_ARCH.
 */
#ifndef W4A8_H_
#define W4A8_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    W4A8_OK = 0,
    W4A8_ERR_NULL = 1,       /* a required pointer is NULL                                   */
    W4A8_ERR_SHAPE = 2,      /* unsupported M, N, K or group                                 */
    W4A8_ERR_ALIGN = 3,      /* a pointer misses its stated alignment                        */
    W4A8_ERR_WORKSPACE = 4,  /* workspace_bytes < w4a8_workspace_bytes(M, N, K, group)       */
    W4A8_ERR_ARCH = 5,       /* current device is not sm_100                                 */
    W4A8_ERR_CUDA = 6,       /* a CUDA runtime/driver call failed                            */
    W4A8_ERR_TIMEOUT = 7     /* a bounded device-side wait expired (seen via check_status)   */
} w4a8_status;

/* Which GEMM kernel family w4a8_gemm_path runs. */
typedef enum {
    W4A8_PATH_AUTO = 0,      /* dispatch by M (what w4a8_gemm does)                          */
    W4A8_PATH_SPLITK = 1,    /* weight-streaming split-K kernel, slices reduced inside a
                                thread-block cluster through distributed shared memory (M <= 64) */
    W4A8_PATH_TCGEN05 = 2,   /* TMA + tcgen05.mma kind::i8 + TMEM kernel (any M)             */
    W4A8_PATH_SPLITK_WORKSPACE = 3, /* split-K kernel that reduces its slices through the global
                                workspace (M <= 64); what w4a8_gemm_static_scratch runs        */
    W4A8_PATH_STRIP = 4,     /* weight-streaming kernel without a K split: one persistent CTA per SM,
                                strips of 16..128 channels over the whole K range dealt out evenly
XX = 5     /* weight-streaming kernel on tcgen05: one persistent CTA per SM, the tiles x
                                groups blobs dealt out evenly, weights unpacked into tensor memory
                                (M <= 16)                                                       */
} w4a8_path;

const char* w4a8_status_string(w4a8_status s);

/* Size in bytes of the packed weight blob for an [N,K] layer; 0 for an unsupported shape. */
size_t w4a8_packed_bytes(int N, int K, int group);

/*
 * Size in bytes of the scratch workspace w4a8_gemm needs for any M <= M_max on this
 * layer shape (split-K slices or the tensor-core kernel's hand-over tiles, which share the space;
 * per-tile arrival counters and hand-over flags; the strip kernel's hand-over slots; one status
 * word); 0 for an unsupported shape.  The first W4A8_WORKSPACE_ZEROED_BYTES bytes (or the whole
 * workspace, if it is smaller) must be zero before the first call (w4a8_workspace_init does that)
 * and are left zero by every call, so one workspace can serve any number of calls that do not
 * overlap on the GPU.
 */
#define W4A8_WORKSPACE_HEADER_BYTES 4096
#define W4A8_WORKSPACE_ZEROED_BYTES (4096 + 192 * 16384)
size_t w4a8_workspace_bytes(int M_max, int N, int K, int group);
w4a8_status w4a8_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/*
 * Offline weight packing (Sec. 3.4: weights are quantised to 4 bits once, offline).  A pure
 * re-ordering of codes, scales and zero points into the layout the GEMM kernels stream.
 *   qw      [N,K] row-major, one code per byte (only the low 4 bits are used)
 *   scales  [K/group, N] fp16 bit patterns
 *   zeros   [K/group, N] one zero point per byte (low 4 bits)
 *   packed_out  w4a8_packed_bytes(N,K,group) bytes, 128-byte aligned
 */
w4a8_status w4a8_pack_weights(const uint8_t* qw, const uint16_t* scales, const uint8_t* zeros,
                              int N, int K, int group, void* packed_out, void* stream);

/* Inverse of w4a8_pack_weights (layout round-trip checks).  Any output pointer may be NULL. */
w4a8_status w4a8_unpack_weights(const void* packed, int N, int K, int group,
                                uint8_t* qw_out, uint16_t* scales_out, uint8_t* zeros_out,
                                void* stream);

/*
 * Per-token dynamic activation quantisation (Sec. 3.4: activations are quantised to 8 bits).
 *   x_bf16  [M,K] row-major, contiguous, 16-byte aligned
 *   qa      [M,K] int8, 16-byte aligned       sa  [M] fp16 bit patterns
 *   asum    [M,K/group] int32 sums of qa over each group (zero-point correction term)
 */
w4a8_status w4a8_quantize_act(const void* x_bf16, int M, int K, int group,
                              int8_t* qa, uint16_t* sa, int32_t* asum, void* stream);

/*
 * The quantised linear itself (Sec. 3.4: INT8 tensor-core matmul on 4-bit weights and
 * 8-bit activations; Sec. 4: memory-bound for decode-sized M, compute-bound for prefill).
 *   qa, sa, asum     outputs of w4a8_quantize_act (qa 16-byte aligned)
 *   packed_w         output of w4a8_pack_weights for the same N, K, group
 *   y_bf16           [M,N] row-major bf16, 16-byte aligned (the kernels store it in 8- and 16-byte pieces
 *                    and through a TMA map; W4A8_ERR_ALIGN otherwise, before anything is enqueued)
 *   workspace        >= w4a8_workspace_bytes(M,N,K,group) bytes, 256-byte aligned, header zeroed once
 *   debug_partials   NULL, or [M,K/group,N] int32 that receives D (slower debug mode)
 * Dispatch: up to 16 tokens the strip weight-streaming kernel, above 64 the tcgen05 kernel, in
 * between the cluster split-K kernel or the tcgen05 kernel, whichever a measured cost model predicts
 * faster for the shape (w4a8_plan tells which).
 * Results are run-to-run deterministic.
 * Programmatic dependent launch: w4a8_quantize_act, the weight-streaming kernels for up to 64
 * tokens and the tensor-core kernel are launched with programmatic stream serialisation (only the
 * workspace variant of the split-K kernel is launched plainly).  When consecutive library calls share a
 * stream, such a kernel may start, and prefetch packed weights, before its predecessor in the
 * stream has finished; it waits on the device before it reads any activation, token scale or group
 * sum, touches the workspace or writes any output.  packed_w is therefore the one argument that
 * must be complete before the call is enqueued: do not produce it with a kernel that sits
 * immediately ahead of the GEMM in the same stream (weights are packed once, offline).
 */
w4a8_status w4a8_gemm(const int8_t* qa, const uint16_t* sa, const int32_t* asum,
                      const void* packed_w, void* y_bf16,
                      int M, int N, int K, int group,
                      void* workspace, size_t workspace_bytes,
                      int32_t* debug_partials, void* stream);

/*
 * What w4a8_gemm would launch for a problem size on the current device (host-only query, nothing is
 * enqueued): the kernel family, for W4A8_PATH_STRIP the strip width, for W4A8_PATH_SPLITK the number of
 * K slices per 128-channel tile (cluster size), for W4A8_PATH_TCGEN05 the token-tile height (64, 128 or 208) and the number of K
 * slices (1 = no split).  Any output pointer may be NULL.  W4A8_ERR_SHAPE for an unsupported shape.
 */
typedef struct {
    w4a8_path family;   /* W4A8_PATH_STRIP, W4A8_PATH_SPLITK or W4A8_PATH_TCGEN05 */
    int tile_m;         /* tcgen05: token rows per tile; strip and split-K: 8 x token blocks per CTA (8, 16, 32 or 64) */
    int k_slices;       /* CTAs that share the K range of one tile (strip: always 1) */
    int ctas;           /* CTAs of the launch */
    int balanced;       /* tcgen05, more tiles than CTAs: 1 if the tiles x groups units are dealt out evenly, so that
                           neighbouring CTAs share a tile and hand partial sums over through the workspace;
                           strip: 1 if the strips do not divide evenly among the CTAs (same hand-over) */
    int strip_rows;     /* strip: output channels per strip (16, 32, 64 or 128); 0 otherwise */
} w4a8_plan_info;
w4a8_status w4a8_plan(int M, int N, int K, int group, w4a8_plan_info* out);

/*
 * w4a8_gemm with the residual stream added in its epilogue (Sec. 3.5, "Kernel Fusion": element-wise steps are
 * merged into their neighbours; the O and down projections of a decoder layer feed the residual stream):
 *   y[m,n] = bf16_rne( sa[m] * sum_groups sw[g,n] * D[m,g,n] + r[m,n] )      one rounding, the sum in fp32
 *   residual  device, bf16 [M,N] row-major, 16-byte aligned; may be the same buffer as y (every element is read by
 *             the thread or warp that then overwrites it)
 *   path      W4A8_PATH_AUTO in production; the strip, cluster split-K and tensor-core families have the epilogue,
 *             W4A8_PATH_SPLITK_WORKSPACE does not (W4A8_ERR_SHAPE)
 * Other arguments, alignment, workspace and errors as for w4a8_gemm.  Judged against the fp64 sum with the
 * projection's band plus half a bf16 step of the sum.
 */
w4a8_status w4a8_gemm_residual(w4a8_path path, const int8_t* qa, const uint16_t* sa, const int32_t* asum,
                               const void* packed_w, const void* residual_bf16, void* y_bf16,
                               int M, int N, int K, int group,
                               void* workspace, size_t workspace_bytes, void* stream);

/*
 * The step after the fused gate+up projection (Sec. 3.5, "Kernel Fusion": gate and up are one GEMM, and
 * the element-wise operations that follow are merged into their neighbours): from the projection's
 * output to the quantised input of the down projection, h never making a round trip as a separate pass.
 *
 *   h[m,c]  = bf16_rne( SiLU(gate[m,c]) * up[m,c] ),  SiLU(v) = v / (1 + exp(-v)),  gate and up the bf16
 *             outputs of the projection; evaluated in fp32 with the fast exponential (h equals the exactly
 *             computed value or its bf16 neighbour)
 *   (qa_h, sa_h, asum_h) = the activation quantisation of w4a8_quantize_act applied to h (bit-exact
 *             given h): the operands w4a8_gemm takes for the down projection.
 *
 * Channel layout of the fused layer (this library's reading; the paper gives none): its N = 2 I output
 * channels alternate in runs of eight - channel n = 16 b + i is gate channel 8 b + i for i < 8 and up
 * channel 8 b + i - 8 for i >= 8.  A 16-byte piece of an output row is thus eight gate values or the eight
 * up values of the same indices, and the gate and up of one channel meet in one thread of the GEMM's
 * epilogue.  The caller orders the rows of the two weight matrices so before w4a8_pack_weights; the
 * packed format itself is unchanged.
 *
 * w4a8_silu_mul_quantize: the step alone, for a projection output that is already in memory.
 *   y_gate_up  device, bf16 [M, 2 I] in the layout above (16-byte aligned)
 *   h          device, bf16 [M, I], receives h; may be NULL
 *   qa_h       device, int8 [M, I]; sa_h fp16 [M]; asum_h int32 [M, I / 128]
 *   I % 128 == 0, group == 128.  One kernel, one CTA per token.
 *
 * w4a8_gate_up_silu_quantize: projection and step together, in one of three forms (results identical bit for bit):
 *   W4A8_GATE_UP_EPILOGUE    the strip kernel's epilogue forms h from its own sums, stores it and keeps each token's
 *                            largest |h| (atomic maxima); y is never stored.  A second, small kernel (one warp per token
 *                            and group of 128) quantises h once the maxima are final: the kernel boundary is the
 *                            grid-wide wait.  Where the strip kernel runs (M <= 16, see w4a8_plan).
 *   W4A8_GATE_UP_ONE_KERNEL  the same epilogue, but the requantisation stays inside the kernel: every CTA counts itself in,
 *                            the last 128 to arrive stay, wait (bounded) until all have, and quantise.  One launch fewer;
 *                            measured slower than the form above on B200 (the stayers' wait for the last stores of h to
 *                            become visible costs more than a dependent launch), kept for comparison.
 *   W4A8_GATE_UP_SEPARATE    w4a8_gemm into y_scratch, then w4a8_silu_mul_quantize.  Any M.
 *   W4A8_GATE_UP_AUTO        EPILOGUE where w4a8_gemm would take the strip kernel, else SEPARATE (w4a8_gate_up_form says
 *                            which, 0 for an unsupported shape).
 *   qa, sa, asum, packed_gate_up, M, N (= 2 I), K, group, workspace: as for w4a8_gemm
 *   h          device, bf16 [M, I]: output, and in the first two forms also the buffer through which h reaches the
 *              warps that quantise it (required)
 *   y_scratch  device, bf16 [M, N]; needed only by the SEPARATE form, else may be NULL
 * Errors as for w4a8_gemm; W4A8_ERR_SHAPE also for I % 128 != 0, an unknown form, or a strip-kernel form where that kernel
 * does not exist (M > 16).  The strip-kernel forms keep 18 words of the workspace header (per-token maxima and two
 * counters) that they leave zero; after W4A8_ERR_TIMEOUT the workspace must be initialised again before its next use.
 */
typedef enum {
    W4A8_GATE_UP_AUTO = 0,
    W4A8_GATE_UP_ONE_KERNEL = 1,
    W4A8_GATE_UP_EPILOGUE = 2,
    W4A8_GATE_UP_SEPARATE = 3
} w4a8_gate_up_form_t;
w4a8_status w4a8_silu_mul_quantize(const void* y_gate_up_bf16, int M, int I, int group, void* h_bf16,
                                   int8_t* qa_h, uint16_t* sa_h, int32_t* asum_h, void* stream);
int w4a8_gate_up_form(int M, int N, int K, int group);
w4a8_status w4a8_gate_up_silu_quantize(int form, const int8_t* qa, const uint16_t* sa, const int32_t* asum,
                                       const void* packed_gate_up, int M, int N, int K, int group,
                                       void* h_bf16, int8_t* qa_h, uint16_t* sa_h, int32_t* asum_h,
                                       void* y_scratch_bf16, void* workspace, size_t workspace_bytes,
                                       void* stream);

/*
 * Two pieces of streaming prefill that sit beside the quantised linears (Sec. 3.1, "Streaming design").
 *
 * w4a8_rope_shifted_keys: keys are cached before the rotary embedding, because a cached token's position changes
 * when the window slides; the rotation is applied at use, at the shifted position pos[t] - delta.  Rotate-half
 * form (this library's reading; the paper names no variant): for i < D/2, theta_i = base^(-2i/D),
 * phi = (pos[t] - delta) theta_i,
 *   out[t,h,i] = k[t,h,i] cos(phi) - k[t,h,i+D/2] sin(phi),  out[t,h,i+D/2] = k[t,h,i+D/2] cos(phi) + k[t,h,i] sin(phi)
 * The angle is formed and reduced in fp64, sine, cosine, products and sums are fp32, one rounding to bf16 (equal to
 * the fp64 definition's bf16 or its neighbour).
 *   k_pre, k_rot  device, bf16 [T,H,D] row-major, 4-byte aligned (may be the same buffer: a thread reads the four
 *                 values it then writes);  pos  device, int32 [T];  D % 4 == 0;  base > 1 (e.g. 1e6)
 *
 * w4a8_streaming_mask: the new frame's tokens take the last-frame place of each camera view (the sequence is
 * view-major: all frames of one view before the next), only they are queries, attention stays causal in that order:
 *   mask[q][j] = 1 iff j <= position of query q,  query q = (view v, token i) at position (v frames + frames - 1) n + i
 *   mask  device, uint8 [views * n, views * frames * n] row-major.  (The paper's figure of the mask is not
 *   available; this is its caption written out.)
 */
w4a8_status w4a8_rope_shifted_keys(const void* k_pre_bf16, const int32_t* pos, int delta, int T, int H, int D,
                                   double base, void* k_rot_bf16, void* stream);
w4a8_status w4a8_streaming_mask(int views, int frames, int tokens_per_frame, uint8_t* mask, void* stream);

/*
 * The weight-only variant the paper contrasts W4A8 with (Sec. 3.4, first paragraph: 4-bit weights with 16-bit
 * activations shrink what the memory-bound decode must load, and leave the arithmetic of the compute-bound
 * prefill in 16-bit floating point).  Same packed weights, activations NOT quantised:
 *   y[m,n] = bf16( sum_groups s_w[g,n] * sum_{k in g} x[m,k] (q_w[n,k] - z[g,n]) )
 * w4a8_a16_gemm: the decode form, 1 <= M <= 16 (W4A8_ERR_SHAPE above): the strip kernel's streaming skeleton with
 * bf16 tensor-core MMAs; a code minus its zero point is an exact bf16 integer, products are exact in fp32, a group's
 * sum is scaled in fp32: no weight is rounded before it is multiplied.  Judged with the same band as w4a8_gemm
 * against the fp64 definition.
 *   x        device, bf16 [M,K] row-major, 16-byte aligned
 *   packed_w, y, N, K, group, workspace: as for w4a8_gemm
 * w4a8_dequantize_weights: the prefill form's first half: W[n,k] = bf16_rne(s_w (q_w - z)), row-major [N,K] bf16
 * (device, 16-byte aligned), for a library bf16 GEMM; one rounding per weight, bit-exact against the definition.
 */
w4a8_status w4a8_a16_gemm(const void* x_bf16, const void* packed_w, void* y_bf16, int M, int N, int K, int group,
                          void* workspace, size_t workspace_bytes, void* stream);
w4a8_status w4a8_dequantize_weights(const void* packed_w, int N, int K, int group, void* w_bf16, void* stream);

/*
 * Variant for weights whose scale does not change along K (per-channel scales: the paper does not
 * give its group size, Sec. 3.4; this is the coarsest choice, group 128 the library's default).
 * Same packed format and the same per-group zero points; the caller guarantees that the scales of
 * a channel are equal in every group (only those of the first group are read).  The int32 sums of
 * all groups then add up in one tensor-memory accumulator and a tile is scaled once:
 *   y[m,n] = bf16( sa[m] * sw[n] * sum_groups D[m,group,n] )
 * which equals w4a8_gemm's result up to fp32 rounding order.  tcgen05 kernel for every M.
 *   debug_sums   NULL, or [M,N] int32 that receives sum_groups D (exact)
 * K <= 2^19.  Other arguments, alignment, workspace and errors as for w4a8_gemm.
 */
w4a8_status w4a8_gemm_per_channel(const int8_t* qa, const uint16_t* sa,
                                  const void* packed_w, void* y_bf16,
                                  int M, int N, int K, int group,
                                  void* workspace, size_t workspace_bytes,
                                  int32_t* debug_sums, void* stream);

/* w4a8_gemm with the kernel family forced (path-consistency tests, benchmarking). */
w4a8_status w4a8_gemm_path(w4a8_path path,
                           const int8_t* qa, const uint16_t* sa, const int32_t* asum,
                           const void* packed_w, void* y_bf16,
                           int M, int N, int K, int group,
                           void* workspace, size_t workspace_bytes,
                           int32_t* debug_partials, void* stream);

/*
 * The whole path on device buffers: y = W4A8 linear of bf16 activations, i.e. w4a8_quantize_act
 * followed by w4a8_gemm on the same stream (Sec. 3.4); two kernel launches, chained with
 * programmatic dependent launch so that the GEMM's weight stream starts under the quantiser.
 * (A single-kernel form, in which the small-M GEMM quantises its own activations, was built and
 * measured slower: every CTA then repeats the row-maximum and division work of the quantiser.)
 *   x_bf16   [M,K] bf16 bits, contiguous, 16-byte aligned
 *   y_bf16   [M,N] bf16 bits, 16-byte aligned, fully overwritten
 *   qa, sa, asum   as for w4a8_quantize_act: required scratch, holding the quantised activations afterwards
 * Same shape rules, workspace and status codes as w4a8_gemm.
 */
w4a8_status w4a8_linear(const void* x_bf16, const void* packed_w, void* y_bf16,
                        int M, int N, int K, int group,
                        int8_t* qa, uint16_t* sa, int32_t* asum,
                        void* workspace, size_t workspace_bytes, void* stream);

/*
 * The whole path for callers whose activations and results live in HOST memory (Sec. 3.5: a
 * pipeline stage is one graph launch fed from the host): enqueues, on `stream`, the copy of
 * x to the device, w4a8_linear, and the copy of y back to the host.
 *   x_host_bf16  HOST [M,K] bf16 (pinned memory makes the copies asynchronous)
 *   y_host_bf16  HOST [M,N] bf16, valid once `stream` has been synchronised by the caller
 *   x_dev, qa, sa, asum, y_dev   DEVICE staging buffers owned by the caller, sized and aligned
 *                as for w4a8_quantize_act / w4a8_gemm ([M,K] bf16, [M,K] int8, [M] fp16,
 *                [M,K/group] int32, [M,N] bf16; x_dev and y_dev 16-byte aligned)
 * Every argument is checked before the first copy is enqueued.  Same shape rules and status codes as w4a8_gemm.
 */
w4a8_status w4a8_linear_host(const void* x_host_bf16, void* y_host_bf16,
                             int M, int N, int K, int group, const void* packed_w,
                             void* x_dev, int8_t* qa, uint16_t* sa, int32_t* asum, void* y_dev,
                             void* workspace, size_t workspace_bytes, void* stream);

/*
 * w4a8_gemm for callers that cannot allocate device memory.  (The paper has no counterpart to
 * this entry point; it exists for deployment reasons only.)  Some hosts of this library may
 * not call cudaMalloc at all: a control loop with a hard deadline cannot afford the
 * device-wide synchronisation and unbounded latency an allocation may cost, and a component
 * running inside another runtime's pre-partitioned memory pool has no allocator of its own to
 * obtain a workspace from.  For them the split-K scratch (slices, arrival counters, status word)
 * is a fixed array of W4A8_STATIC_SCRATCH_BYTES bytes inside the library image; every GPU that
 * loads the library holds that much memory until the process exits.
 *   - Same inputs, output and shape rules as w4a8_gemm, restricted to the split-K path: M <= 64.
 *   - A shape whose scratch need (4096 + S*M*N*4 bytes, S = number of K slices the library
 *     picks for N and K) exceeds W4A8_STATIC_SCRATCH_BYTES is refused with W4A8_ERR_WORKSPACE;
 *     nothing is enqueued.
 *   - Calls no cudaMalloc, cudaFree or other allocating routine.  The first call on each device
 *     performs a one-time set-up (it looks up the array's device address and sets a kernel
 *     attribute); make that first call before starting any stream capture.
 *   - All calls on a device share the one array, and each call zeroes the array's arrival
 *     counters on `stream` before its kernel: two calls that overlap on the GPU (different
 *     streams) race.  Serialise them on one stream.
 *   - y_bf16 needs only 2-byte alignment here (this kernel stores element by element).
 *   - The status word of this path sits in the array too: w4a8_static_scratch_status reads it
 *     the way w4a8_check_status reads a workspace's (synchronises `stream`; W4A8_OK, or
 *     W4A8_ERR_TIMEOUT if a kernel of an earlier call gave up on a bounded wait; clears it).
 */
#define W4A8_STATIC_SCRATCH_BYTES (4096 + 4 * 1024 * 1024)
w4a8_status w4a8_gemm_static_scratch(const int8_t* qa, const uint16_t* sa, const int32_t* asum,
                                     const void* packed_w, void* y_bf16,
                                     int M, int N, int K, int group, void* stream);
w4a8_status w4a8_static_scratch_status(void* stream);

/*
 * Self-test of the kernels' give-up path (no counterpart in the paper).  Runs the workspace split-K kernel on the
 * given problem (M <= 64) in a form in which every CTA leaves one of its weight copies out and waits for at most
 * 200 microseconds: the wait expires, the CTA records W4A8_ERR_TIMEOUT in the workspace status word, waits (again
 * bounded) for its copies in flight and the kernel returns normally.  y_bf16 is written but invalid.  Afterwards
 * w4a8_check_status returns W4A8_ERR_TIMEOUT once and the workspace is usable as before.  Nothing faults or hangs.
 */
w4a8_status w4a8_selftest_wait_timeout(const int8_t* qa, const uint16_t* sa, const int32_t* asum, const void* packed_w,
                                       void* y_bf16, int M, int N, int K, int group, void* workspace,
                                       size_t workspace_bytes, void* stream);

/*
 * Reads back the workspace status word: synchronises `stream`, returns W4A8_OK or
 * W4A8_ERR_TIMEOUT (a kernel gave up on a bounded wait; its output is then invalid), and
 * clears the word.  Host-synchronising: for tests and debugging, not for the hot path.
 */
w4a8_status w4a8_check_status(void* workspace, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* W4A8_H_ */
