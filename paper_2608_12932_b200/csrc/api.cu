// extern "C" boundary of libw4a8: argument validation, dispatch by M, status codes.
// Every step of the path runs in the CUDA kernels; nothing here touches the data.
#include <cuda_runtime.h>
#include "w4a8_internal.cuh"

using namespace w4a8;

namespace {

bool shape_ok(int N, int K, int group) {
    return group == GROUP && N > 0 && K > 0 && N % TILE_N == 0 && K % GROUP == 0 && N / TILE_N <= MAX_N_TILES;
}
bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

w4a8_status arch_check() {
    static int cached[64] = {0};      // 0 unknown, 1 ok, 2 wrong arch
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return W4A8_ERR_CUDA;
    if (dev < 0 || dev >= 64) return W4A8_ERR_CUDA;
    if (!cached[dev]) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return W4A8_ERR_CUDA;
        cached[dev] = (major == 10) ? 1 : 2;
    }
    return cached[dev] == 1 ? W4A8_OK : W4A8_ERR_ARCH;
}

}  // namespace

namespace w4a8 {

int device_sm_count() {
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (!cached[dev]) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

// Between 17 and 64 tokens both kernel families are valid.  Measured on B200 (nanoseconds, cold
// weights): the streaming kernel costs about 4200 + 570 per group a CTA walks, times the number of
// CTAs per SM, up to 32 tokens; above, where it walks the token blocks twice, about 7000 + 1140 per
// group.  The tensor-core kernel's estimate comes from its own planner (tile height, K split, walk).
bool small_m_prefers_tcgen05(int M, int N, int K, int sms) {
    if (M <= 16 || M > SPLITK_MAX_M) return M > SPLITK_MAX_M;
    const long G = K / GROUP, tiles = N / TILE_N, S = cluster_num_slices(M, N, K);
    const long groups = ((G + S - 1) / S) * ((tiles * S + sms - 1) / sms);
    const long streaming_ns = M <= 32 ? 4200 + 570 * groups : 7000 + 1140 * groups;
    int tile_m = 0, split = 0, balanced = 0;
    return tcgen05_plan(M, N, K, sms, &tile_m, &split, 4, &balanced) < streaming_ns;      // as the launcher calls it
}

}  // namespace w4a8

namespace {

// Where w4a8_gemm takes the strip kernel: up to 8 tokens always; from 9 to 16 tokens (two token blocks per warp:
// the activation tiles then crowd the ring of a narrow strip) only on layers wide enough for strips of 32 rows,
// where it is measured faster than the cluster split-K kernel on B200.
bool auto_takes_strip(int M, int N, int K) {
    if (!strip_supported(M, N, K)) return false;
    return M <= 8 || N / 32 >= (device_sm_count() * 5) / 4;
}

size_t slices_bytes(int M, int N, int K) {
    const int m = M < SPLITK_MAX_M ? M : SPLITK_MAX_M;
    const int S = splitk_num_slices(m, N, K);
    return S > 1 ? (size_t)S * m * N * sizeof(float) : 0;
}

}  // namespace

extern "C" {

const char* w4a8_status_string(w4a8_status s) {
    switch (s) {
        case W4A8_OK: return "ok";
        case W4A8_ERR_NULL: return "null pointer";
        case W4A8_ERR_SHAPE: return "unsupported shape (need group == 128, K % 128 == 0, N % 128 == 0, M >= 0)";
        case W4A8_ERR_ALIGN: return "misaligned pointer";
        case W4A8_ERR_WORKSPACE: return "workspace too small";
        case W4A8_ERR_ARCH: return "device is not sm_100";
        case W4A8_ERR_CUDA: return "CUDA call failed";
        case W4A8_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

size_t w4a8_packed_bytes(int N, int K, int group) {
    if (!shape_ok(N, K, group)) return 0;
    return (size_t)(N / TILE_N) * (K / GROUP) * BLOB_BYTES;
}

size_t w4a8_workspace_bytes(int M_max, int N, int K, int group) {
    if (!shape_ok(N, K, group) || M_max < 0) return 0;
    // header, then the strip kernel's hand-over slots (zero between calls), then an area shared by the split-K
    // slices and the tensor-core kernel's hand-over tiles, which are never in use at once
    if (M_max == 0) return WS_HEADER_BYTES;
    const size_t a = slices_bytes(M_max, N, K), b = handover_bytes(M_max, N, K);
    return WS_SHARED_OFF + (a > b ? a : b);
}

w4a8_status w4a8_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
    if (!workspace) return W4A8_ERR_NULL;
    if (workspace_bytes < WS_HEADER_BYTES) return W4A8_ERR_WORKSPACE;
    if (!aligned(workspace, 256)) return W4A8_ERR_ALIGN;
    const size_t zeroed = workspace_bytes < (size_t)W4A8_WORKSPACE_ZEROED_BYTES ? workspace_bytes : (size_t)W4A8_WORKSPACE_ZEROED_BYTES;
    if (cudaMemsetAsync(workspace, 0, zeroed, static_cast<cudaStream_t>(stream)) != cudaSuccess)
        return W4A8_ERR_CUDA;
    return W4A8_OK;
}

w4a8_status w4a8_pack_weights(const uint8_t* qw, const uint16_t* scales, const uint8_t* zeros,
                              int N, int K, int group, void* packed_out, void* stream) {
    if (!shape_ok(N, K, group)) return W4A8_ERR_SHAPE;
    if (!qw || !scales || !zeros || !packed_out) return W4A8_ERR_NULL;
    if (!aligned(qw, 8) || !aligned(scales, 2) || !aligned(packed_out, 128)) return W4A8_ERR_ALIGN;
    w4a8_status a = arch_check();
    if (a != W4A8_OK) return a;
    return launch_pack_weights(qw, scales, zeros, N, K, packed_out, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? W4A8_OK : W4A8_ERR_CUDA;
}

w4a8_status w4a8_unpack_weights(const void* packed, int N, int K, int group,
                                uint8_t* qw_out, uint16_t* scales_out, uint8_t* zeros_out, void* stream) {
    if (!shape_ok(N, K, group)) return W4A8_ERR_SHAPE;
    if (!packed) return W4A8_ERR_NULL;
    if (!aligned(packed, 128) || (qw_out && !aligned(qw_out, 8)) || (scales_out && !aligned(scales_out, 2)))
        return W4A8_ERR_ALIGN;
    w4a8_status a = arch_check();
    if (a != W4A8_OK) return a;
    return launch_unpack_weights(packed, N, K, qw_out, scales_out, zeros_out, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? W4A8_OK : W4A8_ERR_CUDA;
}

w4a8_status w4a8_quantize_act(const void* x_bf16, int M, int K, int group,
                              int8_t* qa, uint16_t* sa, int32_t* asum, void* stream) {
    if (group != GROUP || K <= 0 || K % GROUP != 0 || M < 0) return W4A8_ERR_SHAPE;
    if (M == 0) return W4A8_OK;
    if (!x_bf16 || !qa || !sa || !asum) return W4A8_ERR_NULL;
    if (!aligned(x_bf16, 16) || !aligned(qa, 16) || !aligned(sa, 2) || !aligned(asum, 4)) return W4A8_ERR_ALIGN;
    w4a8_status a = arch_check();
    if (a != W4A8_OK) return a;
    return launch_quantize_act(x_bf16, M, K, qa, sa, asum, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? W4A8_OK : W4A8_ERR_CUDA;
}

static w4a8_status gemm_impl(w4a8_path path,
                             const int8_t* qa, const uint16_t* sa, const int32_t* asum,
                             const void* packed_w, void* y_bf16, const void* residual,
                             int M, int N, int K, int group,
                             void* workspace, size_t workspace_bytes,
                             int32_t* debug_partials, void* stream) {
    if (!shape_ok(N, K, group) || M < 0) return W4A8_ERR_SHAPE;
    if (path != W4A8_PATH_AUTO && path != W4A8_PATH_SPLITK && path != W4A8_PATH_TCGEN05 &&
        path != W4A8_PATH_SPLITK_WORKSPACE && path != W4A8_PATH_STRIP)
        return W4A8_ERR_SHAPE;
    if ((path == W4A8_PATH_SPLITK || path == W4A8_PATH_SPLITK_WORKSPACE) && M > SPLITK_MAX_M) return W4A8_ERR_SHAPE;
    if (path == W4A8_PATH_STRIP && M > 0 && !strip_supported(M, N, K)) return W4A8_ERR_SHAPE;
    if (M == 0) return W4A8_OK;
    if (!qa || !sa || !asum || !packed_w || !y_bf16 || !workspace) return W4A8_ERR_NULL;
    // the kernels store y in 8- and 16-byte pieces and through a TMA map (16-byte base); only the
    // workspace variant of the split-K kernel stores element by element
    if (!aligned(qa, 16) || !aligned(sa, 2) || !aligned(asum, 4) || !aligned(packed_w, 128) ||
        !aligned(y_bf16, path == W4A8_PATH_SPLITK_WORKSPACE ? 2 : 16) || !aligned(workspace, 256) ||
        (debug_partials && !aligned(debug_partials, 4)) || (residual && !aligned(residual, 16)))
        return W4A8_ERR_ALIGN;
    if (residual && path == W4A8_PATH_SPLITK_WORKSPACE) return W4A8_ERR_SHAPE;     // that variant has no residual epilogue
    if (workspace_bytes < w4a8_workspace_bytes(M, N, K, group)) return W4A8_ERR_WORKSPACE;
    w4a8_status a = arch_check();
    if (a != W4A8_OK) return a;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    if (path == W4A8_PATH_SPLITK_WORKSPACE)
        e = launch_gemm_splitk(qa, sa, asum, packed_w, y_bf16, M, N, K, workspace,
                               reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + WS_SHARED_OFF), debug_partials, st);
    else if (path == W4A8_PATH_STRIP || (path == W4A8_PATH_AUTO && auto_takes_strip(M, N, K)))
        e = launch_gemm_strip(qa, sa, asum, packed_w, y_bf16, residual, M, N, K, workspace, debug_partials, st);
    else if (path == W4A8_PATH_SPLITK || (path == W4A8_PATH_AUTO && !small_m_prefers_tcgen05(M, N, K, device_sm_count())))
        e = launch_gemm_cluster(qa, sa, asum, packed_w, y_bf16, residual, M, N, K, workspace, debug_partials, st);
    else
        e = launch_gemm_tcgen05(qa, sa, packed_w, y_bf16, residual, M, N, K, workspace, debug_partials, st);
    return e == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
}

w4a8_status w4a8_gemm_path(w4a8_path path,
                           const int8_t* qa, const uint16_t* sa, const int32_t* asum,
                           const void* packed_w, void* y_bf16,
                           int M, int N, int K, int group,
                           void* workspace, size_t workspace_bytes,
                           int32_t* debug_partials, void* stream) {
    return gemm_impl(path, qa, sa, asum, packed_w, y_bf16, nullptr, M, N, K, group, workspace, workspace_bytes, debug_partials, stream);
}

w4a8_status w4a8_gemm_residual(w4a8_path path, const int8_t* qa, const uint16_t* sa, const int32_t* asum, const void* packed_w,
                               const void* residual_bf16, void* y_bf16, int M, int N, int K, int group,
                               void* workspace, size_t workspace_bytes, void* stream) {
    if (M > 0 && !residual_bf16) return W4A8_ERR_NULL;
    return gemm_impl(path, qa, sa, asum, packed_w, y_bf16, residual_bf16, M, N, K, group, workspace, workspace_bytes, nullptr, stream);
}

w4a8_status w4a8_silu_mul_quantize(const void* y_gate_up_bf16, int M, int I, int group, void* h_bf16,
                                   int8_t* qa_h, uint16_t* sa_h, int32_t* asum_h, void* stream) {
    if (group != GROUP || I <= 0 || I % GROUP != 0 || M < 0) return W4A8_ERR_SHAPE;
    if (M == 0) return W4A8_OK;
    if (!y_gate_up_bf16 || !qa_h || !sa_h || !asum_h) return W4A8_ERR_NULL;
    if (!aligned(y_gate_up_bf16, 16) || !aligned(qa_h, 16) || !aligned(sa_h, 2) || !aligned(asum_h, 4) ||
        (h_bf16 && !aligned(h_bf16, 16)))
        return W4A8_ERR_ALIGN;
    w4a8_status a = arch_check();
    if (a != W4A8_OK) return a;
    return launch_silu_mul_quantize(y_gate_up_bf16, M, I, h_bf16, qa_h, sa_h, asum_h, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? W4A8_OK : W4A8_ERR_CUDA;
}

int w4a8_gate_up_form(int M, int N, int K, int group) {
    if (!shape_ok(N, K, group) || M < 1 || (N / 2) % GROUP != 0) return 0;
    return auto_takes_strip(M, N, K) ? W4A8_GATE_UP_EPILOGUE : W4A8_GATE_UP_SEPARATE;
}

w4a8_status w4a8_gate_up_silu_quantize(int form, const int8_t* qa, const uint16_t* sa, const int32_t* asum,
                                       const void* packed_gate_up, int M, int N, int K, int group, void* h_bf16,
                                       int8_t* qa_h, uint16_t* sa_h, int32_t* asum_h, void* y_scratch_bf16,
                                       void* workspace, size_t workspace_bytes, void* stream) {
    if (!shape_ok(N, K, group) || M < 0 || (N / 2) % GROUP != 0) return W4A8_ERR_SHAPE;
    if (form != W4A8_GATE_UP_AUTO && form != W4A8_GATE_UP_ONE_KERNEL && form != W4A8_GATE_UP_EPILOGUE &&
        form != W4A8_GATE_UP_SEPARATE)
        return W4A8_ERR_SHAPE;
    if (M == 0) return W4A8_OK;
    if (form == W4A8_GATE_UP_AUTO) form = w4a8_gate_up_form(M, N, K, group);
    // the two forms that live in the strip kernel's epilogue exist where that kernel does
    if (form != W4A8_GATE_UP_SEPARATE && !strip_supported(M, N, K)) return W4A8_ERR_SHAPE;
    if (!qa || !sa || !asum || !packed_gate_up || !h_bf16 || !qa_h || !sa_h || !asum_h || !workspace) return W4A8_ERR_NULL;
    if (form == W4A8_GATE_UP_SEPARATE && !y_scratch_bf16) return W4A8_ERR_NULL;
    if (!aligned(qa, 16) || !aligned(sa, 2) || !aligned(asum, 4) || !aligned(packed_gate_up, 128) || !aligned(h_bf16, 16) ||
        !aligned(qa_h, 16) || !aligned(sa_h, 2) || !aligned(asum_h, 4) || !aligned(workspace, 256) ||
        (y_scratch_bf16 && !aligned(y_scratch_bf16, 16)))
        return W4A8_ERR_ALIGN;
    if (workspace_bytes < w4a8_workspace_bytes(M, N, K, group)) return W4A8_ERR_WORKSPACE;
    w4a8_status a = arch_check();
    if (a != W4A8_OK) return a;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (form != W4A8_GATE_UP_SEPARATE)
        return launch_gemm_strip_gate_up(qa, sa, asum, packed_gate_up, M, N, K, h_bf16, qa_h, sa_h, asum_h,
                                         form == W4A8_GATE_UP_ONE_KERNEL, workspace, st) == cudaSuccess
                   ? W4A8_OK : W4A8_ERR_CUDA;
    w4a8_status g = w4a8_gemm_path(W4A8_PATH_AUTO, qa, sa, asum, packed_gate_up, y_scratch_bf16, M, N, K, group, workspace,
                                   workspace_bytes, nullptr, stream);
    if (g != W4A8_OK) return g;
    return launch_silu_mul_quantize(y_scratch_bf16, M, N / 2, h_bf16, qa_h, sa_h, asum_h, st) == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
}

w4a8_status w4a8_rope_shifted_keys(const void* k_pre_bf16, const int32_t* pos, int delta, int T, int H, int D, double base,
                                   void* k_rot_bf16, void* stream) {
    if (T < 0 || H <= 0 || D <= 0 || D % 4 != 0 || !(base > 1.0)) return W4A8_ERR_SHAPE;
    if (T == 0) return W4A8_OK;
    if (!k_pre_bf16 || !pos || !k_rot_bf16) return W4A8_ERR_NULL;
    if (!aligned(k_pre_bf16, 4) || !aligned(k_rot_bf16, 4) || !aligned(pos, 4)) return W4A8_ERR_ALIGN;
    w4a8_status a = arch_check();
    if (a != W4A8_OK) return a;
    return launch_rope_shifted_keys(k_pre_bf16, pos, delta, T, H, D, base, k_rot_bf16, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? W4A8_OK : W4A8_ERR_CUDA;
}

w4a8_status w4a8_streaming_mask(int views, int frames, int tokens_per_frame, uint8_t* mask, void* stream) {
    if (views <= 0 || frames <= 0 || tokens_per_frame <= 0) return W4A8_ERR_SHAPE;
    if (!mask) return W4A8_ERR_NULL;
    w4a8_status a = arch_check();
    if (a != W4A8_OK) return a;
    return launch_streaming_mask(views, frames, tokens_per_frame, mask, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? W4A8_OK : W4A8_ERR_CUDA;
}

w4a8_status w4a8_a16_gemm(const void* x_bf16, const void* packed_w, void* y_bf16, int M, int N, int K, int group,
                          void* workspace, size_t workspace_bytes, void* stream) {
    if (!shape_ok(N, K, group) || M < 0) return W4A8_ERR_SHAPE;
    if (M > 0 && !a16_supported(M, N, K)) return W4A8_ERR_SHAPE;
    if (M == 0) return W4A8_OK;
    if (!x_bf16 || !packed_w || !y_bf16 || !workspace) return W4A8_ERR_NULL;
    if (!aligned(x_bf16, 16) || !aligned(packed_w, 128) || !aligned(y_bf16, 16) || !aligned(workspace, 256)) return W4A8_ERR_ALIGN;
    if (workspace_bytes < w4a8_workspace_bytes(M, N, K, group)) return W4A8_ERR_WORKSPACE;
    w4a8_status a = arch_check();
    if (a != W4A8_OK) return a;
    return launch_gemm_strip_a16(x_bf16, packed_w, y_bf16, M, N, K, workspace, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? W4A8_OK : W4A8_ERR_CUDA;
}

w4a8_status w4a8_dequantize_weights(const void* packed_w, int N, int K, int group, void* w_bf16, void* stream) {
    if (!shape_ok(N, K, group)) return W4A8_ERR_SHAPE;
    if (!packed_w || !w_bf16) return W4A8_ERR_NULL;
    if (!aligned(packed_w, 128) || !aligned(w_bf16, 16)) return W4A8_ERR_ALIGN;
    w4a8_status a = arch_check();
    if (a != W4A8_OK) return a;
    return launch_dequantize_weights(packed_w, N, K, w_bf16, static_cast<cudaStream_t>(stream)) == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
}

w4a8_status w4a8_gemm_per_channel(const int8_t* qa, const uint16_t* sa, const void* packed_w, void* y_bf16,
                                  int M, int N, int K, int group, void* workspace, size_t workspace_bytes,
                                  int32_t* debug_sums, void* stream) {
    if (!shape_ok(N, K, group) || M < 0 || K > (1 << 19)) return W4A8_ERR_SHAPE;    // int32 sums: 15 * 127 * K < 2^31
    if (M == 0) return W4A8_OK;
    if (!qa || !sa || !packed_w || !y_bf16 || !workspace) return W4A8_ERR_NULL;
    if (!aligned(qa, 16) || !aligned(sa, 2) || !aligned(packed_w, 128) || !aligned(y_bf16, 16) ||
        !aligned(workspace, 256) || (debug_sums && !aligned(debug_sums, 4)))
        return W4A8_ERR_ALIGN;
    if (workspace_bytes < w4a8_workspace_bytes(M, N, K, group)) return W4A8_ERR_WORKSPACE;
    w4a8_status a = arch_check();
    if (a != W4A8_OK) return a;
    return launch_gemm_tcgen05_per_channel(qa, sa, packed_w, y_bf16, M, N, K, workspace, debug_sums,
                                           static_cast<cudaStream_t>(stream)) == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
}

w4a8_status w4a8_plan(int M, int N, int K, int group, w4a8_plan_info* out) {
    if (!shape_ok(N, K, group) || M <= 0) return W4A8_ERR_SHAPE;
    const int sms = device_sm_count(), tiles = N / TILE_N;
    w4a8_plan_info p;
    if (auto_takes_strip(M, N, K)) {
        int rows = 0, ctas = 0;
        strip_plan(M, N, K, &rows, &ctas);
        p.family = W4A8_PATH_STRIP;
        p.tile_m = M <= 8 ? 8 : 16;
        p.k_slices = 1;
        p.ctas = ctas;
        p.strip_rows = rows;
        p.balanced = (N / rows) % ctas != 0;
    } else if (!small_m_prefers_tcgen05(M, N, K, sms)) {
        p.strip_rows = 0;
        p.family = W4A8_PATH_SPLITK;
        p.tile_m = M <= 8 ? 8 : (M <= 16 ? 16 : (M <= 32 ? 32 : 64));
        p.k_slices = cluster_num_slices(M, N, K);
        p.ctas = tiles * p.k_slices;
        p.balanced = 0;
    } else {
        p.family = W4A8_PATH_TCGEN05;
        p.strip_rows = 0;
        tcgen05_plan(M, N, K, sms, &p.tile_m, &p.k_slices, 4, &p.balanced);       // the launcher's own call
        const int all = ((M + p.tile_m - 1) / p.tile_m) * tiles;
        p.ctas = p.k_slices > 1 ? all * p.k_slices : (all < sms ? all : sms);
    }
    if (out) *out = p;
    return W4A8_OK;
}

w4a8_status w4a8_gemm(const int8_t* qa, const uint16_t* sa, const int32_t* asum,
                      const void* packed_w, void* y_bf16,
                      int M, int N, int K, int group,
                      void* workspace, size_t workspace_bytes,
                      int32_t* debug_partials, void* stream) {
    return w4a8_gemm_path(W4A8_PATH_AUTO, qa, sa, asum, packed_w, y_bf16, M, N, K, group,
                          workspace, workspace_bytes, debug_partials, stream);
}

w4a8_status w4a8_linear(const void* x_bf16, const void* packed_w, void* y_bf16,
                        int M, int N, int K, int group,
                        int8_t* qa, uint16_t* sa, int32_t* asum,
                        void* workspace, size_t workspace_bytes, void* stream) {
    if (!shape_ok(N, K, group) || M < 0) return W4A8_ERR_SHAPE;
    if (M == 0) return W4A8_OK;
    // everything the second call would refuse is refused before the first one is enqueued
    if (!x_bf16 || !qa || !sa || !asum || !packed_w || !y_bf16 || !workspace) return W4A8_ERR_NULL;
    if (!aligned(packed_w, 128) || !aligned(y_bf16, 16) || !aligned(workspace, 256)) return W4A8_ERR_ALIGN;
    if (workspace_bytes < w4a8_workspace_bytes(M, N, K, group)) return W4A8_ERR_WORKSPACE;
    w4a8_status s = w4a8_quantize_act(x_bf16, M, K, group, qa, sa, asum, stream);
    if (s != W4A8_OK) return s;
    return w4a8_gemm(qa, sa, asum, packed_w, y_bf16, M, N, K, group, workspace, workspace_bytes, nullptr, stream);
}

w4a8_status w4a8_linear_host(const void* x_host_bf16, void* y_host_bf16,
                             int M, int N, int K, int group, const void* packed_w,
                             void* x_dev, int8_t* qa, uint16_t* sa, int32_t* asum, void* y_dev,
                             void* workspace, size_t workspace_bytes, void* stream) {
    if (!shape_ok(N, K, group) || M < 0) return W4A8_ERR_SHAPE;
    if (M == 0) return W4A8_OK;
    if (!x_host_bf16 || !y_host_bf16 || !x_dev || !y_dev || !qa || !sa || !asum || !packed_w || !workspace)
        return W4A8_ERR_NULL;
    if (!aligned(x_dev, 16) || !aligned(qa, 16) || !aligned(sa, 2) || !aligned(asum, 4) || !aligned(packed_w, 128) ||
        !aligned(y_dev, 16) || !aligned(workspace, 256))
        return W4A8_ERR_ALIGN;
    if (workspace_bytes < w4a8_workspace_bytes(M, N, K, group)) return W4A8_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(x_dev, x_host_bf16, (size_t)M * K * 2, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return W4A8_ERR_CUDA;
    w4a8_status s = w4a8_linear(x_dev, packed_w, y_dev, M, N, K, group, qa, sa, asum, workspace, workspace_bytes, stream);
    if (s != W4A8_OK) return s;
    if (cudaMemcpyAsync(y_host_bf16, y_dev, (size_t)M * N * 2, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return W4A8_ERR_CUDA;
    return W4A8_OK;
}

w4a8_status w4a8_check_status(void* workspace, void* stream) {
    if (!workspace) return W4A8_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t word = 0;
    if (cudaMemcpyAsync(&word, static_cast<uint8_t*>(workspace) + WS_STATUS_OFF, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return W4A8_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return W4A8_ERR_CUDA;
    if (word == 0) return W4A8_OK;
    if (cudaMemsetAsync(static_cast<uint8_t*>(workspace) + WS_STATUS_OFF, 0, 4, st) != cudaSuccess) return W4A8_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return W4A8_ERR_CUDA;
    return word == W4A8_ERR_TIMEOUT ? W4A8_ERR_TIMEOUT : W4A8_ERR_CUDA;
}

w4a8_status w4a8_selftest_wait_timeout(const int8_t* qa, const uint16_t* sa, const int32_t* asum, const void* packed_w,
                                       void* y_bf16, int M, int N, int K, int group, void* workspace,
                                       size_t workspace_bytes, void* stream) {
    if (!shape_ok(N, K, group) || M <= 0 || M > SPLITK_MAX_M) return W4A8_ERR_SHAPE;
    if (!qa || !sa || !asum || !packed_w || !y_bf16 || !workspace) return W4A8_ERR_NULL;
    if (!aligned(qa, 16) || !aligned(sa, 2) || !aligned(asum, 4) || !aligned(packed_w, 128) || !aligned(y_bf16, 2) ||
        !aligned(workspace, 256))
        return W4A8_ERR_ALIGN;
    if (workspace_bytes < w4a8_workspace_bytes(M, N, K, group)) return W4A8_ERR_WORKSPACE;
    w4a8_status a = arch_check();
    if (a != W4A8_OK) return a;
    return launch_gemm_splitk(qa, sa, asum, packed_w, y_bf16, M, N, K, workspace,
                              reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + WS_SHARED_OFF), withhold_marker(),
                              static_cast<cudaStream_t>(stream)) == cudaSuccess ? W4A8_OK : W4A8_ERR_CUDA;
}

w4a8_status w4a8_static_scratch_status(void* stream) {
    void* scratch = static_scratch_address();        // looks the array's device address up; allocates nothing
    if (!scratch) return W4A8_ERR_CUDA;
    return w4a8_check_status(scratch, stream);
}

}  // extern "C"
