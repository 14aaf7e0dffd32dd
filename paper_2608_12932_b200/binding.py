"""ctypes binding of libw4a8.so: same names as the C ABI, argument marshalling only.

PyTorch is used for device memory and streams; every step of the path runs in the
library's CUDA kernels.  There is no CPU or eager fallback: if the shared library is
missing the first call raises.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libw4a8.so")

GROUP = 128
OK, ERR_NULL, ERR_SHAPE, ERR_ALIGN, ERR_WORKSPACE, ERR_ARCH, ERR_CUDA, ERR_TIMEOUT = range(8)
PATH_AUTO, PATH_SPLITK, PATH_TCGEN05, PATH_SPLITK_WORKSPACE, PATH_STRIP = 0, 1, 2, 3, 4
WORKSPACE_HEADER_BYTES = 4096
WORKSPACE_ZEROED_BYTES = 4096 + 192 * 16384

EXPORTS = ("w4a8_status_string", "w4a8_packed_bytes", "w4a8_workspace_bytes", "w4a8_workspace_init",
           "w4a8_pack_weights", "w4a8_unpack_weights", "w4a8_quantize_act", "w4a8_gemm", "w4a8_gemm_path",
           "w4a8_linear", "w4a8_linear_host", "w4a8_gemm_static_scratch", "w4a8_check_status", "w4a8_plan",
           "w4a8_gemm_per_channel", "w4a8_static_scratch_status", "w4a8_selftest_wait_timeout",
           "w4a8_silu_mul_quantize", "w4a8_gate_up_form", "w4a8_gate_up_silu_quantize", "w4a8_a16_gemm",
           "w4a8_dequantize_weights", "w4a8_gemm_residual", "w4a8_rope_shifted_keys",
           "w4a8_streaming_mask")

_lib = None


class W4A8Error(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


def lib():
    """The loaded shared library; raises if it has not been built (python -m paper_2608_12932_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2608_12932_b200.build`; "
                               "there is no fallback path")
        L = ctypes.CDLL(LIB_PATH)
        vp, ci, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        L.w4a8_status_string.restype = ctypes.c_char_p
        L.w4a8_status_string.argtypes = [ci]
        L.w4a8_packed_bytes.restype = sz
        L.w4a8_packed_bytes.argtypes = [ci, ci, ci]
        L.w4a8_workspace_bytes.restype = sz
        L.w4a8_workspace_bytes.argtypes = [ci, ci, ci, ci]
        L.w4a8_workspace_init.restype = ci
        L.w4a8_workspace_init.argtypes = [vp, sz, vp]
        L.w4a8_pack_weights.restype = ci
        L.w4a8_pack_weights.argtypes = [vp, vp, vp, ci, ci, ci, vp, vp]
        L.w4a8_unpack_weights.restype = ci
        L.w4a8_unpack_weights.argtypes = [vp, ci, ci, ci, vp, vp, vp, vp]
        L.w4a8_quantize_act.restype = ci
        L.w4a8_quantize_act.argtypes = [vp, ci, ci, ci, vp, vp, vp, vp]
        L.w4a8_gemm.restype = ci
        L.w4a8_gemm.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, vp, sz, vp, vp]
        L.w4a8_gemm_path.restype = ci
        L.w4a8_gemm_path.argtypes = [ci, vp, vp, vp, vp, vp, ci, ci, ci, ci, vp, sz, vp, vp]
        L.w4a8_gemm_per_channel.restype = ci
        L.w4a8_gemm_per_channel.argtypes = [vp, vp, vp, vp, ci, ci, ci, ci, vp, sz, vp, vp]
        L.w4a8_plan.restype = ci
        L.w4a8_plan.argtypes = [ci, ci, ci, ci, vp]
        L.w4a8_silu_mul_quantize.restype = ci
        L.w4a8_silu_mul_quantize.argtypes = [vp, ci, ci, ci, vp, vp, vp, vp, vp]
        L.w4a8_rope_shifted_keys.restype = ci
        L.w4a8_rope_shifted_keys.argtypes = [vp, vp, ci, ci, ci, ci, ctypes.c_double, vp, vp]
        L.w4a8_streaming_mask.restype = ci
        L.w4a8_streaming_mask.argtypes = [ci, ci, ci, vp, vp]
        L.w4a8_gemm_residual.restype = ci
        L.w4a8_gemm_residual.argtypes = [ci, vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, vp, sz, vp]
        L.w4a8_a16_gemm.restype = ci
        L.w4a8_a16_gemm.argtypes = [vp, vp, vp, ci, ci, ci, ci, vp, sz, vp]
        L.w4a8_dequantize_weights.restype = ci
        L.w4a8_dequantize_weights.argtypes = [vp, ci, ci, ci, vp, vp]
        L.w4a8_gate_up_form.restype = ci
        L.w4a8_gate_up_form.argtypes = [ci, ci, ci, ci]
        L.w4a8_gate_up_silu_quantize.restype = ci
        L.w4a8_gate_up_silu_quantize.argtypes = [ci, vp, vp, vp, vp, ci, ci, ci, ci, vp, vp, vp, vp, vp, vp, sz, vp]
        L.w4a8_linear.restype = ci
        L.w4a8_linear.argtypes = [vp, vp, vp, ci, ci, ci, ci, vp, vp, vp, vp, sz, vp]
        L.w4a8_linear_host.restype = ci
        L.w4a8_linear_host.argtypes = [vp, vp, ci, ci, ci, ci, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.w4a8_gemm_static_scratch.restype = ci
        L.w4a8_gemm_static_scratch.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, vp]
        L.w4a8_check_status.restype = ci
        L.w4a8_check_status.argtypes = [vp, vp]
        L.w4a8_selftest_wait_timeout.restype = ci
        L.w4a8_selftest_wait_timeout.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, vp, sz, vp]
        L.w4a8_static_scratch_status.restype = ci
        L.w4a8_static_scratch_status.argtypes = [vp]
        _lib = L
    return _lib


def status_string(code):
    return lib().w4a8_status_string(int(code)).decode()


def _check(code, where):
    if code != OK:
        raise W4A8Error(code, where)


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _ptr(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else None


def _dev(t, dtype, name):
    if not (t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: need a contiguous CUDA tensor of {dtype}, got {t.dtype} on {t.device}")
    return t


def w4a8_packed_bytes(N, K, group=GROUP):
    return int(lib().w4a8_packed_bytes(N, K, group))


def w4a8_workspace_bytes(M_max, N, K, group=GROUP):
    return int(lib().w4a8_workspace_bytes(M_max, N, K, group))


def new_workspace(M_max, N, K, group=GROUP, device="cuda", stream=None):
    """Allocates (through torch) and initialises a workspace for w4a8_gemm on this layer shape."""
    nbytes = w4a8_workspace_bytes(M_max, N, K, group)
    if nbytes == 0:
        raise W4A8Error(ERR_SHAPE, "w4a8_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    _check(lib().w4a8_workspace_init(_ptr(ws), nbytes, _stream(stream)), "w4a8_workspace_init")
    return ws


def w4a8_pack_weights(qw, scales, zeros, group=GROUP, out=None, stream=None):
    """qw uint8 [N,K] codes, scales fp16 [G,N], zeros uint8 [G,N] -> packed uint8 blob (device)."""
    _dev(qw, torch.uint8, "qw"), _dev(scales, torch.float16, "scales"), _dev(zeros, torch.uint8, "zeros")
    N, K = qw.shape
    nbytes = w4a8_packed_bytes(N, K, group)
    if nbytes == 0 or tuple(scales.shape) != (K // group, N) or tuple(zeros.shape) != (K // group, N):
        raise W4A8Error(ERR_SHAPE, "w4a8_pack_weights")
    if out is None:
        out = torch.empty(nbytes, dtype=torch.uint8, device=qw.device)
    _check(lib().w4a8_pack_weights(_ptr(qw), _ptr(scales), _ptr(zeros), N, K, group, _ptr(out), _stream(stream)),
           "w4a8_pack_weights")
    return out


def w4a8_unpack_weights(packed, N, K, group=GROUP, stream=None):
    _dev(packed, torch.uint8, "packed")
    G = K // group
    qw = torch.empty((N, K), dtype=torch.uint8, device=packed.device)
    scales = torch.empty((G, N), dtype=torch.float16, device=packed.device)
    zeros = torch.empty((G, N), dtype=torch.uint8, device=packed.device)
    _check(lib().w4a8_unpack_weights(_ptr(packed), N, K, group, _ptr(qw), _ptr(scales), _ptr(zeros), _stream(stream)),
           "w4a8_unpack_weights")
    return qw, scales, zeros


def w4a8_quantize_act(x, group=GROUP, out=None, stream=None):
    """x bf16 [M,K] -> (qa int8 [M,K], sa fp16 [M], asum int32 [M,K/group])."""
    _dev(x, torch.bfloat16, "x")
    M, K = x.shape
    if out is None:
        qa = torch.empty((M, K), dtype=torch.int8, device=x.device)
        sa = torch.empty((M,), dtype=torch.float16, device=x.device)
        asum = torch.empty((M, max(K // group, 0)), dtype=torch.int32, device=x.device)
    else:
        qa, sa, asum = out
    _check(lib().w4a8_quantize_act(_ptr(x), M, K, group, _ptr(qa), _ptr(sa), _ptr(asum), _stream(stream)),
           "w4a8_quantize_act")
    return qa, sa, asum


def w4a8_gemm(qa, sa, asum, packed_w, N, workspace, group=GROUP, out=None, debug_partials=None,
              path=PATH_AUTO, stream=None):
    """y bf16 [M,N] = the W4A8 linear of quantised activations against a packed layer."""
    _dev(qa, torch.int8, "qa"), _dev(sa, torch.float16, "sa"), _dev(asum, torch.int32, "asum")
    _dev(packed_w, torch.uint8, "packed_w"), _dev(workspace, torch.uint8, "workspace")
    M, K = qa.shape
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=qa.device)
    else:
        _dev(out, torch.bfloat16, "out")
    if debug_partials is not None:
        _dev(debug_partials, torch.int32, "debug_partials")
    if path == PATH_AUTO:
        code = lib().w4a8_gemm(_ptr(qa), _ptr(sa), _ptr(asum), _ptr(packed_w), _ptr(out), M, N, K, group,
                               _ptr(workspace), workspace.numel(), _ptr(debug_partials), _stream(stream))
    else:
        code = lib().w4a8_gemm_path(path, _ptr(qa), _ptr(sa), _ptr(asum), _ptr(packed_w), _ptr(out), M, N, K, group,
                                    _ptr(workspace), workspace.numel(), _ptr(debug_partials), _stream(stream))
    _check(code, "w4a8_gemm")
    return out


def w4a8_gemm_per_channel(qa, sa, packed_w, N, workspace, group=GROUP, out=None, debug_sums=None, stream=None):
    """w4a8_gemm for a packed layer whose scales are equal in every group of a channel: one drain per tile."""
    _dev(qa, torch.int8, "qa"), _dev(sa, torch.float16, "sa")
    _dev(packed_w, torch.uint8, "packed_w"), _dev(workspace, torch.uint8, "workspace")
    M, K = qa.shape
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=qa.device)
    else:
        _dev(out, torch.bfloat16, "out")
    if debug_sums is not None:
        _dev(debug_sums, torch.int32, "debug_sums")
    _check(lib().w4a8_gemm_per_channel(_ptr(qa), _ptr(sa), _ptr(packed_w), _ptr(out), M, N, K, group,
                                       _ptr(workspace), workspace.numel(), _ptr(debug_sums), _stream(stream)),
           "w4a8_gemm_per_channel")
    return out


def gate_up_row_order(I):
    """Row order of the fused gate+up layer: entry n is the row of the concatenation [gate rows; up rows] (2 I rows)
    that becomes output channel n - runs of eight gate channels alternating with the eight up channels of the same
    indices (see w4a8_gate_up_silu_quantize in the header).  Index arithmetic only."""
    import numpy as np
    n = np.arange(2 * I)
    b, i = n // 16, n % 16
    return np.where(i < 8, 8 * b + i, I + 8 * b + i - 8)


def _h_outputs(M, I, group, device, out):
    if out is not None:
        return out
    return (torch.empty((M, I), dtype=torch.bfloat16, device=device), torch.empty((M, I), dtype=torch.int8, device=device),
            torch.empty((M,), dtype=torch.float16, device=device), torch.empty((M, I // group), dtype=torch.int32, device=device))


def w4a8_silu_mul_quantize(y_gate_up, group=GROUP, out=None, stream=None):
    """y bf16 [M, 2 I] of a fused gate+up layer -> (h bf16 [M,I], qa_h int8 [M,I], sa_h fp16 [M], asum_h int32 [M,I/group])."""
    _dev(y_gate_up, torch.bfloat16, "y_gate_up")
    M, N = y_gate_up.shape
    I = N // 2
    h, qa_h, sa_h, asum_h = _h_outputs(M, I, group, y_gate_up.device, out)
    _check(lib().w4a8_silu_mul_quantize(_ptr(y_gate_up), M, I, group, _ptr(h), _ptr(qa_h), _ptr(sa_h), _ptr(asum_h),
                                        _stream(stream)), "w4a8_silu_mul_quantize")
    return h, qa_h, sa_h, asum_h


GATE_UP_AUTO, GATE_UP_ONE_KERNEL, GATE_UP_EPILOGUE, GATE_UP_SEPARATE = 0, 1, 2, 3


def w4a8_gate_up_form(M, N, K, group=GROUP):
    """The form GATE_UP_AUTO takes for this size (0 for an unsupported shape)."""
    return int(lib().w4a8_gate_up_form(M, N, K, group))


def w4a8_gate_up_silu_quantize(qa, sa, asum, packed_gate_up, N, workspace, group=GROUP, form=GATE_UP_AUTO, y_scratch=None,
                               out=None, stream=None):
    """Fused gate+up projection, SiLU(gate) * up and the down projection's activation quantisation; see the header for
    the three forms.  Returns (h, qa_h, sa_h, asum_h)."""
    _dev(qa, torch.int8, "qa"), _dev(sa, torch.float16, "sa"), _dev(asum, torch.int32, "asum")
    _dev(packed_gate_up, torch.uint8, "packed_gate_up"), _dev(workspace, torch.uint8, "workspace")
    M, K = qa.shape
    I = N // 2
    h, qa_h, sa_h, asum_h = _h_outputs(M, I, group, qa.device, out)
    separate = form == GATE_UP_SEPARATE or (form == GATE_UP_AUTO and w4a8_gate_up_form(M, N, K, group) == GATE_UP_SEPARATE)
    if y_scratch is None and M > 0 and separate:
        y_scratch = torch.empty((M, N), dtype=torch.bfloat16, device=qa.device)
    _check(lib().w4a8_gate_up_silu_quantize(form, _ptr(qa), _ptr(sa), _ptr(asum), _ptr(packed_gate_up), M, N, K, group,
                                            _ptr(h), _ptr(qa_h), _ptr(sa_h), _ptr(asum_h), _ptr(y_scratch),
                                            _ptr(workspace), workspace.numel(), _stream(stream)),
           "w4a8_gate_up_silu_quantize")
    return h, qa_h, sa_h, asum_h


def w4a8_gemm_residual(qa, sa, asum, packed_w, residual, N, workspace, group=GROUP, out=None, path=PATH_AUTO, stream=None):
    """y = bf16(linear + residual), one rounding; out may be the residual tensor itself."""
    _dev(qa, torch.int8, "qa"), _dev(sa, torch.float16, "sa"), _dev(asum, torch.int32, "asum")
    _dev(packed_w, torch.uint8, "packed_w"), _dev(workspace, torch.uint8, "workspace"), _dev(residual, torch.bfloat16, "residual")
    M, K = qa.shape
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=qa.device)
    else:
        _dev(out, torch.bfloat16, "out")
    _check(lib().w4a8_gemm_residual(path, _ptr(qa), _ptr(sa), _ptr(asum), _ptr(packed_w), _ptr(residual), _ptr(out), M, N, K, group,
                                    _ptr(workspace), workspace.numel(), _stream(stream)), "w4a8_gemm_residual")
    return out


def w4a8_rope_shifted_keys(k_pre, pos, delta, base, out=None, stream=None):
    """k_pre bf16 [T,H,D], pos int32 [T] -> keys rotated at positions pos - delta (rotate-half rotary embedding)."""
    _dev(k_pre, torch.bfloat16, "k_pre"), _dev(pos, torch.int32, "pos")
    T, H, D = k_pre.shape
    if out is None:
        out = torch.empty_like(k_pre)
    _check(lib().w4a8_rope_shifted_keys(_ptr(k_pre), _ptr(pos), int(delta), T, H, D, float(base), _ptr(out), _stream(stream)),
           "w4a8_rope_shifted_keys")
    return out


def w4a8_streaming_mask(views, frames, tokens_per_frame, device="cuda", stream=None):
    """uint8 [views * n, views * frames * n]: which keys the newest frame's tokens may attend."""
    mask = torch.empty((views * tokens_per_frame, views * frames * tokens_per_frame), dtype=torch.uint8, device=device)
    _check(lib().w4a8_streaming_mask(views, frames, tokens_per_frame, _ptr(mask), _stream(stream)), "w4a8_streaming_mask")
    return mask


def w4a8_a16_gemm(x, packed_w, N, workspace, group=GROUP, out=None, stream=None):
    """W4A16: y bf16 [M,N] from bf16 activations x [M,K] (M <= 16) and a packed layer."""
    _dev(x, torch.bfloat16, "x"), _dev(packed_w, torch.uint8, "packed_w"), _dev(workspace, torch.uint8, "workspace")
    M, K = x.shape
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=x.device)
    else:
        _dev(out, torch.bfloat16, "out")
    _check(lib().w4a8_a16_gemm(_ptr(x), _ptr(packed_w), _ptr(out), M, N, K, group, _ptr(workspace), workspace.numel(),
                               _stream(stream)), "w4a8_a16_gemm")
    return out


def w4a8_dequantize_weights(packed_w, N, K, group=GROUP, out=None, stream=None):
    """Packed layer -> bf16 [N,K] weights s_w (q_w - z)."""
    _dev(packed_w, torch.uint8, "packed_w")
    if out is None:
        out = torch.empty((N, K), dtype=torch.bfloat16, device=packed_w.device)
    else:
        _dev(out, torch.bfloat16, "out")
    _check(lib().w4a8_dequantize_weights(_ptr(packed_w), N, K, group, _ptr(out), _stream(stream)), "w4a8_dequantize_weights")
    return out


class PlanInfo(ctypes.Structure):
    _fields_ = [("family", ctypes.c_int), ("tile_m", ctypes.c_int), ("k_slices", ctypes.c_int), ("ctas", ctypes.c_int),
                ("balanced", ctypes.c_int), ("strip_rows", ctypes.c_int)]


def w4a8_plan(M, N, K, group=GROUP):
    """What w4a8_gemm would launch for this size on the current device: dict(family, tile_m, k_slices, ctas)."""
    info = PlanInfo()
    _check(lib().w4a8_plan(M, N, K, group, ctypes.byref(info)), "w4a8_plan")
    return {"family": info.family, "tile_m": info.tile_m, "k_slices": info.k_slices, "ctas": info.ctas,
            "balanced": info.balanced, "strip_rows": info.strip_rows}


def w4a8_linear(x, packed_w, N, workspace, group=GROUP, out=None, scratch=None, stream=None):
    """y bf16 [M,N] = W4A8 linear of bf16 activations [M,K]: quantise, then multiply (two kernels on
    one stream).  `scratch` = (qa, sa, asum) buffers as w4a8_quantize_act returns them (allocated
    here when absent); they hold the quantised activations afterwards."""
    _dev(x, torch.bfloat16, "x"), _dev(packed_w, torch.uint8, "packed_w"), _dev(workspace, torch.uint8, "workspace")
    M, K = x.shape
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=x.device)
    else:
        _dev(out, torch.bfloat16, "out")
    if scratch is None:
        scratch = (torch.empty((M, K), dtype=torch.int8, device=x.device),
                   torch.empty((M,), dtype=torch.float16, device=x.device),
                   torch.empty((M, max(K // group, 1)), dtype=torch.int32, device=x.device))
    qa, sa, asum = scratch
    _dev(qa, torch.int8, "qa"), _dev(sa, torch.float16, "sa"), _dev(asum, torch.int32, "asum")
    _check(lib().w4a8_linear(_ptr(x), _ptr(packed_w), _ptr(out), M, N, K, group, _ptr(qa), _ptr(sa), _ptr(asum),
                             _ptr(workspace), workspace.numel(), _stream(stream)), "w4a8_linear")
    return out


STATIC_SCRATCH_BYTES = 4096 + 4 * 1024 * 1024


def w4a8_gemm_static_scratch(qa, sa, asum, packed_w, N, group=GROUP, out=None, stream=None):
    """w4a8_gemm without a workspace argument, for callers that cannot allocate device memory:
    the split-K scratch is a fixed array inside the library (M <= 64, scratch need at most
    STATIC_SCRATCH_BYTES).  `out` must be given by such callers; it is allocated here otherwise."""
    _dev(qa, torch.int8, "qa"), _dev(sa, torch.float16, "sa"), _dev(asum, torch.int32, "asum")
    _dev(packed_w, torch.uint8, "packed_w")
    M, K = qa.shape
    if out is None:
        out = torch.empty((M, N), dtype=torch.bfloat16, device=qa.device)
    else:
        _dev(out, torch.bfloat16, "out")
    _check(lib().w4a8_gemm_static_scratch(_ptr(qa), _ptr(sa), _ptr(asum), _ptr(packed_w), _ptr(out), M, N, K, group,
                                          _stream(stream)), "w4a8_gemm_static_scratch")
    return out


def w4a8_check_status(workspace, stream=None):
    _check(lib().w4a8_check_status(_ptr(workspace), _stream(stream)), "w4a8_check_status")


def w4a8_selftest_wait_timeout(qa, sa, asum, packed_w, N, workspace, group=GROUP, stream=None):
    """Runs the split-K kernel with one weight copy withheld per CTA and a 200 us wait limit (see w4a8.h); returns y (invalid)."""
    M, K = qa.shape
    out = torch.empty((M, N), dtype=torch.bfloat16, device=qa.device)
    _check(lib().w4a8_selftest_wait_timeout(_ptr(qa), _ptr(sa), _ptr(asum), _ptr(packed_w), _ptr(out), M, N, K, group,
                                            _ptr(workspace), workspace.numel(), _stream(stream)), "w4a8_selftest_wait_timeout")
    return out


def w4a8_static_scratch_status(stream=None):
    """The status word of w4a8_gemm_static_scratch's fixed array on the current device (synchronises the stream)."""
    _check(lib().w4a8_static_scratch_status(_stream(stream)), "w4a8_static_scratch_status")


class HostLinear:
    """Device staging buffers for w4a8_linear_host on one layer shape (allocated once, through torch)."""

    def __init__(self, M, N, K, packed_w, workspace, group=GROUP, device="cuda"):
        self.M, self.N, self.K, self.group = M, N, K, group
        self.packed_w, self.workspace = packed_w, workspace
        self.x_dev = torch.empty((M, K), dtype=torch.bfloat16, device=device)
        self.qa = torch.empty((M, K), dtype=torch.int8, device=device)
        self.sa = torch.empty((M,), dtype=torch.float16, device=device)
        self.asum = torch.empty((M, K // group), dtype=torch.int32, device=device)
        self.y_dev = torch.empty((M, N), dtype=torch.bfloat16, device=device)

    def __call__(self, x_host, y_host, stream=None):
        """x_host, y_host: CPU bf16 tensors (pinned for asynchronous copies); enqueues the whole path."""
        if x_host.is_cuda or y_host.is_cuda or x_host.dtype != torch.bfloat16 or y_host.dtype != torch.bfloat16:
            raise TypeError("w4a8_linear_host takes CPU bf16 tensors")
        if tuple(x_host.shape) != (self.M, self.K) or tuple(y_host.shape) != (self.M, self.N):
            raise W4A8Error(ERR_SHAPE, "w4a8_linear_host")
        _check(lib().w4a8_linear_host(_ptr(x_host), _ptr(y_host), self.M, self.N, self.K, self.group,
                                      _ptr(self.packed_w), _ptr(self.x_dev), _ptr(self.qa), _ptr(self.sa),
                                      _ptr(self.asum), _ptr(self.y_dev), _ptr(self.workspace),
                                      self.workspace.numel(), _stream(stream)), "w4a8_linear_host")
        return y_host
