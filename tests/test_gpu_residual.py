"""GPU parity of w4a8_gemm_residual (Sec. 3.5: the residual add merged into the projection's epilogue) on every kernel
family that has the epilogue: the sum is rounded once, judged against the fp64 sum with the projection's band plus
half a bf16 step of the sum; in place on the residual buffer; a zero residual reproduces w4a8_gemm bit for bit."""
import numpy as np
import pytest
import torch

from oracle import cfast
from oracle import w4a8_oracle as onp
from paper_2608_12932_b200 import binding as B
from paper_2608_12932_b200 import workload as wl
from tests.gpu_util import bits, t_u16

pytestmark = pytest.mark.gpu

# (M, K, N, path): strip kernel (every strip width, shared strips, two token blocks), cluster split-K kernel (one and
# several slices), tensor-core kernel (64 / 128 / 208-row tiles, ragged last tile, K split over a cluster, balanced walk)
CASES = [(1, 256, 256, B.PATH_AUTO), (8, 4096, 4096, B.PATH_AUTO), (8, 12288, 4096, B.PATH_AUTO), (5, 512, 24576, B.PATH_AUTO),
         (8, 1024, 6144, B.PATH_AUTO), (13, 4096, 6144, B.PATH_AUTO), (16, 4096, 4096, B.PATH_AUTO), (7, 384, 640, B.PATH_STRIP),
         (8, 4096, 4096, B.PATH_SPLITK), (24, 1024, 384, B.PATH_SPLITK), (40, 512, 1024, B.PATH_AUTO), (64, 12288, 4096, B.PATH_AUTO),
         (64, 512, 256, B.PATH_TCGEN05), (130, 384, 640, B.PATH_AUTO), (300, 256, 1024, B.PATH_AUTO), (1024, 512, 4096, B.PATH_AUTO),
         (1000, 1024, 20480, B.PATH_AUTO)]


@pytest.mark.parametrize("M,K,N,path", CASES)
def test_residual_epilogue(M, K, N, path):
    c = wl.make_layer(K, N, 7000 + M + N, M)
    rng = np.random.default_rng(M * 7 + N)
    r_bits = wl.f32_to_bf16_bits((rng.standard_normal((M, N)) * 4).astype(np.float32))
    r_bits[0, : N // 2] = 0
    packed = B.w4a8_pack_weights(torch.from_numpy(c["qw"]).cuda(), t_u16(c["sw"], torch.float16), torch.from_numpy(c["z"]).cuda())
    ws = B.new_workspace(M, N, K)
    qa, sa, asum = B.w4a8_quantize_act(t_u16(c["x"], torch.bfloat16))
    res = t_u16(r_bits, torch.bfloat16)
    y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.w4a8_gemm_residual(qa, sa, asum, packed, res, N, ws, out=y, path=path)
    B.w4a8_check_status(ws)
    lin = cfast.w4a8_linear(c["x"], c["qw"], c["sw"], c["z"], 128)["ref"]
    ref = lin + onp.bf16_bits_to_f64(r_bits)
    err = np.abs(onp.bf16_bits_to_f64(bits(y)) - ref)
    band = onp.residual_tolerance(lin, ref)
    assert np.all(err <= band), f"worst err/band {float((err / band).max()):.3f}"
    # one rounding: on average closer to the fp64 sum than rounding the projection first and adding then
    y_plain = B.w4a8_gemm(qa, sa, asum, packed, N, ws, path=path)
    two = (y_plain.float() + res.float()).to(torch.bfloat16)
    err_two = np.abs(onp.bf16_bits_to_f64(bits(two)) - ref)
    assert err.mean() <= err_two.mean() * 1.001
    # in place on the residual buffer
    B.w4a8_gemm_residual(qa, sa, asum, packed, res, N, ws, out=res, path=path)
    B.w4a8_check_status(ws)
    assert np.array_equal(bits(res), bits(y))
    # a zero residual: w4a8_gemm, bit for bit (where the sum is -0 the plain kernel may say -0 and this one +0)
    zero = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    y0 = B.w4a8_gemm_residual(qa, sa, asum, packed, zero, N, ws, path=path)
    B.w4a8_check_status(ws)
    a, b = bits(y0), bits(y_plain)
    assert np.array_equal(a & 0x7FFF, b & 0x7FFF) and np.all((a == b) | ((a & 0x7FFF) == 0))


def test_residual_argument_checks():
    M, K, N = 8, 256, 256
    c = wl.random_codes(np.random.default_rng(1), M, N, K)
    packed = B.w4a8_pack_weights(torch.from_numpy(c["qw"]).cuda(), t_u16(c["sw"], torch.float16), torch.from_numpy(c["z"]).cuda())
    ws = B.new_workspace(M, N, K)
    qa, sa, asum = B.w4a8_quantize_act(t_u16(c["x"], torch.bfloat16))
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    L = B.lib()
    base = [B._ptr(qa), B._ptr(sa), B._ptr(asum), B._ptr(packed)]
    tail = [B._ptr(y), M, N, K, 128, B._ptr(ws), ws.numel(), None]
    assert L.w4a8_gemm_residual(B.PATH_AUTO, *base, None, *tail) == B.ERR_NULL
    assert L.w4a8_gemm_residual(B.PATH_AUTO, *base, y.data_ptr() + 2, *tail) == B.ERR_ALIGN
    assert L.w4a8_gemm_residual(B.PATH_SPLITK_WORKSPACE, *base, B._ptr(y), *tail) == B.ERR_SHAPE
    torch.cuda.synchronize()
