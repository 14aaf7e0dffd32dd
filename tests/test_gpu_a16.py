"""GPU parity of the weight-only variant (W4A16, Sec. 3.4 first paragraph) on the same packed weights: the small-M
kernel against the fp64 definition within the band of the W4A8 path, the dequantised weights bit for bit."""
import numpy as np
import pytest
import torch

from oracle import w4a8_oracle as onp
from paper_2608_12932_b200 import binding as B
from paper_2608_12932_b200 import workload as wl
from tests.gpu_util import bits, t_u16

pytestmark = pytest.mark.gpu


def pack(c):
    return B.w4a8_pack_weights(torch.from_numpy(c["qw"]).cuda(), t_u16(c["sw"], torch.float16), torch.from_numpy(c["z"]).cuda())


@pytest.mark.parametrize("N,K", [(128, 128), (256, 384), (640, 1024), (4096, 512)])
def test_dequantised_weights_are_bit_exact(N, K):
    c = wl.random_codes(np.random.default_rng(N + K), 1, N, K)
    W = B.w4a8_dequantize_weights(pack(c), N, K)
    torch.cuda.synchronize()
    _, w_bits = onp.dequantize_weights(c["qw"], c["sw"], c["z"], 128)
    assert np.array_equal(bits(W), w_bits)


# (M, K, N): one and two token blocks, every strip width the plan can pick (32 / 64 rows), a ragged last stage
# (K / 128 not a multiple of the groups per stage), strips shared by two CTAs (more strips than CTAs), real layer shapes
SHAPES = [(1, 128, 128), (8, 256, 256), (5, 384, 640), (3, 1152, 384), (8, 4096, 6144), (16, 4096, 6144), (11, 640, 2304),
          (8, 512, 24576), (4, 4096, 24576), (16, 512, 24576), (7, 12288, 4096), (2, 256, 37888)]


@pytest.mark.parametrize("M,K,N", SHAPES)
def test_w4a16_gemm_against_the_definition(M, K, N):
    c = wl.make_layer(K, N, 4000 + M + N, M)
    packed = pack(c)
    ws = B.new_workspace(16, N, K)
    x = t_u16(c["x"], torch.bfloat16)
    ys = []
    for rep in range(3):                                        # the hand-over words must come back to zero each time
        y = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
        B.w4a8_a16_gemm(x, packed, N, ws, out=y)
        torch.cuda.synchronize()
        B.w4a8_check_status(ws)
        ys.append(bits(y))
    assert np.array_equal(ys[0], ys[1]) and np.array_equal(ys[0], ys[2])
    ref = onp.w4a16_linear(c["x"], c["qw"], c["sw"], c["z"], 128)
    ok, worst = onp.within_tolerance(ys[0], ref)
    assert ok, f"worst |err|/bound {worst:.3f}"
    # the W4A8 kernels still work on the same workspace afterwards
    qa, sa, asum = B.w4a8_quantize_act(x)
    y8 = B.w4a8_gemm(qa, sa, asum, packed, N, ws)
    B.w4a8_check_status(ws)
    r8 = onp.w4a8_linear(c["x"], c["qw"], c["sw"], c["z"], 128)["ref"] if M * K * N <= 2 ** 28 else None
    if r8 is not None:
        assert onp.within_tolerance(bits(y8), r8)[0]


def test_w4a16_special_inputs():
    M, K, N = 8, 512, 256
    rng = np.random.default_rng(3)
    c = wl.random_codes(rng, M, N, K)
    G = K // 128
    # every code equal to its zero point: the product is exactly zero whatever x is
    c["qw"] = np.repeat(c["z"].T, 128, axis=1).astype(np.uint8).reshape(N, K)
    ws = B.new_workspace(16, N, K)
    y = B.w4a8_a16_gemm(t_u16(c["x"], torch.bfloat16), pack(c), N, ws)
    torch.cuda.synchronize()
    assert not (bits(y) & 0x7FFF).any()
    # extreme codes and zero points, large and tiny activations: still the definition
    c = wl.random_codes(rng, M, N, K)
    c["qw"][: N // 2] = 15
    c["z"][:, : N // 2] = 0
    c["qw"][N // 2:] = 0
    c["z"][:, N // 2:] = 15
    xf = rng.standard_normal((M, K)).astype(np.float32)
    xf[0] *= 1e4
    xf[1] *= 1e-6
    xf[2] = 0
    c["x"] = wl.f32_to_bf16_bits(xf)
    y = B.w4a8_a16_gemm(t_u16(c["x"], torch.bfloat16), pack(c), N, ws)
    torch.cuda.synchronize()
    B.w4a8_check_status(ws)
    ref = onp.w4a16_linear(c["x"], c["qw"], c["sw"], c["z"], 128)
    # per token: the band with that token's own rms (the rows differ by ten orders of magnitude)
    for m in range(M):
        ok, worst = onp.within_tolerance(bits(y)[m:m + 1], ref[m:m + 1])
        assert ok, (m, worst)
    assert not (bits(y)[2] & 0x7FFF).any()


def test_w4a16_shape_rules():
    K, N = 256, 256
    c = wl.random_codes(np.random.default_rng(0), 17, N, K)
    packed = pack(c)
    ws = B.new_workspace(16, N, K)
    x = t_u16(c["x"], torch.bfloat16)
    assert B.w4a8_a16_gemm(x[:0].contiguous(), packed, N, ws).shape == (0, N)
    with pytest.raises(B.W4A8Error) as e:
        B.w4a8_a16_gemm(x, packed, N, ws)                       # 17 tokens: the decode form stops at 16
    assert e.value.code == B.ERR_SHAPE
    L = B.lib()
    y = torch.empty((8, N), dtype=torch.bfloat16, device="cuda")
    assert L.w4a8_a16_gemm(B._ptr(x) , B._ptr(packed), None, 8, N, K, 128, B._ptr(ws), ws.numel(), None) == B.ERR_NULL
    assert L.w4a8_a16_gemm(x.data_ptr() + 2, B._ptr(packed), B._ptr(y), 8, N, K, 128, B._ptr(ws), ws.numel(), None) == B.ERR_ALIGN
    assert L.w4a8_a16_gemm(B._ptr(x), B._ptr(packed), B._ptr(y), 8, N, K, 128, B._ptr(ws), 1024, None) == B.ERR_WORKSPACE
    torch.cuda.synchronize()
