"""The allocation-free GEMM entry point against the regular one.

w4a8_gemm_static_scratch exists for callers that may not allocate device memory (a
deadline-driven control loop, a component living inside someone else's memory pool): its
split-K scratch is a fixed array inside the library instead of a caller-provided workspace.
It runs the same kernel as w4a8_gemm, so on the same inputs it must give the same bf16
output - checked here on two calls in a row, because the second call finds the shared
array as the first one left it.  Collected last on purpose (the file name sorts after
the other tests), and it passes alone in a fresh process as well as after them.
"""
import numpy as np
import pytest
import torch

from oracle import cfast
from oracle import w4a8_oracle as onp
from paper_2608_12932_b200 import binding as B
from paper_2608_12932_b200 import workload as wl
from tests.gpu_util import DeviceLayer, bits

pytestmark = pytest.mark.gpu


def test_static_scratch_matches_workspace_entry_point_twice():
    case = wl.make_layer(1024, 384, 41, 16)
    layer = DeviceLayer(case, 16)
    for call, M in enumerate((8, 16)):          # two calls in a row, different token counts
        qa, sa, asum = layer.quantize(case["x"][:M])
        want, _ = layer.gemm(qa, sa, asum, path=B.PATH_SPLITK_WORKSPACE)   # the same kernel, caller's workspace
        auto, _ = layer.gemm(qa, sa, asum)                                  # what w4a8_gemm picks by itself
        y = torch.full((M, layer.N), float("nan"), dtype=torch.bfloat16, device="cuda")
        B.w4a8_gemm_static_scratch(qa, sa, asum, layer.packed, layer.N, out=y)
        torch.cuda.synchronize()
        got = bits(y)
        # the tolerance the parity tests use, with the regular entry point's output as reference
        ok, ratio = onp.within_tolerance(got, onp.bf16_bits_to_f64(want))
        assert ok, f"call {call}: worst |err|/bound = {ratio}"
        assert np.array_equal(got, want), f"call {call}: same kernel, same inputs, different bits"
        ok, ratio = onp.within_tolerance(got, onp.bf16_bits_to_f64(auto))
        assert ok, f"call {call} against w4a8_gemm: worst |err|/bound = {ratio}"
        # and against the CPU oracle, which shares nothing with either entry point
        ref = cfast.w4a8_linear(case["x"][:M], case["qw"], case["sw"], case["z"], case["group"])
        ok, ratio = onp.within_tolerance(got, ref["ref"])
        assert ok, f"call {call} against the oracle: worst |err|/bound = {ratio}"
        # the status word of this path lives in the fixed array: readable without a workspace pointer
        B.w4a8_static_scratch_status()


def test_static_scratch_second_call_same_shape_and_limits():
    case = wl.make_config("tiny")
    layer = DeviceLayer(case, 16)
    qa, sa, asum = layer.quantize(case["x"])
    want, _ = layer.gemm(qa, sa, asum, path=B.PATH_SPLITK_WORKSPACE)
    for _ in range(2):
        y = B.w4a8_gemm_static_scratch(qa, sa, asum, layer.packed, layer.N)
        torch.cuda.synchronize()
        assert np.array_equal(bits(y), want)
    # a shape whose split-K slices exceed the fixed array is refused, nothing is launched
    L = B.lib()
    big_n, big_k = 24576, 4096          # 4 slices x 64 tokens x 24576 channels x 4 B = 25 MB > 4 MiB
    one = torch.zeros(16, dtype=torch.uint8, device="cuda")
    code = L.w4a8_gemm_static_scratch(qa.data_ptr(), sa.data_ptr(), asum.data_ptr(), layer.packed.data_ptr(),
                                      one.data_ptr(), 64, big_n, big_k, 128, None)
    assert code == B.ERR_WORKSPACE
    assert L.w4a8_gemm_static_scratch(qa.data_ptr(), sa.data_ptr(), asum.data_ptr(), layer.packed.data_ptr(),
                                      one.data_ptr(), 65, 256, 256, 128, None) == B.ERR_SHAPE
    assert L.w4a8_gemm_static_scratch(None, None, None, None, None, 0, 256, 256, 128, None) == B.OK
