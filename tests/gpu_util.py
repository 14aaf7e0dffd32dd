"""Helpers for the GPU parity tests: move a synthetic case to the device, run the library
through its C ABI (via the ctypes binding), bring results back as numpy bit patterns."""
import numpy as np
import torch

from paper_2608_12932_b200 import binding as B


def t_u16(a, dtype):
    """numpy uint16 bit patterns -> CUDA tensor of a 16-bit float dtype."""
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).cuda().view(dtype)


def bits(t):
    """CUDA 16-bit float tensor -> numpy uint16 bit patterns."""
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


class DeviceLayer:
    """A packed layer on the device plus its workspace."""

    def __init__(self, case, m_max):
        self.N, self.K, self.group = case["N"], case["K"], case["group"]
        self.qw = torch.from_numpy(case["qw"]).cuda()
        self.sw = t_u16(case["sw"], torch.float16)
        self.z = torch.from_numpy(case["z"]).cuda()
        self.packed = B.w4a8_pack_weights(self.qw, self.sw, self.z, self.group)
        self.ws = B.new_workspace(m_max, self.N, self.K, self.group)

    def quantize(self, x_bits):
        x = t_u16(x_bits, torch.bfloat16)
        return B.w4a8_quantize_act(x, self.group)

    def gemm(self, qa, sa, asum, path=B.PATH_AUTO, debug=False):
        M = qa.shape[0]
        D = None
        if debug:
            D = torch.full((M, self.K // self.group, self.N), 0x7FFFFFFF, dtype=torch.int32, device="cuda")
        y = torch.full((M, self.N), float("nan"), dtype=torch.bfloat16, device="cuda")
        B.w4a8_gemm(qa, sa, asum, self.packed, self.N, self.ws, self.group, out=y, debug_partials=D, path=path)
        B.w4a8_check_status(self.ws)
        return bits(y), (D.cpu().numpy() if debug else None)
