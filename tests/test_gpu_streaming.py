"""GPU parity of the streaming-prefill pieces (Sec. 3.1): rotary embedding of pre-rotation cached keys at shifted
positions - the bf16 result equals the fp64 definition's or is its neighbour (sine and cosine are fp32) - and the
streaming attention mask, byte for byte."""
import numpy as np
import pytest
import torch

from oracle import streaming as so
from oracle import w4a8_oracle as onp
from paper_2608_12932_b200 import binding as B
from paper_2608_12932_b200 import workload as wl
from tests.gpu_util import bits, t_u16

pytestmark = pytest.mark.gpu


def ordered(b):
    b = b.astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)


@pytest.mark.parametrize("T,H,D,base,pmax", [(1, 1, 4, 1.0e4, 10), (77, 8, 128, 1.0e6, 5000), (300, 2, 64, 1.0e4, 100000),
                                            (33, 4, 256, 5.0e5, 40000), (4096, 8, 128, 1.0e6, 8192), (5, 3, 12, 1.0e4, 50)])
def test_rope_shifted_keys(T, H, D, base, pmax):
    rng = np.random.default_rng(T + D)
    k = wl.f32_to_bf16_bits((rng.standard_normal((T, H, D)) * 3).astype(np.float32))
    pos = rng.integers(0, pmax, size=T).astype(np.int32)
    delta = int(rng.integers(0, 64))
    pos[0] = delta                                              # one token at the shifted position 0: unchanged
    out = B.w4a8_rope_shifted_keys(t_u16(k, torch.bfloat16), torch.from_numpy(pos).cuda(), delta, base)
    torch.cuda.synchronize()
    ref, ref_bits = so.rope_shifted_keys(k, pos, delta, base)
    got = bits(out)
    assert np.array_equal(got[0], k[0])
    d = np.abs(ordered(got) - ordered(ref_bits))
    # where the two products nearly cancel the result is small against its terms: an fp32 error of 1e-6 of the terms may
    # then be several steps of the result
    kf = onp.bf16_bits_to_f64(k)
    half = D // 2
    terms = np.abs(kf[:, :, :half]) + np.abs(kf[:, :, half:])
    terms = np.concatenate([terms, terms], axis=2)
    small = np.abs(onp.bf16_bits_to_f64(got) - ref) <= 1e-6 * terms
    d = np.where(small, np.minimum(d, 1), d)
    assert d.max() <= 1, f"{d.max()} bf16 steps from the definition"
    assert np.count_nonzero(ordered(got) != ordered(ref_bits)) <= 0.01 * d.size + 2
    # in place
    buf = t_u16(k, torch.bfloat16)
    B.w4a8_rope_shifted_keys(buf, torch.from_numpy(pos).cuda(), delta, base, out=buf)
    torch.cuda.synchronize()
    assert np.array_equal(bits(buf), got)


@pytest.mark.parametrize("V,F,n", [(1, 1, 6), (3, 4, 5), (4, 4, 180), (2, 7, 33)])
def test_streaming_mask(V, F, n):
    m = B.w4a8_streaming_mask(V, F, n)
    torch.cuda.synchronize()
    assert np.array_equal(m.cpu().numpy(), so.streaming_mask(V, F, n))


def test_streaming_argument_checks():
    L = B.lib()
    k = torch.zeros((2, 2, 8), dtype=torch.bfloat16, device="cuda")
    pos = torch.zeros((2,), dtype=torch.int32, device="cuda")
    assert L.w4a8_rope_shifted_keys(B._ptr(k), B._ptr(pos), 0, 2, 2, 6, 1.0e4, B._ptr(k), None) == B.ERR_SHAPE      # D % 4
    assert L.w4a8_rope_shifted_keys(B._ptr(k), None, 0, 2, 2, 8, 1.0e4, B._ptr(k), None) == B.ERR_NULL
    assert L.w4a8_rope_shifted_keys(B._ptr(k), B._ptr(pos), 0, 2, 2, 8, 1.0, B._ptr(k), None) == B.ERR_SHAPE       # base
    assert L.w4a8_streaming_mask(0, 1, 1, B._ptr(k), None) == B.ERR_SHAPE
    torch.cuda.synchronize()
