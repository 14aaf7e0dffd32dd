"""GPU parity: activation quantiser and weight packer against the CPU oracle, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import cfast
from oracle import w4a8_oracle as onp
from paper_2608_12932_b200 import binding as B
from paper_2608_12932_b200 import workload as wl
from tests.gpu_util import DeviceLayer, bits, t_u16

pytestmark = pytest.mark.gpu


def gpu_quantize(x_bits, group=128):
    qa, sa, asum = B.w4a8_quantize_act(t_u16(x_bits, torch.bfloat16), group)
    torch.cuda.synchronize()
    return qa.cpu().numpy(), bits(sa), asum.cpu().numpy()


def assert_quantize_parity(x_bits):
    qa, sa, asum = gpu_quantize(x_bits)
    rq, rs, ra = cfast.quantize_act(x_bits, 128)
    assert np.array_equal(sa, rs), "token scales differ"
    assert np.array_equal(qa, rq), f"codes differ at {np.argwhere(qa != rq)[:5]}"
    assert np.array_equal(asum, ra), "group sums differ"
    return qa, sa, asum


@pytest.mark.parametrize("M,K,seed", [(16, 256, 0), (8, 4096, 0), (1, 128, 1), (37, 12288, 2), (5, 16512, 3),
                                      (1024, 4096, 4), (3, 2048 + 128, 5),
                                      # every threads-per-row variant of the kernel, short and long rows
                                      (100, 4096, 6), (128, 128, 7), (70, 16512, 8), (400, 12288, 9), (513, 1024, 10)])
def test_quantize_matches_oracle(M, K, seed):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((M, K), dtype=np.float32)
    idx = rng.choice(K, max(1, round(0.01 * K)), replace=False)
    x[:, idx] *= 20
    qa, sa, _ = assert_quantize_parity(wl.f32_to_bf16_bits(x))
    assert np.abs(qa).max() == 127


def test_quantize_numpy_oracle_agrees_too():
    c = wl.make_config("tiny")
    qa, sa, asum = gpu_quantize(c["x"])
    rq, rs, ra = onp.quantize_act(c["x"], 128)
    assert np.array_equal(qa, rq) and np.array_equal(sa, rs) and np.array_equal(asum, ra)


def test_quantize_golden_examples(golden):
    """The hand-worked examples, zero-padded to one group of 128."""
    g = golden("worked_example_w4a8.txt")
    t = golden("tie_and_clamp_examples.txt")
    rows, want_q, want_s = [], [], []
    rows.append(g["x"]); want_q.append(g["qa"]); want_s.append(g["sa"][0])
    for case in "ABCDE":
        rows.append(t[f"case{case}_x"]); want_q.append(t[f"case{case}_qa"]); want_s.append(t[f"case{case}_sa"][0])
    x = np.zeros((len(rows), 128), dtype=np.float32)
    for i, r in enumerate(rows):
        x[i, :len(r)] = r
    xb = wl.f32_to_bf16_bits(x)
    assert np.array_equal(wl.bf16_bits_to_f32(xb), x)
    qa, sa, asum = gpu_quantize(xb)
    for i, (q, s) in enumerate(zip(want_q, want_s)):
        assert qa[i, :len(q)].tolist() == q, f"row {i}"
        assert not qa[i, len(q):].any()
        assert onp.fp16_bits_to_f64(sa)[i] == s, f"row {i}"
        assert asum[i, 0] == sum(q)


def test_quantize_edge_rows():
    rng = np.random.default_rng(7)
    K = 1024
    x = rng.standard_normal((12, K), dtype=np.float32)
    x[0] = 0.0
    x[1] = -0.0
    x[2] *= np.float32(2.0 ** 100)          # scale saturates at 65504
    x[3] *= np.float32(2.0 ** -12)          # scale is an fp16 subnormal
    x[4] *= np.float32(2.0 ** -40)          # scale underflows to zero
    x[5, :] = 3.96875 / 127                 # every quotient equal
    x[5, 0] = 3.96875
    x[6] = np.arange(K, dtype=np.float32) * np.float32(0.015625) - 8   # many exact ties under scale 2^-5 * k
    x[6, 0] = 3.96875 * 2
    x[7] = 1.0
    x[8, :] = 0.0
    x[8, 77] = -5.0                         # a single non-zero
    x[9] = np.float32(65280.0)              # large equal values
    x[10] = np.where(rng.random(K) < 0.5, 1.0, -1.0).astype(np.float32) * np.float32(0.0078125)
    xb = wl.f32_to_bf16_bits(x)
    qa, sa, asum = assert_quantize_parity(xb)
    assert sa[0] == 0 and sa[1] == 0 and not qa[:2].any()
    assert sa[2] == 0x7BFF                 # 65504
    assert 0 < sa[3] < 0x0400              # subnormal
    assert sa[4] == 0 and not qa[4].any()
    assert qa[8, 77] == -127 and np.count_nonzero(qa[8]) == 1
    assert qa.min() >= -127


def test_quantize_empty_and_errors():
    x = torch.empty((0, 256), dtype=torch.bfloat16, device="cuda")
    qa, sa, asum = B.w4a8_quantize_act(x)
    assert qa.shape == (0, 256) and sa.shape == (0,)
    x = torch.zeros((2, 200), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.W4A8Error) as e:
        B.w4a8_quantize_act(x)
    assert e.value.code == B.ERR_SHAPE
    x = torch.zeros((2, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.W4A8Error) as e:
        B.w4a8_quantize_act(x, group=64)
    assert e.value.code == B.ERR_SHAPE
    # misaligned input (offset by one bf16 element = 2 bytes)
    buf = torch.zeros(2 * 256 + 8, dtype=torch.bfloat16, device="cuda")
    mis = buf[1:1 + 512].view(2, 256)
    with pytest.raises(B.W4A8Error) as e:
        B.w4a8_quantize_act(mis)
    assert e.value.code == B.ERR_ALIGN


@pytest.mark.parametrize("N,K,seed", [(128, 128, 0), (256, 384, 1), (6144, 4096, 2)])
def test_pack_unpack_round_trip(N, K, seed):
    rng = np.random.default_rng(seed)
    c = wl.random_codes(rng, 0, N, K)
    layer = DeviceLayer(c, 1)
    assert layer.packed.numel() == N * K // 2 + (K // 128) * N * 5 // 2       # exactly the algorithmic bytes
    qw, sw, z = B.w4a8_unpack_weights(layer.packed, N, K)
    torch.cuda.synchronize()
    assert np.array_equal(qw.cpu().numpy(), c["qw"])
    assert np.array_equal(bits(sw), c["sw"])
    assert np.array_equal(z.cpu().numpy(), c["z"])


def test_pack_is_a_permutation_of_nibbles():
    """Every code lands in exactly one nibble: pack a one-hot pattern per position and count."""
    N, K = 128, 256
    rng = np.random.default_rng(3)
    qw = np.zeros((N, K), np.uint8)
    hot = [(int(rng.integers(N)), int(rng.integers(K))) for _ in range(64)]
    for i, (n, k) in enumerate(hot):
        qw[n, k] = 1 + (i % 15)
    c = dict(qw=qw, sw=np.full((2, N), 0x3C00, np.uint16), z=np.zeros((2, N), np.uint8), N=N, K=K, group=128)
    layer = DeviceLayer(c, 1)
    blob = layer.packed.cpu().numpy().reshape(2, -1)[:, :8192]
    nib = np.concatenate([blob & 0xF, blob >> 4], axis=1)
    assert np.count_nonzero(nib) == len(set(hot))
    assert sorted(nib[nib != 0].tolist()) == sorted(int(qw[n, k]) for n, k in set(hot))


def test_pack_errors():
    qw = torch.zeros((100, 256), dtype=torch.uint8, device="cuda")
    with pytest.raises(B.W4A8Error) as e:
        B.w4a8_pack_weights(qw, torch.zeros((2, 100), dtype=torch.float16, device="cuda"),
                            torch.zeros((2, 100), dtype=torch.uint8, device="cuda"))
    assert e.value.code == B.ERR_SHAPE
    assert B.w4a8_packed_bytes(100, 256) == 0 and B.w4a8_packed_bytes(128, 200) == 0
    assert B.w4a8_packed_bytes(128, 256, 64) == 0
