"""GPU parity of w4a8_gemm_per_channel (scales constant along K: one drain per tile) against the CPU
oracle, through the C ABI.  The int32 sums over all groups (debug mode) must be bit-exact; the bf16
output must satisfy |gpu - ref| <= 2^-7 |ref| + 1e-3 rms(ref), and must agree with w4a8_gemm on the
same packed layer within the same band (the two differ only in fp32 rounding order).
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


def per_channel_case(seed, M, N, K, group=128):
    """Random codes and zero points per group; one fp16 scale per channel, repeated in every group."""
    rng = np.random.default_rng(seed)
    c = wl.random_codes(rng, M, N, K, group)
    G = K // group
    c["sw"] = np.repeat(c["sw"][:1], G, axis=0).copy()
    c.update(N=N, K=K, group=group)
    return c


def run(case, layer, M, debug=True):
    qa, sa, asum = layer.quantize(case["x"][:M])
    sums = torch.full((M, layer.N), 0x7FFFFFFF, dtype=torch.int32, device="cuda") if debug else None
    y = torch.full((M, layer.N), float("nan"), dtype=torch.bfloat16, device="cuda")
    B.w4a8_gemm_per_channel(qa, sa, layer.packed, layer.N, layer.ws, layer.group, out=y, debug_sums=sums)
    B.w4a8_check_status(layer.ws)
    return (qa, sa, asum), bits(y), (sums.cpu().numpy() if debug else None)


def check(case, layer, M, debug=True, rows=None):
    quant, y, sums = run(case, layer, M, debug)
    sel = np.arange(M) if rows is None else np.asarray(rows)
    r = cfast.w4a8_linear(case["x"][:M][sel], case["qw"], case["sw"], case["z"], case["group"], want_partials=True)
    if debug:
        want = r["D"].astype(np.int64).sum(axis=1)
        bad = np.argwhere(sums[sel] != want)
        assert bad.size == 0, f"{len(bad)} sums differ, first (row,n) = {bad[:4].tolist()}"
    rms = float(np.sqrt(np.mean(r["ref"] ** 2)))
    ok, ratio = onp.within_tolerance(y[sel], r["ref"], rms_ref=rms)
    assert ok, f"bf16 output outside tolerance: worst |err|/bound = {ratio:.3f}"
    return quant, y


@pytest.fixture(scope="module")
def pc_case():
    case = per_channel_case(21, 640, 384, 1024)
    return case, DeviceLayer(case, 640)


@pytest.mark.parametrize("M", [1, 16, 64, 65, 128, 129, 207, 208, 209, 300, 416, 417, 640])
def test_token_counts_and_tile_heights(pc_case, M):
    case, layer = pc_case
    check(case, layer, M)
    check(case, layer, M, debug=False)


def test_matches_the_per_group_kernel(pc_case):
    """Same packed layer through w4a8_gemm: equal up to fp32 rounding order, i.e. within the band."""
    case, layer = pc_case
    M = 300
    (qa, sa, asum), y_pc, sums = run(case, layer, M)
    y_pg, D = layer.gemm(qa, sa, asum, path=B.PATH_TCGEN05, debug=True)
    assert np.array_equal(D.astype(np.int64).sum(axis=1), sums)
    ref = onp.bf16_bits_to_f64(y_pg)
    ok, ratio = onp.within_tolerance(y_pc, ref)
    assert ok, ratio


def test_several_tiles_per_cta_and_both_buffers():
    """More tiles than SMs, three or more per CTA: the accumulator buffers alternate and are re-zeroed."""
    case = per_channel_case(22, 2000, 5120, 512)
    layer = DeviceLayer(case, 2000)
    rng = np.random.default_rng(5)
    rows = np.unique(np.concatenate([[0, 207, 208, 1999], rng.integers(0, 2000, 24)]))
    check(case, layer, 2000, debug=True, rows=rows)
    # run to run: the same bits
    _, y1, _ = run(case, layer, 2000, debug=False)
    _, y2, _ = run(case, layer, 2000, debug=False)
    assert np.array_equal(y1, y2)


def test_long_k_and_single_group():
    case = per_channel_case(23, 130, 256, 12288)         # 96 groups: |sum| far beyond one group's range
    check(case, DeviceLayer(case, 130), 130)
    case = per_channel_case(24, 64, 20480, 128)          # one group per tile, more tiles than SMs: the two
    check(case, DeviceLayer(case, 64), 64)               # issuing threads take the tiles of a CTA in turn
    case = per_channel_case(25, 420, 640, 384)           # odd number of groups, several tiles per CTA at small N
    check(case, DeviceLayer(case, 420), 420)


def test_errors(pc_case):
    case, layer = pc_case
    qa, sa, asum = layer.quantize(case["x"][:8])
    with pytest.raises(B.W4A8Error) as e:
        B.w4a8_gemm_per_channel(qa, sa, layer.packed, layer.N, layer.ws, group=64)
    assert e.value.code == B.ERR_SHAPE
    small = torch.zeros(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.W4A8Error):
        B.w4a8_gemm_per_channel(qa, sa, layer.packed, layer.N, small)
    y = B.w4a8_gemm_per_channel(qa[:0], sa[:0], layer.packed, layer.N, layer.ws)      # M = 0: nothing to do
    assert tuple(y.shape) == (0, layer.N)
