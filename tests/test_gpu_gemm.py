"""GPU parity of w4a8_gemm against the CPU oracle, through the C ABI.

Per-group int32 partials D (debug mode) must be bit-exact; the bf16 output must satisfy
|gpu - ref| <= 2^-7 |ref| + 1e-3 rms(ref).  Both kernel families are exercised on shapes
that span several tiles and ragged tails; full-size configurations are checked on sampled
token rows (every output channel of those rows), which the oracle computes one by one.
"""
import numpy as np
import pytest
import torch

from oracle import cfast
from oracle import w4a8_oracle as onp
from paper_2608_12932_b200 import binding as B
from paper_2608_12932_b200 import workload as wl
from tests.gpu_util import DeviceLayer, bits, t_u16

pytestmark = pytest.mark.gpu

PATHS = {"splitk": B.PATH_SPLITK, "splitk_ws": B.PATH_SPLITK_WORKSPACE, "tcgen05": B.PATH_TCGEN05, "auto": B.PATH_AUTO,
         "strip": B.PATH_STRIP}


def check_case(case, layer, M, path, debug=True, rows=None):
    """Run quantise + gemm on the first M rows; compare with the oracle (all rows, or `rows`)."""
    x = case["x"][:M]
    qa, sa, asum = layer.quantize(x)
    y, D = layer.gemm(qa, sa, asum, path=PATHS[path], debug=debug)
    sel = np.arange(M) if rows is None else np.asarray(rows)
    r = cfast.w4a8_linear(x[sel], case["qw"], case["sw"], case["z"], case["group"], want_partials=debug)
    assert np.array_equal(qa.cpu().numpy()[sel], r["qa"])
    assert np.array_equal(bits(sa)[sel], r["sa"])
    if debug:
        bad = np.argwhere(D[sel] != r["D"])
        assert bad.size == 0, f"{len(bad)} partials differ, first (row,g,n) = {bad[:4].tolist()}"
    rms = float(np.sqrt(np.mean(r["ref"] ** 2)))
    ok, ratio = onp.within_tolerance(y[sel], r["ref"], rms_ref=rms)
    assert ok, f"bf16 output outside tolerance: worst |err|/bound = {ratio:.3f}"
    return y, D, r


# ------------------------------------------------------------------ tiny configuration ---
@pytest.mark.parametrize("path", ["splitk", "splitk_ws", "tcgen05", "auto", "strip"])
def test_tiny_config(path):
    case = wl.make_config("tiny")
    layer = DeviceLayer(case, 16)
    y, D, r = check_case(case, layer, 16, path)
    # the numpy oracle agrees with the C one here, so it pins the same result
    rn = onp.w4a8_linear(case["x"], case["qw"], case["sw"], case["z"], 128)
    assert np.array_equal(D, rn["D"])


@pytest.mark.parametrize("path", ["splitk", "splitk_ws", "tcgen05", "strip"])
def test_worked_example_on_gpu(golden, path):
    """The hand-worked example embedded in a 128x128 layer (group 128): same D and y."""
    g = golden("worked_example_w4a8.txt")
    N, K = 128, 128
    x = np.zeros((1, K), np.float32)
    x[0, :8] = g["x"]
    qw = np.zeros((N, K), np.uint8)
    z = np.zeros((1, N), np.uint8)
    sw = np.full((1, N), 0x3C00, np.uint16)
    # the example's two groups of 4 become one group of 128 with a single zero point and scale per row:
    # use its first group only (codes beyond k = 4 equal the zero point, so they contribute nothing)
    for n, (row, zr, sr) in enumerate([(g["qw_row0"], g["z_row0"], g["sw_row0"]), (g["qw_row1"], g["z_row1"], g["sw_row1"])]):
        qw[n, :] = zr[0]
        qw[n, :4] = row[:4]
        z[0, n] = zr[0]
        sw[0, n] = np.float16(sr[0]).view(np.uint16)
    case = dict(x=wl.f32_to_bf16_bits(x), qw=qw, sw=sw, z=z, N=N, K=K, group=128)
    layer = DeviceLayer(case, 1)
    y, D, r = check_case(case, layer, 1, path)
    assert D[0, 0, 0] == g["D_row0"][0] and D[0, 0, 1] == g["D_row1"][0]
    want0 = g["sa"][0] * g["sw_row0"][0] * g["D_row0"][0]
    want1 = g["sa"][0] * g["sw_row1"][0] * g["D_row1"][0]
    assert y[0, 0] == onp.f64_to_bf16_bits(np.array([want0]))[0]
    assert y[0, 1] == onp.f64_to_bf16_bits(np.array([want1]))[0]


# ---------------------------------------------------------------- ragged token counts ---
@pytest.fixture(scope="module")
def mid_case():
    case = wl.make_layer(1024, 384, 31, 600)          # G = 8, three channel tiles
    return case, DeviceLayer(case, 600)


@pytest.mark.parametrize("path", ["splitk", "splitk_ws"])
@pytest.mark.parametrize("M", [1, 3, 8, 9, 16, 17, 32, 33, 63, 64])
def test_splitk_token_counts(mid_case, M, path):
    case, layer = mid_case
    check_case(case, layer, M, path)


@pytest.mark.parametrize("M", [1, 2, 3, 7, 8, 9, 15, 16])
def test_strip_token_counts(mid_case, M):
    """Three channel tiles of eight groups: 16-channel strips, one or two per CTA."""
    case, layer = mid_case
    check_case(case, layer, M, "strip")


# layer shapes chosen for the strip widths the planner picks on 148 SMs and for how the strips fall on the CTAs
STRIP_SHAPES = [
    (512, 128, 16),       # 8 strips of 16 channels, 8 CTAs with one strip each, one ragged stage per strip
    (1280, 2432, 16),     # 152 strips of 16, one per CTA; 10 groups in stages of 16
    (1024, 4864, 16),     # 304 strips of 16 on 296 CTAs: nearly every strip is shared by two CTAs
    (3072, 6144, 32),     # 192 strips of 32, 24 groups in stages of 8
    (640, 12288, 32),     # 384 strips of 32 on 296 CTAs, 5 groups in stages of 8 (one ragged stage per strip)
    (896, 37888, 128),    # 296 strips of 128: exactly one per CTA
    (384, 24576, 64),     # 384 strips of 64, 3 groups in stages of 4
    (1024, 49152, 128),   # 384 strips of 128 on 296 CTAs: ranges of 1.3 strips, hand-over
    (4096, 24576, 64),    # 384 strips of 64, 32 groups: the ring re-used
]


@pytest.mark.parametrize("K,N,rows", STRIP_SHAPES)
def test_strip_widths_and_hand_over(K, N, rows):
    """Every strip width, with and without strips shared between neighbouring CTAs; partials bit-exact, output in
    tolerance; twice in a row on one workspace, since the hand-over flags must be back at zero for the next call,
    and bit-identical both times."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    case = wl.make_layer(K, N, 50 + rows, 16)
    layer = DeviceLayer(case, 16)
    for M in (8, 16, 5):
        plan = B.w4a8_plan(M, N, K)
        if plan["family"] == B.PATH_STRIP:
            assert plan["k_slices"] == 1 and plan["ctas"] <= min(2 * sms, N // plan["strip_rows"])
            if sms == 148:
                assert plan["strip_rows"] == (rows if M <= 8 else 32), plan
        y1, _, _ = check_case(case, layer, M, "strip", debug=(K * N <= 1 << 26))
        y2, _, _ = check_case(case, layer, M, "strip", debug=False)
        assert np.array_equal(y1, y2)
        check_case(case, layer, M, "auto", debug=False)


# token tiles are 64, 128 or 208 rows; a 208-row tile is drained in column pieces of 32, 32, 32 and 8
@pytest.mark.parametrize("M", [1, 16, 64, 65, 96, 97, 104, 105, 128, 129, 200, 207, 208, 209, 255, 256, 257, 300, 415, 416, 417,
                               520, 600])
def test_tcgen05_token_counts(mid_case, M):
    case, layer = mid_case
    check_case(case, layer, M, "tcgen05")


@pytest.fixture(scope="module")
def wide_case():
    case = wl.make_layer(1024, 5120, 36, 1000)        # 40 channel tiles
    return case, DeviceLayer(case, 1000)


@pytest.mark.parametrize("M", [300, 417, 624, 625, 1000])
def test_tcgen05_tile_heights_and_waves(wide_case, M):
    """Token counts on both sides of the dispatch's choice between 128- and 208-row tiles, with more
    tiles than SMs for the larger ones (a CTA then walks several tiles)."""
    case, layer = wide_case
    check_case(case, layer, M, "tcgen05")
    check_case(case, layer, M, "auto", debug=False)


@pytest.mark.parametrize("M", [1, 8, 64, 65, 300])
def test_auto_dispatch(mid_case, M):
    case, layer = mid_case
    check_case(case, layer, M, "auto")


def test_long_k_many_slices():
    case = wl.make_layer(3072, 256, 32, 70)           # G = 24: several slices, uneven split
    layer = DeviceLayer(case, 70)
    for M in (5, 16, 40):
        check_case(case, layer, M, "splitk")
        check_case(case, layer, M, "splitk_ws")
    check_case(case, layer, 70, "tcgen05")


def test_tcgen05_k_split_uneven_slices():
    """Few tiles, so the tensor-core kernel splits K over a cluster: 13 groups over 2 or 3 slices
    (uneven shares), 24 groups over 4; debug partials from every slice land at their own group index."""
    case = wl.make_layer(1664, 256, 37, 210)          # G = 13, two channel tiles
    layer = DeviceLayer(case, 210)
    for M in (33, 64, 100, 128, 129, 210):
        check_case(case, layer, M, "tcgen05")
    case = wl.make_layer(3072, 384, 38, 64)           # G = 24, three channel tiles
    layer = DeviceLayer(case, 64)
    for M in (17, 64):
        check_case(case, layer, M, "tcgen05")
        check_case(case, layer, M, "auto", debug=False)


def test_ring_reuse_many_groups_per_cta():
    """Wide layer, few slices: each CTA walks more groups than its ring has stages."""
    case = wl.make_layer(4096, 4096, 34, 24)         # 32 tiles -> 8 slices of 4 groups; and
    layer = DeviceLayer(case, 24)
    check_case(case, layer, 24, "splitk")
    case = wl.make_layer(2048, 24576, 35, 8)         # 192 tiles -> 2 slices of 8 groups > 6 stages
    layer = DeviceLayer(case, 8)
    check_case(case, layer, 8, "splitk")
    check_case(case, layer, 5, "splitk", debug=False)


def test_many_token_tiles_and_very_wide_layer():
    """Index ranges: 97 token tiles of one channel tile (20001 tokens, a ragged last tile), and 296 channel
    tiles (two per SM on the split-K path, two rounds of tiles on the tensor-core path)."""
    case = wl.make_layer(256, 128, 39, 20001)
    layer = DeviceLayer(case, 20001)
    rng = np.random.default_rng(3)
    rows = np.unique(np.concatenate([[0, 207, 208, 19967, 19968, 20000], rng.integers(0, 20001, 40)]))
    check_case(case, layer, 20001, "tcgen05", debug=True, rows=rows)
    case = wl.make_layer(256, 296 * 128, 40, 300)
    layer = DeviceLayer(case, 300)
    check_case(case, layer, 8, "splitk")
    check_case(case, layer, 16, "splitk")
    check_case(case, layer, 300, "tcgen05", rows=[0, 1, 207, 208, 299])


def test_balanced_walk_hands_partial_tiles_over():
    """160 tiles of 48 groups on at most 148 CTAs: the launcher deals the 7680 tile-groups out evenly (52 per CTA
    instead of 96 for the CTAs with two whole tiles), so most tiles are summed by two neighbouring CTAs and
    meet in the workspace's hand-over area.  Partials bit-exact, output in tolerance, on sampled rows of every
    token tile; twice, since the hand-over flags must be back at zero for the next call."""
    case = wl.make_layer(6144, 4096, 41, 1024)
    layer = DeviceLayer(case, 1024)
    plan = B.w4a8_plan(1024, 4096, 6144)
    assert plan["tile_m"] == 208 and plan["balanced"] == 1 and plan["k_slices"] == 1
    rng = np.random.default_rng(4)
    rows = np.unique(np.concatenate([[0, 207, 208, 415, 416, 831, 832, 1023], rng.integers(0, 1024, 16)]))
    y1, _, _ = check_case(case, layer, 1024, "tcgen05", debug=True, rows=rows)
    y2, _, _ = check_case(case, layer, 1024, "auto", debug=False, rows=rows)
    assert np.array_equal(y1, y2)


def test_persistent_tiles_more_than_sms():
    """160 output tiles over at most 148 CTAs: some CTAs run two tiles back to back."""
    case = wl.make_layer(512, 5120, 33, 1024)
    layer = DeviceLayer(case, 1024)
    check_case(case, layer, 1024, "tcgen05", debug=True)
    check_case(case, layer, 1000, "tcgen05", debug=False)


# -------------------------------------------------------- invariants on the device -------
@pytest.mark.parametrize("path,M", [("splitk", 8), ("splitk_ws", 8), ("splitk", 40), ("tcgen05", 130), ("strip", 8), ("strip", 13)])
def test_zero_point_invariant_and_determinism(mid_case, path, M):
    case, layer = mid_case
    c2 = dict(case)
    c2["qw"] = np.repeat(case["z"].T, 128, axis=1).astype(np.uint8)      # every code equals its zero point
    l2 = DeviceLayer(c2, M)
    qa, sa, asum = l2.quantize(case["x"][:M])
    y, D = l2.gemm(qa, sa, asum, path=PATHS[path], debug=True)
    assert not D.any() and not y.any()                                    # exact zeros, +0 bit patterns
    # run-to-run determinism on the real weights
    qa, sa, asum = layer.quantize(case["x"][:M])
    y1, _ = layer.gemm(qa, sa, asum, path=PATHS[path])
    y2, _ = layer.gemm(qa, sa, asum, path=PATHS[path])
    assert np.array_equal(y1, y2)


@pytest.mark.parametrize("path,M", [("splitk", 5), ("splitk", 16), ("splitk_ws", 8), ("tcgen05", 40), ("tcgen05", 209),
                                    ("strip", 5), ("strip", 16)])
def test_extreme_codes_zero_points_and_symmetric_scheme(path, M):
    """Every activation code at +-127 (rows of constant magnitude) against groups whose codes and zero
    points sit at the ends of their ranges (q - z = +-15: the largest partials, |D| = 243840), the
    symmetric scheme (z = 8 in every group) and random groups: partials bit-exact, output in tolerance."""
    rng = np.random.default_rng(11)
    K, N, g = 1024, 256, 128
    G = K // g
    qw = rng.integers(0, 16, size=(N, K), dtype=np.uint8)
    z = rng.integers(0, 16, size=(G, N), dtype=np.uint8)
    qw[:, 0 * g:1 * g], z[0] = 15, 0                      # q - z = +15 everywhere
    qw[:, 1 * g:2 * g], z[1] = 0, 15                      # q - z = -15 everywhere
    z[2], z[3] = 8, 8                                     # symmetric int4, random codes
    qw[:, 4 * g:5 * g] = np.where(rng.random((N, g)) < 0.5, 0, 15).astype(np.uint8)
    z[4] = np.where(rng.random(N) < 0.5, 0, 15).astype(np.uint8)       # codes and zero points at both ends
    sw = (rng.random((G, N)) * 0.01 + 0.001).astype(np.float16).view(np.uint16)
    mag = rng.choice(np.array([0.25, 1.0, 3.0, 20.0]), size=(M, 1))
    sign = np.where(rng.random((M, K)) < 0.5, -1.0, 1.0)
    sign[0], sign[M - 1] = 1.0, -1.0                      # whole rows at +127 and at -127
    x = wl.f32_to_bf16_bits((mag * sign).astype(np.float32))
    case = dict(x=x, qw=qw, sw=sw, z=z, group=g, N=N, K=K)
    layer = DeviceLayer(case, M)
    y, D, r = check_case(case, layer, M, path)
    assert set(np.unique(np.abs(r["qa"]))) == {127}
    assert D[0, 0].max() == 243840 and D[0, 1].min() == -243840 and D[M - 1, 0].min() == -243840


def test_both_paths_give_identical_partials(mid_case):
    case, layer = mid_case
    M = 48
    qa, sa, asum = layer.quantize(case["x"][:M])
    y1, D1 = layer.gemm(qa, sa, asum, path=B.PATH_SPLITK, debug=True)
    y2, D2 = layer.gemm(qa, sa, asum, path=B.PATH_TCGEN05, debug=True)
    y4, D4 = layer.gemm(qa, sa, asum, path=B.PATH_SPLITK_WORKSPACE, debug=True)
    assert np.array_equal(D1, D2) and np.array_equal(D1, D4)
    # row independence: row 5 of the M = 48 call equals the M = 1 call on that row
    y3, D3 = layer.gemm(qa[5:6].contiguous(), sa[5:6].contiguous(), asum[5:6].contiguous(), path=B.PATH_SPLITK, debug=True)
    assert np.array_equal(D3[0], D1[5])
    # the strip kernel on the first 16 of those rows
    y5, D5 = layer.gemm(qa[:16].contiguous(), sa[:16].contiguous(), asum[:16].contiguous(), path=B.PATH_STRIP, debug=True)
    assert np.array_equal(D5, D1[:16])


def test_scale_linearity_on_gpu(mid_case):
    case, layer = mid_case
    M = 8
    qa, sa, asum = layer.quantize(case["x"][:M])
    y1, _ = layer.gemm(qa, sa, asum)
    c4 = dict(case)
    c4["sw"] = (onp.fp16_bits_to_f64(case["sw"]) * 4).astype(np.float16).view(np.uint16)
    l4 = DeviceLayer(c4, M)
    y4, _ = l4.gemm(qa, sa, asum)
    assert np.array_equal(onp.bf16_bits_to_f64(y4), onp.bf16_bits_to_f64(y1) * 4)


# --------------------------------------------------------------------------- errors ------
def test_gemm_errors(mid_case):
    case, layer = mid_case
    qa, sa, asum = layer.quantize(case["x"][:8])
    small_ws = torch.zeros(B.WORKSPACE_HEADER_BYTES, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.W4A8Error) as e:
        B.w4a8_gemm(qa, sa, asum, layer.packed, layer.N, small_ws)
    assert e.value.code == B.ERR_WORKSPACE
    with pytest.raises(B.W4A8Error) as e:
        B.w4a8_gemm(qa, sa, asum, layer.packed, 100, layer.ws)
    assert e.value.code == B.ERR_SHAPE
    qa70 = torch.zeros((70, case["K"]), dtype=torch.int8, device="cuda")
    with pytest.raises(B.W4A8Error) as e:
        B.w4a8_gemm(qa70, torch.zeros(70, dtype=torch.float16, device="cuda"),
                    torch.zeros((70, 8), dtype=torch.int32, device="cuda"), layer.packed, layer.N, layer.ws,
                    path=B.PATH_SPLITK)
    assert e.value.code == B.ERR_SHAPE
    # M = 0 is a no-op
    y = B.w4a8_gemm(qa[:0], sa[:0], asum[:0], layer.packed, layer.N, layer.ws)
    assert y.shape == (0, layer.N)
    # NULL pointer through the raw ABI
    code = B.lib().w4a8_gemm(None, None, None, None, None, 8, layer.N, case["K"], 128, None, 0, None, None)
    assert code == B.ERR_NULL


def test_bounded_wait_runs_out_and_the_kernel_returns(mid_case):
    """The give-up path, made to happen without a fault: a self-test form of the split-K kernel withholds one weight
    copy per CTA and waits 200 microseconds at most.  The kernel returns, the status word reads TIMEOUT exactly once,
    and the same workspace then serves a normal call whose result is right."""
    case, layer = mid_case
    qa, sa, asum = layer.quantize(case["x"][:8])
    B.w4a8_selftest_wait_timeout(qa, sa, asum, layer.packed, layer.N, layer.ws)
    torch.cuda.synchronize()                      # the kernel has returned: nothing hangs
    with pytest.raises(B.W4A8Error) as e:
        B.w4a8_check_status(layer.ws)
    assert e.value.code == B.ERR_TIMEOUT
    B.w4a8_check_status(layer.ws)                 # cleared by the read
    for path in ("splitk_ws", "splitk", "strip"):
        check_case(case, layer, 8, path)


# ------------------------------------------------- full-size configurations (sampled) ---
def sample_rows(M, rng, k=20):
    edges = [0, M - 1] + [m for m in (63, 64, 127, 128, 255, 256, 257, 511, 512, 1023) if m < M]
    extra = rng.choice(M, size=min(k, M), replace=False).tolist()
    return sorted(set(edges + extra))


def test_spec_verify_full_size():
    """M = 8, K = 4096, N = 6144 in the launch configuration the benchmark times: every output, every partial."""
    case = wl.make_config("spec_verify")
    layer = DeviceLayer(case, 8)
    check_case(case, layer, 8, "strip", debug=True)
    check_case(case, layer, 8, "auto", debug=True)
    check_case(case, layer, 8, "auto", debug=False)
    check_case(case, layer, 8, "splitk", debug=False)
    check_case(case, layer, 8, "tcgen05", debug=False)


@pytest.mark.parametrize("name", ["prefill_gate_up", "prefill_down"])
def test_prefill_full_size_sampled_rows(name):
    case = wl.make_config(name)
    M = case["M"]
    layer = DeviceLayer(case, M)
    rows = sample_rows(M, np.random.default_rng(1))
    x = case["x"]
    qa, sa, asum = layer.quantize(x)
    # non-debug launch: the configuration the benchmark times
    y, _ = layer.gemm(qa, sa, asum)
    r = cfast.w4a8_linear(x[rows], case["qw"], case["sw"], case["z"], 128, want_partials=True)
    assert np.array_equal(qa.cpu().numpy()[rows], r["qa"])
    rms = float(np.sqrt(np.mean(r["ref"] ** 2)))
    ok, ratio = onp.within_tolerance(y[rows], r["ref"], rms_ref=rms)
    assert ok, f"worst |err|/bound = {ratio:.3f}"
    # rms(ref) above is taken over the sampled rows; the tolerance is stated over the whole result: the two agree
    # (the rms of the whole GPU output, every row, is within 2 % of the sample's)
    rms_all = float(np.sqrt(np.mean(onp.bf16_bits_to_f64(y) ** 2)))
    assert abs(rms_all / rms - 1.0) < 0.02, (rms_all, rms)
    # debug launch: partials of the sampled rows, gathered on the device
    G = case["K"] // 128
    D = torch.full((M, G, case["N"]), 0x7FFFFFFF, dtype=torch.int32, device="cuda")
    B.w4a8_gemm(qa, sa, asum, layer.packed, case["N"], layer.ws, debug_partials=D)
    B.w4a8_check_status(layer.ws)
    Ds = D[torch.tensor(rows, device="cuda")].cpu().numpy()
    assert np.array_equal(Ds, r["D"])
    # properties that hold at any size: no output left unwritten, finite everywhere
    yt = torch.from_numpy(y.view(np.int16)).view(torch.bfloat16).float()
    assert torch.isfinite(yt).all()


def test_decoder_layer_sweep_sampled():
    """All four linears of the layer at every M of the sweep; sampled rows against the oracle."""
    rng = np.random.default_rng(2)
    for lname in wl.LAYERS:
        case = wl.make_sweep_layer(lname)
        layer = DeviceLayer(case, 4096)
        for M in wl.SWEEP_M + (32, 24):          # 32 and 24: the remaining small-M template variants
            x = case["x"][:M]
            qa, sa, asum = layer.quantize(x)
            y, _ = layer.gemm(qa, sa, asum)
            rows = sample_rows(M, rng, k=6)
            r = cfast.w4a8_linear(x[rows], case["qw"], case["sw"], case["z"], 128)
            assert np.array_equal(qa.cpu().numpy()[rows], r["qa"]), (lname, M)
            assert np.array_equal(bits(sa)[rows], r["sa"]), (lname, M)
            assert np.array_equal(asum.cpu().numpy()[rows], r["asum"]), (lname, M)
            rms = float(np.sqrt(np.mean(r["ref"] ** 2)))
            ok, ratio = onp.within_tolerance(y[rows], r["ref"], rms_ref=rms)
            assert ok, f"{lname} M={M}: worst |err|/bound = {ratio:.3f}"
        del layer
        torch.cuda.empty_cache()


# ------------------------------------------- w4a8_linear: quantise + multiply, one call ---
def _linear(case, layer, M):
    x = t_u16(case["x"][:M], torch.bfloat16)
    y = B.w4a8_linear(x, layer.packed, case["N"], layer.ws)
    torch.cuda.synchronize()
    B.w4a8_check_status(layer.ws)
    return bits(y)


@pytest.mark.parametrize("M", [1, 2, 7, 8, 9, 15, 16, 17, 40])
def test_linear_matches_two_step_path_and_oracle(mid_case, M):
    """w4a8_linear gives the very bits of w4a8_quantize_act followed by w4a8_gemm."""
    case, layer = mid_case
    y1 = _linear(case, layer, M)
    qa, sa, asum = layer.quantize(case["x"][:M])
    y2, _ = layer.gemm(qa, sa, asum)
    assert np.array_equal(y1, y2)
    r = cfast.w4a8_linear(case["x"][:M], case["qw"], case["sw"], case["z"], case["group"])
    ok, ratio = onp.within_tolerance(y1, r["ref"])
    assert ok, f"worst |err|/bound = {ratio:.3f}"


def test_linear_edge_rows_and_many_slices():
    """Zero rows, a saturating row, a subnormal scale, exact ties, on a layer whose K is split over
    several slices with an uneven number of groups each."""
    case = wl.make_layer(3072, 256, 41, 16)
    rng = np.random.default_rng(9)
    x = wl.bf16_bits_to_f32(case["x"]).copy()
    x[0] = 0.0
    x[1] *= np.float32(2.0 ** 100)
    x[2] *= np.float32(2.0 ** -12)
    x[3] *= np.float32(2.0 ** -40)
    x[4] = np.arange(3072, dtype=np.float32) * np.float32(0.015625) - 8
    x[5] = 1.0
    x[6, :] = 0.0
    x[6, 1500] = -5.0
    case = dict(case, x=wl.f32_to_bf16_bits(x))
    layer = DeviceLayer(case, 16)
    for M in (7, 8, 16):
        y1 = _linear(case, layer, M)
        qa, sa, asum = layer.quantize(case["x"][:M])
        y2, _ = layer.gemm(qa, sa, asum)
        assert np.array_equal(y1, y2)
        r = cfast.w4a8_linear(case["x"][:M], case["qw"], case["sw"], case["z"], case["group"])
        finite = np.isfinite(r["ref"]).all(axis=1)
        rms = float(np.sqrt(np.mean(r["ref"][finite] ** 2)))
        ok, ratio = onp.within_tolerance(y1[finite], r["ref"][finite], rms_ref=rms)
        assert ok, f"worst |err|/bound = {ratio:.3f}"


def test_linear_full_size_spec_verify():
    case = wl.make_config("spec_verify")
    layer = DeviceLayer(case, case["M"])
    y = _linear(case, layer, case["M"])
    r = cfast.w4a8_linear(case["x"], case["qw"], case["sw"], case["z"], case["group"])
    ok, ratio = onp.within_tolerance(y, r["ref"])
    assert ok, f"worst |err|/bound = {ratio:.3f}"
    for name in ("o", "gate_up", "down"):
        c = wl.make_sweep_layer(name, 8)
        lay = DeviceLayer(c, 8)
        for M in (1, 4, 8):
            yy = _linear(c, lay, M)
            rr = cfast.w4a8_linear(c["x"][:M], c["qw"], c["sw"], c["z"], c["group"])
            ok, ratio = onp.within_tolerance(yy, rr["ref"])
            assert ok, f"{name} M={M}: worst |err|/bound = {ratio:.3f}"


def test_linear_errors():
    case, M = wl.make_config("tiny"), 4
    layer = DeviceLayer(case, 16)
    x = t_u16(case["x"][:M], torch.bfloat16)
    with pytest.raises(B.W4A8Error) as e:
        B.w4a8_linear(x, layer.packed, 100, layer.ws)
    assert e.value.code == B.ERR_SHAPE
    buf = torch.zeros(4 * 256 + 8, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.W4A8Error) as e:
        B.w4a8_linear(buf[1:1 + 1024].view(4, 256), layer.packed, case["N"], layer.ws)
    assert e.value.code == B.ERR_ALIGN
    y = B.w4a8_linear(torch.empty((0, 256), dtype=torch.bfloat16, device="cuda"), layer.packed, case["N"], layer.ws)
    assert y.shape == (0, case["N"])


def test_plan_matches_the_device():
    """On the GPU the planner may split K over a cluster when a problem has few tiles; whatever it
    picks fits the machine, and the result of the dispatch it describes is right."""
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    p = B.w4a8_plan(64, 4096, 12288)                  # down projection, 32 tiles, 96 groups
    assert p["family"] == B.PATH_TCGEN05 and p["k_slices"] > 1 and p["ctas"] <= sms
    p = B.w4a8_plan(8, 6144, 4096)
    assert (p["family"] == B.PATH_STRIP and p["ctas"] == min(2 * sms, 6144 // p["strip_rows"]) and p["k_slices"] == 1) or \
        (p["family"] == B.PATH_SPLITK and p["ctas"] == 48 * p["k_slices"])
    p = B.w4a8_plan(40, 6144, 4096)
    assert (p["family"] == B.PATH_SPLITK and p["ctas"] == 48 * p["k_slices"]) or p["family"] == B.PATH_TCGEN05
    p = B.w4a8_plan(1024, 24576, 4096)
    assert p == {"family": B.PATH_TCGEN05, "tile_m": 208, "k_slices": 1, "ctas": sms, "balanced": 0, "strip_rows": 0}
    p = B.w4a8_plan(1024, 4096, 12288)                # 160 tiles of 96 groups: evenly dealt out
    assert p == {"family": B.PATH_TCGEN05, "tile_m": 208, "k_slices": 1, "ctas": sms, "balanced": 1, "strip_rows": 0}
