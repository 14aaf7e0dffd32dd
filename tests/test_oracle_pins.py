"""Pins for the CPU oracle: none of these compares an oracle with a retyped copy of itself.

Worked examples (tests/golden), exact-rational brute force, the dequantise-then-dgemm
identity, invariants that the mathematics fixes, and the a-priori quantisation bound.
"""
from fractions import Fraction

import numpy as np
import pytest

from oracle import cfast, exact
from oracle import w4a8_oracle as onp
from paper_2608_12932_b200 import workload as wl

IMPLS = ["numpy", "c"]


def run_impl(impl, x_bits, qw, sw_bits, z, group):
    if impl == "numpy":
        return onp.w4a8_linear(x_bits, qw, sw_bits, z, group)
    return cfast.w4a8_linear(x_bits, qw, sw_bits, z, group, want_partials=True)


def quantize_impl(impl, x_bits, group):
    return onp.quantize_act(x_bits, group) if impl == "numpy" else cfast.quantize_act(x_bits, group)


def bits_bf16(vals):
    a = np.asarray(vals, dtype=np.float32)
    b = wl.f32_to_bf16_bits(a)
    assert np.array_equal(wl.bf16_bits_to_f32(b), a), "fixture value is not a bf16 number"
    return b


def bits_fp16(vals):
    a = np.asarray(vals, dtype=np.float64)
    h = a.astype(np.float16)
    assert np.array_equal(h.astype(np.float64), a), "fixture value is not an fp16 number"
    return h.view(np.uint16)


# ---------------------------------------------------------------- worked example ------
@pytest.mark.parametrize("impl", IMPLS)
def test_worked_example(golden, impl):
    g = golden("worked_example_w4a8.txt")
    group = g["group"][0]
    x = bits_bf16([g["x"]])
    qw = np.array([g["qw_row0"], g["qw_row1"]], dtype=np.uint8)
    z = np.array([g["z_row0"], g["z_row1"]], dtype=np.uint8).T.copy()          # [G,N]
    sw = bits_fp16(np.array([g["sw_row0"], g["sw_row1"]]).T.copy())             # [G,N]
    r = run_impl(impl, x, qw, sw, z, group)
    assert r["sa"].tolist() == g["sa_bits"]
    assert onp.fp16_bits_to_f64(r["sa"]).tolist() == g["sa"]
    assert r["qa"][0].tolist() == g["qa"]
    assert r["asum"][0].tolist() == g["asum"]
    assert r["D"][0, :, 0].tolist() == g["D_row0"]
    assert r["D"][0, :, 1].tolist() == g["D_row1"]
    assert r["ref"][0].tolist() == g["ref"]           # products here are exact in fp64
    assert onp.f64_to_bf16_bits(r["ref"])[0].tolist() == g["y_bf16_bits"]
    assert onp.bf16_bits_to_f64(g["y_bf16_bits"]).tolist() == g["y_bf16"]
    # P = D + z*A restates the uncorrected dot products of the example
    P0 = [d + zz * a for d, zz, a in zip(g["D_row0"], g["z_row0"], g["asum"])]
    P1 = [d + zz * a for d, zz, a in zip(g["D_row1"], g["z_row1"], g["asum"])]
    assert P0 == g["P_row0"] and P1 == g["P_row1"]


def test_worked_example_exact_rational(golden):
    g = golden("worked_example_w4a8.txt")
    x = [[Fraction(v) for v in g["x"]]]
    qw = [g["qw_row0"], g["qw_row1"]]
    z = [[g["z_row0"][i], g["z_row1"][i]] for i in range(2)]
    sw = [[Fraction(g["sw_row0"][i]), Fraction(g["sw_row1"][i])] for i in range(2)]
    r = exact.linear(x, qw, sw, z, g["group"][0])
    assert r["sa"] == [Fraction(g["sa"][0])]
    assert r["qa"] == [g["qa"]]
    assert r["asum"] == [g["asum"]]
    assert [r["D"][0][0][0], r["D"][0][1][0]] == g["D_row0"]
    assert [r["D"][0][0][1], r["D"][0][1][1]] == g["D_row1"]
    assert [float(v) for v in r["y"][0]] == g["ref"]
    assert [float(exact.bf16_rne(v)) for v in r["y"][0]] == g["y_bf16"]


@pytest.mark.parametrize("impl", IMPLS + ["exact"])
@pytest.mark.parametrize("case", "ABCDE")
def test_tie_and_clamp_examples(golden, impl, case):
    g = golden("tie_and_clamp_examples.txt")
    xs, sa, qa = g[f"case{case}_x"], g[f"case{case}_sa"][0], g[f"case{case}_qa"]
    if impl == "exact":
        s, q = exact.quantize_act_row([Fraction(v) for v in xs])
        assert float(s) == sa and q == qa
    else:
        q, s, asum = quantize_impl(impl, bits_bf16([xs]), len(xs))
        assert onp.fp16_bits_to_f64(s)[0] == sa
        assert q[0].tolist() == qa
        assert asum[0, 0] == sum(qa)


def test_weight_quantizer_example(golden):
    g = golden("weight_quantizer_example.txt")
    qw, sw, z = wl.quantize_weights_uint4(np.array([g["w"]], dtype=np.float32), group=4)
    assert qw[0].tolist() == g["qw"]
    assert onp.fp16_bits_to_f64(sw)[0, 0] == g["sw"][0]
    assert z[0, 0] == g["z"][0]


# ------------------------------------------------------- format helpers vs libraries ---
def test_exact_fp16_rounding_matches_numpy_cast():
    rng = np.random.default_rng(1)
    vals = np.concatenate([rng.uniform(0, 70000, 300), rng.uniform(0, 1e-4, 300),
                           rng.uniform(0, 2e-7, 200), [0.0, 65504.0, 65519.9, 2.0 ** -25, 2.0 ** -24]])
    for v in vals:
        want = float(np.float16(min(v, 65504.0)))
        assert float(exact.fp16_rne(Fraction(float(v)))) == want
    # a tie at the subnormal boundary and one in the normal range
    assert exact.fp16_rne(Fraction(3, 2) * Fraction(2) ** -24) == Fraction(2) ** -23
    assert exact.fp16_rne(Fraction(2049)) == 2048 and exact.fp16_rne(Fraction(2051)) == 2052


def test_bf16_rounding_helpers_agree():
    import torch
    rng = np.random.default_rng(2)
    v = np.concatenate([rng.standard_normal(2000) * 10.0 ** rng.integers(-6, 6, 2000),
                        [1.00390625, 1.01171875, -1.00390625, 0.0]])     # includes exact ties
    got = onp.f64_to_bf16_bits(v)
    # torch rounds fp64 -> bf16 through fp32 for most builds; compare only where fp32 is exact
    v32 = v.astype(np.float32).astype(np.float64)
    same = v32 == v
    want = torch.from_numpy(v[same]).to(torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got[same], want)
    for val in v[:200]:
        assert onp.bf16_bits_to_f64(onp.f64_to_bf16_bits(np.array([val])))[0] == float(exact.bf16_rne(Fraction(float(val))))
    # generator-side cast is the same rounding
    f = v.astype(np.float32)
    assert np.array_equal(wl.f32_to_bf16_bits(f), onp.f64_to_bf16_bits(f.astype(np.float64)))


# --------------------------------------------------------- brute force on tiny inputs --
def _exact_inputs(case):
    x = [[Fraction(float(v)) for v in row] for row in wl.bf16_bits_to_f32(case["x"])]
    sw = [[Fraction(float(v)) for v in row] for row in onp.fp16_bits_to_f64(case["sw"])]
    return x, case["qw"].tolist(), sw, case["z"].tolist()


@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("M,N,K,group", [(1, 1, 1, 1), (2, 3, 4, 2), (3, 5, 8, 4), (4, 8, 16, 8), (2, 4, 32, 16)])
def test_brute_force_random_tiny(impl, M, N, K, group):
    for seed in range(4):
        rng = np.random.default_rng(100 + seed)
        case = wl.random_codes(rng, M, N, K, group)
        if seed == 3:      # outlier-heavy rows so that many codes are 0 and some clamp
            xf = wl.bf16_bits_to_f32(case["x"]).copy()
            xf[:, 0] *= 50
            case["x"] = wl.f32_to_bf16_bits(xf)
        r = run_impl(impl, case["x"], case["qw"], case["sw"], case["z"], group)
        e = exact.linear(*_exact_inputs(case), group)
        assert r["qa"].tolist() == e["qa"]
        assert onp.fp16_bits_to_f64(r["sa"]).tolist() == [float(s) for s in e["sa"]]
        assert r["asum"].tolist() == e["asum"]
        assert r["D"].tolist() == e["D"]
        want = np.array([[float(v) for v in row] for row in e["y"]])
        assert np.allclose(r["ref"], want, rtol=1e-13, atol=0)


@pytest.mark.parametrize("impl", IMPLS)
def test_partials_exhaustive_codes_and_zero_points(impl):
    """K = g = 2: every (code, code, zero point) against the definition typed as integers."""
    qa = np.array([[127, -127], [5, -3], [0, 1]], dtype=np.int8)
    codes = np.array([[a, b] for a in range(16) for b in range(16)], dtype=np.uint8)   # N = 256
    for zp in range(16):
        z = np.full((1, 256), zp, dtype=np.uint8)
        if impl == "numpy":
            D = onp.group_partials(qa, codes, z, 2)
        else:
            one = np.full((1, 256), 0x3C00, dtype=np.uint16)
            _, D = cfast.linear(qa, np.full(3, 0x3C00, np.uint16), codes, one, z, 2, want_partials=True)
        for m in range(3):
            for n in range(256):
                a, b = int(codes[n, 0]), int(codes[n, 1])
                assert D[m, 0, n] == (a - zp) * int(qa[m, 0]) + (b - zp) * int(qa[m, 1])


@pytest.mark.parametrize("impl", IMPLS)
def test_extreme_codes_closed_form(impl):
    """Largest partials a group of 128 can hold: codes 15 (or 0) against zero point 0 (or 15) with every
    activation code at +-127 give D = +-15 * 127 * 128 = +-243840 by hand; with unit scales and
    s_a = 1 the output is the sum over groups, bf16-rounded.  The symmetric scheme (z = 8 everywhere)
    with all codes 8 +- 7 gives +-7 * 127 * 128 = +-113792."""
    K, g = 512, 128
    x = np.full((2, K), 127.0)
    x[1] = -127.0                                           # s_a = fp16(127/127) = 1, q_a = +-127
    xb = bits_bf16(x)
    #            group 0      group 1       group 2       group 3
    code = np.array([15, 0, 15, 1], dtype=np.uint8)         # channel 0
    zero = np.array([0, 15, 8, 8], dtype=np.uint8)
    qw = np.repeat(code, g)[None, :].copy()                 # N = 1
    z = zero[:, None].copy()
    one = np.full((4, 1), 0x3C00, dtype=np.uint16)
    if impl == "numpy":
        r = onp.w4a8_linear(xb, qw, one, z, g)
    else:
        r = cfast.w4a8_linear(xb, qw, one, z, g, want_partials=True)
    assert list(r["sa"]) == [0x3C00, 0x3C00]
    want = np.array([243840, -243840, 113792, -113792])
    assert np.array_equal(r["D"][0, :, 0], want) and np.array_equal(r["D"][1, :, 0], -want)
    assert r["ref"][0, 0] == 0.0 and r["ref"][1, 0] == 0.0            # the four groups cancel exactly
    # without the last group: 243840 - 243840 + 113792 = 113792 exactly
    r3 = (onp if impl == "numpy" else cfast).w4a8_linear(xb[:, :384], qw[:, :384], one[:3], z[:3], g)
    assert r3["ref"][0, 0] == 113792.0 and r3["ref"][1, 0] == -113792.0


# ---------------------------------------------- reduction to library routines (dgemm) --
@pytest.mark.parametrize("impl", IMPLS)
@pytest.mark.parametrize("name,M", [("tiny", 16), ("mid", 24)])
def test_equals_dequantise_then_dgemm(impl, name, M):
    case = wl.make_config("tiny") if name == "tiny" else wl.make_layer(640, 384, 7, M)
    g = case["group"]
    r = run_impl(impl, case["x"], case["qw"], case["sw"], case["z"], g)
    sa = onp.fp16_bits_to_f64(r["sa"])
    sw = onp.fp16_bits_to_f64(case["sw"])                       # [G,N]
    wdq = (case["qw"].astype(np.float64) - np.repeat(case["z"].T.astype(np.float64), g, axis=1)) \
        * np.repeat(sw.T, g, axis=1)                            # [N,K] dequantised weights
    want = (r["qa"].astype(np.float64) * sa[:, None]) @ wdq.T   # BLAS dgemm
    scale = np.abs(r["qa"].astype(np.float64) * sa[:, None]) @ np.abs(wdq).T
    assert np.all(np.abs(r["ref"] - want) <= 1e-12 * scale + 1e-300)
    # integer part alone: dgemm on integers below 2^53 is exact
    K = case["K"]
    for gi in range(K // g):
        ks = slice(gi * g, (gi + 1) * g)
        Dg = r["qa"][:, ks].astype(np.float64) @ (case["qw"][:, ks].astype(np.float64)
                                                   - case["z"][gi].astype(np.float64)[:, None]).T
        assert np.array_equal(Dg, r["D"][:, gi, :].astype(np.float64))


@pytest.mark.parametrize("impl", IMPLS)
def test_reduces_to_signed_integer_matmul(impl):
    """sw == 1, z == 8 and a token scale of exactly 1: the path is a plain int8 x int4 matmul."""
    rng = np.random.default_rng(5)
    M, N, K, g = 5, 12, 64, 16
    xi = rng.integers(-126, 127, size=(M, K)).astype(np.float32)
    xi[:, 0] = 127.0                                             # amax = 127 -> s_a = 1 exactly
    qw = rng.integers(0, 16, size=(N, K), dtype=np.uint8)
    z = np.full((K // g, N), 8, np.uint8)
    sw = np.full((K // g, N), 0x3C00, np.uint16)
    r = run_impl(impl, bits_bf16(xi), qw, sw, z, g)
    assert np.array_equal(r["qa"], xi.astype(np.int8))
    assert np.all(r["sa"] == 0x3C00)
    want = xi.astype(np.int64) @ (qw.astype(np.int64) - 8).T
    assert np.array_equal(r["ref"], want.astype(np.float64))
    assert np.array_equal(r["D"].sum(axis=1), want)


# ------------------------------------------------------------------------ invariants ---
@pytest.mark.parametrize("impl", IMPLS)
def test_weight_equal_to_zero_point_contributes_nothing(impl):
    rng = np.random.default_rng(6)
    c = wl.random_codes(rng, 6, 16, 256, 128)
    c["qw"] = np.repeat(c["z"].T, 128, axis=1).astype(np.uint8)         # every code == its zero point
    r = run_impl(impl, c["x"], c["qw"], c["sw"], c["z"], 128)
    assert not r["D"].any() and not r["ref"].any()
    c["qw"][:] = 0
    c["z"][:] = 0
    r = run_impl(impl, c["x"], c["qw"], c["sw"], c["z"], 128)
    assert not r["D"].any() and not r["ref"].any()


@pytest.mark.parametrize("impl", IMPLS)
def test_linear_in_each_scale(impl):
    rng = np.random.default_rng(8)
    c = wl.random_codes(rng, 4, 8, 256, 128)
    base = run_impl(impl, c["x"], c["qw"], c["sw"], c["z"], 128)
    # weight scales times 4: fp16 exponent + 2
    sw4 = (onp.fp16_bits_to_f64(c["sw"]) * 4).astype(np.float16).view(np.uint16)
    r = run_impl(impl, c["x"], c["qw"], sw4, c["z"], 128)
    assert np.array_equal(r["D"], base["D"]) and np.array_equal(r["ref"], base["ref"] * 4)
    # activations times 2^-3: same codes, token scale and output times 2^-3
    x8 = wl.f32_to_bf16_bits(wl.bf16_bits_to_f32(c["x"]) * np.float32(0.125))
    r = run_impl(impl, x8, c["qw"], c["sw"], c["z"], 128)
    assert np.array_equal(r["qa"], base["qa"]) and np.array_equal(r["ref"], base["ref"] * 0.125)
    # one group's scale doubled changes the result by exactly that group's term
    sw2 = onp.fp16_bits_to_f64(c["sw"]).copy()
    sw2[1] *= 2
    r = run_impl(impl, c["x"], c["qw"], sw2.astype(np.float16).view(np.uint16), c["z"], 128)
    sa = onp.fp16_bits_to_f64(base["sa"])
    term = sa[:, None] * onp.fp16_bits_to_f64(c["sw"])[1][None, :] * base["D"][:, 1, :]
    assert np.allclose(r["ref"] - base["ref"], term, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("impl", IMPLS)
def test_permutation_and_independence(impl):
    rng = np.random.default_rng(9)
    c = wl.random_codes(rng, 5, 12, 384, 128)
    base = run_impl(impl, c["x"], c["qw"], c["sw"], c["z"], 128)
    # permute k inside each group, identically for x and qw: same D
    perm = np.concatenate([g * 128 + rng.permutation(128) for g in range(3)])
    r = run_impl(impl, c["x"][:, perm], c["qw"][:, perm], c["sw"], c["z"], 128)
    assert np.array_equal(r["D"], base["D"]) and np.array_equal(r["sa"], base["sa"])
    # permute whole groups (with their scales and zero points): D permuted, sum unchanged up to fp64 order
    gp = np.array([2, 0, 1])
    kperm = np.concatenate([np.arange(g * 128, (g + 1) * 128) for g in gp])
    r = run_impl(impl, c["x"][:, kperm], c["qw"][:, kperm], c["sw"][gp], c["z"][gp], 128)
    assert np.array_equal(r["D"], base["D"][:, gp, :])
    assert np.allclose(r["ref"], base["ref"], rtol=1e-12, atol=1e-12)
    # rows and columns are independent
    r = run_impl(impl, c["x"][2:3], c["qw"][4:9], c["sw"][:, 4:9], c["z"][:, 4:9], 128)
    assert np.array_equal(r["D"], base["D"][2:3, :, 4:9]) and np.array_equal(r["ref"], base["ref"][2:3, 4:9])
    # group sums of the activation codes equal the partials for all-ones codes with zero point 0
    ones = np.ones_like(c["qw"])
    r = run_impl(impl, c["x"], ones, c["sw"], np.zeros_like(c["z"]), 128)
    assert np.array_equal(r["D"], np.repeat(base["asum"][:, :, None], 12, axis=2))


@pytest.mark.parametrize("impl", IMPLS)
def test_a_priori_bound_against_unquantised_activations(impl):
    """|ref - x . w_deq| <= (s_a/2) sum|w_deq| when nothing clamps: pins the quantiser's semantics."""
    c = wl.make_layer(512, 64, 11, 12)
    r = run_impl(impl, c["x"], c["qw"], c["sw"], c["z"], 128)
    x = wl.bf16_bits_to_f32(c["x"]).astype(np.float64)
    sa = onp.fp16_bits_to_f64(r["sa"])
    assert np.all(np.abs(x / sa[:, None]) <= 127.5)                      # no clamp in this draw
    wdq = (c["qw"].astype(np.float64) - np.repeat(c["z"].T.astype(np.float64), 128, axis=1)) \
        * np.repeat(onp.fp16_bits_to_f64(c["sw"]).T, 128, axis=1)
    err = np.abs(r["ref"] - x @ wdq.T)
    bound = 0.5 * sa[:, None] * np.abs(wdq).sum(axis=1)[None, :]
    assert np.all(err <= bound * (1 + 1e-9))
    assert err.max() > 0.01 * bound.max()                                 # the bound is not vacuous
    # and the quantised result tracks the unquantised product
    assert np.corrcoef(r["ref"].ravel(), (x @ wdq.T).ravel())[0, 1] > 0.99


# --------------------------------------------------- the two oracles on bigger shapes --
def test_c_oracle_equals_numpy_oracle_on_tiny_config():
    c = wl.make_config("tiny")
    a = onp.w4a8_linear(c["x"], c["qw"], c["sw"], c["z"], 128)
    b = cfast.w4a8_linear(c["x"], c["qw"], c["sw"], c["z"], 128, want_partials=True)
    for k in ("qa", "sa", "asum", "D"):
        assert np.array_equal(a[k], b[k]), k
    assert np.allclose(a["ref"], b["ref"], rtol=1e-13, atol=0)
    assert len(c["outlier_channels"]) == 3
    # outlier channels dominate the per-token maximum, so ordinary channels use few codes
    assert np.abs(a["qa"]).max() == 127 and np.median(np.abs(a["qa"])) <= 8


def test_c_oracle_equals_numpy_oracle_ragged_shape_and_zero_rows():
    c = wl.make_layer(384, 200, 21, 19)
    xf = wl.bf16_bits_to_f32(c["x"]).copy()
    xf[3] = 0.0
    xf[7] = -0.0
    c["x"] = wl.f32_to_bf16_bits(xf)
    a = onp.w4a8_linear(c["x"], c["qw"], c["sw"], c["z"], 128)
    b = cfast.w4a8_linear(c["x"], c["qw"], c["sw"], c["z"], 128, want_partials=True)
    for k in ("qa", "sa", "asum", "D"):
        assert np.array_equal(a[k], b[k]), k
    assert np.allclose(a["ref"], b["ref"], rtol=1e-13, atol=0)
    assert a["sa"][3] == 0 and not a["qa"][3].any() and not a["ref"][3].any()
    assert not a["ref"][7].any()


def test_empty_inputs():
    q, s, a = onp.quantize_act(np.zeros((0, 256), np.uint16), 128)
    assert q.shape == (0, 256) and s.shape == (0,) and a.shape == (0, 2)
    q, s, a = cfast.quantize_act(np.zeros((0, 256), np.uint16), 128)
    assert q.shape == (0, 256) and s.shape == (0,) and a.shape == (0, 2)


def test_tolerance_band():
    ref = np.array([[1.0, -2.0], [0.0, 4.0]])
    rms = np.sqrt((1 + 4 + 0 + 16) / 4)
    assert np.allclose(onp.tolerance(ref), np.abs(ref) / 128 + 1e-3 * rms)
    y = onp.f64_to_bf16_bits(ref)
    ok, ratio = onp.within_tolerance(y, ref)
    assert ok and ratio == 0.0
    bad = onp.f64_to_bf16_bits(ref * 1.05)
    ok, ratio = onp.within_tolerance(bad, ref)
    assert not ok and ratio > 1


# ---- SiLU(gate) * up and the requantisation that follows (Sec. 3.5, "Kernel Fusion") ----------------
def read_silu_golden():
    rows = []
    import os
    with open(os.path.join(os.path.dirname(__file__), "golden", "silu_mul_examples.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            g, u, prod, h = line.split()
            rows.append((int(g, 16), int(u, 16), float(prod), int(h, 16)))
    return rows


def test_silu_mul_matches_hand_worked_examples():
    rows = read_silu_golden()
    g = np.array([[r[0] for r in rows]], dtype=np.uint16)
    u = np.array([[r[1] for r in rows]], dtype=np.uint16)
    h, h_bits = onp.silu_mul(g, u)
    assert np.allclose(h[0], [r[2] for r in rows], rtol=0, atol=6e-11)
    assert h_bits[0].tolist() == [r[3] for r in rows]


def test_silu_mul_against_library_routines_and_identities():
    import torch
    from scipy.special import expit
    rng = np.random.default_rng(5)
    gb = wl.f32_to_bf16_bits((rng.standard_normal((7, 64)) * 6).astype(np.float32))
    ub = wl.f32_to_bf16_bits((rng.standard_normal((7, 64)) * 3).astype(np.float32))
    g, u = onp.bf16_bits_to_f64(gb), onp.bf16_bits_to_f64(ub)
    h, h_bits = onp.silu_mul(gb, ub)
    # SiLU(v) = v * logistic(v): scipy's logistic function and torch's silu, both in fp64
    assert np.allclose(h, g * expit(g) * u, rtol=1e-14, atol=0)
    assert np.allclose(h, (torch.nn.functional.silu(torch.from_numpy(g)) * torch.from_numpy(u)).numpy(), rtol=1e-14, atol=0)
    # SiLU(v) - SiLU(-v) = v, with up = 1 (bit pattern 0x3F80) and the sign bit of gate flipped
    one = np.full_like(gb, 0x3F80)
    hp, _ = onp.silu_mul(gb, one)
    hm, _ = onp.silu_mul(gb ^ np.uint16(0x8000), one)
    assert np.allclose(hp - hm, g, rtol=1e-14, atol=1e-300)
    # exact linearity in up for powers of two, oddness in up, zero gate -> zero
    h2, _ = onp.silu_mul(gb, wl.f32_to_bf16_bits((onp.bf16_bits_to_f64(ub) * 4.0).astype(np.float32)))
    assert np.array_equal(h2, 4.0 * h)
    hn, hn_bits = onp.silu_mul(gb, ub ^ np.uint16(0x8000))
    assert np.array_equal(hn, -h) and np.array_equal(hn_bits, h_bits ^ np.uint16(0x8000))
    hz, hz_bits = onp.silu_mul(np.zeros_like(gb), ub)
    assert not hz.any() and not (hz_bits & 0x7FFF).any()
    # far out the function is the identity on one side and zero on the other; no overflow to NaN at -90 (exp(90) is finite
    # in fp64) nor at the largest bf16 magnitudes
    big = wl.f32_to_bf16_bits(np.array([[40.0, -40.0, 90.0, -90.0, 3.0e38, -3.0e38]], dtype=np.float32))
    hb, hb_bits = onp.silu_mul(big, np.full_like(big, 0x3F80))
    assert hb[0, 0] == 40.0 and abs(hb[0, 1]) < 1e-15 and hb[0, 2] == 90.0 and abs(hb[0, 3]) < 1e-37
    assert hb[0, 4] == onp.bf16_bits_to_f64(big)[0, 4] and hb[0, 5] == 0.0 and np.all(np.isfinite(hb))
    # the rounding is the pinned bf16 rounding of the fp64 value
    assert np.array_equal(h_bits, onp.f64_to_bf16_bits(h))


def test_silu_mul_quantize_is_the_quantiser_on_h():
    rng = np.random.default_rng(6)
    gb = wl.f32_to_bf16_bits((rng.standard_normal((3, 256)) * 4).astype(np.float32))
    ub = wl.f32_to_bf16_bits((rng.standard_normal((3, 256)) * 2).astype(np.float32))
    gb[1] = 0                                                   # a token whose h is all zero: scale 0, codes 0
    r = onp.silu_mul_quantize(gb, ub, 128)
    h = onp.bf16_bits_to_f64(r["h_bits"])
    sa = onp.fp16_bits_to_f64(r["sa"])
    assert sa[1] == 0.0 and not r["qa"][1].any()
    for m in (0, 2):
        # the a-priori statement of the quantiser: |h - sa q| <= sa / 2 wherever nothing was clamped, and the largest
        # magnitude maps to +-127
        assert np.all(np.abs(h[m] - sa[m] * r["qa"][m]) <= sa[m] / 2 + 1e-12)
        assert np.abs(r["qa"][m]).max() == 127
    assert np.array_equal(r["asum"], r["qa"].astype(np.int64).reshape(3, 2, 128).sum(axis=2))
    # worked example through the golden fixture: the six h values as one token (padded to a group of 8)
    rows = read_silu_golden()
    g8 = np.array([[r_[0] for r_ in rows] + [0, 0]], dtype=np.uint16)
    u8 = np.array([[r_[1] for r_ in rows] + [0, 0]], dtype=np.uint16)
    q = onp.silu_mul_quantize(g8, u8, 8)
    # amax = 2.1875 -> sa = fp16(2.1875 / 127 = 0.017224409...) ; fp16 step in [2^-6, 2^-5) is 2^-16: 1128.82 -> 1129 * 2^-16
    assert onp.fp16_bits_to_f64(q["sa"])[0] == 1129 * 2.0 ** -16
    # codes: h / sa = 126.98, -51.02, -125.16, 0, 18.03, -0.156 -> 127, -51, -125, 0, 18, 0
    assert q["qa"][0].tolist() == [127, -51, -125, 0, 18, 0, 0, 0]
    assert q["asum"][0].tolist() == [127 - 51 - 125 + 18]


# ---- W4A16: the weight-only variant (Sec. 3.4, first paragraph) -------------------------------------
def test_w4a16_worked_example(golden):
    g8 = golden("worked_example_w4a8.txt")
    g16 = golden("worked_example_w4a16.txt")
    group = g8["group"][0]
    x = bits_bf16([g8["x"]])
    qw = np.array([g8["qw_row0"], g8["qw_row1"]], dtype=np.uint8)
    z = np.array([g8["z_row0"], g8["z_row1"]], dtype=np.uint8).T.copy()
    sw = bits_fp16(np.array([g8["sw_row0"], g8["sw_row1"]]).T.copy())
    ref = onp.w4a16_linear(x, qw, sw, z, group)
    assert ref[0].tolist() == g16["ref"]
    assert onp.f64_to_bf16_bits(ref)[0].tolist() == g16["y_bf16_bits"]
    w, w_bits = onp.dequantize_weights(qw, sw, z, group)
    assert w[0].tolist() == g16["w_row0"] and w[1].tolist() == g16["w_row1"]
    assert np.array_equal(onp.bf16_bits_to_f64(w_bits), w)                     # these happen to be bf16 numbers


def test_w4a16_brute_force_on_exact_rationals():
    rng = np.random.default_rng(21)
    for M, N, K, group in ((2, 3, 8, 4), (1, 2, 12, 4), (3, 1, 16, 8)):
        c = wl.random_codes(rng, M, N, K, group)
        ref = onp.w4a16_linear(c["x"], c["qw"], c["sw"], c["z"], group)
        x = [[Fraction(float(v)) for v in row] for row in onp.bf16_bits_to_f64(c["x"])]
        sw = [[Fraction(float(v)) for v in row] for row in onp.fp16_bits_to_f64(c["sw"])]
        for m in range(M):
            for n in range(N):
                y = sum(x[m][k] * sw[k // group][n] * (int(c["qw"][n, k]) - int(c["z"][k // group, n])) for k in range(K))
                assert abs(float(y) - ref[m, n]) <= 1e-13 * max(1.0, abs(float(y)))


def test_w4a16_reduces_to_dgemm_and_meets_w4a8_where_quantisation_is_exact():
    rng = np.random.default_rng(22)
    M, N, K, group = 5, 24, 256, 128
    c = wl.random_codes(rng, M, N, K, group)
    ref = onp.w4a16_linear(c["x"], c["qw"], c["sw"], c["z"], group)
    w, w_bits = onp.dequantize_weights(c["qw"], c["sw"], c["z"], group)
    assert np.allclose(ref, onp.bf16_bits_to_f64(c["x"]) @ w.T, rtol=1e-12, atol=1e-12)            # library dgemm
    # dequantised weights: one exact product per element, and the bf16 rounding is the pinned one
    assert np.array_equal(w_bits, onp.f64_to_bf16_bits(w))
    assert np.abs(onp.bf16_bits_to_f64(w_bits) - w).max() <= 2.0 ** -8 * np.abs(w).max()
    # Activations that the W4A8 quantiser reproduces exactly (integers -127..127 times a power of two, the largest
    # magnitude 127 so that the scale is that power of two): both schemes then compute the same sum.
    q = rng.integers(-127, 128, size=(M, K))
    q[:, 0] = 127
    xq = wl.f32_to_bf16_bits((q * 2.0 ** -5).astype(np.float32))
    r8 = onp.w4a8_linear(xq, c["qw"], c["sw"], c["z"], group)
    assert np.array_equal(r8["qa"], q.astype(np.int8)) and np.all(onp.fp16_bits_to_f64(r8["sa"]) == 2.0 ** -5)
    r16 = onp.w4a16_linear(xq, c["qw"], c["sw"], c["z"], group)
    assert np.allclose(r16, r8["ref"], rtol=1e-13, atol=0)
    # and in general the two differ by no more than the activation quantisation allows: |x - sa qa| <= sa / 2
    r8 = onp.w4a8_linear(c["x"], c["qw"], c["sw"], c["z"], group)
    sa = onp.fp16_bits_to_f64(r8["sa"])
    assert np.all(np.abs(ref - r8["ref"]) <= (sa[:, None] / 2) * np.abs(w).sum(axis=1)[None, :] + 1e-9)
    # linear in x (exactly, for a power of two), columns independent
    x2 = wl.f32_to_bf16_bits((onp.bf16_bits_to_f64(c["x"]) * 4.0).astype(np.float32))
    assert np.array_equal(onp.w4a16_linear(x2, c["qw"], c["sw"], c["z"], group), 4.0 * ref)
    assert np.array_equal(onp.w4a16_linear(c["x"], c["qw"][5:9], c["sw"][:, 5:9], c["z"][:, 5:9], group), ref[:, 5:9])


# ---- projection + residual (Sec. 3.5) ----------------------------------------------------------------
def test_residual_add_worked_example_and_special_cases(golden):
    g = golden("worked_example_w4a8.txt")
    group = g["group"][0]
    x = bits_bf16([g["x"]])
    qw = np.array([g["qw_row0"], g["qw_row1"]], dtype=np.uint8)
    z = np.array([g["z_row0"], g["z_row1"]], dtype=np.uint8).T.copy()
    sw = bits_fp16(np.array([g["sw_row0"], g["sw_row1"]]).T.copy())
    # by hand: -9.8419189453125 + 10 = 0.1580810546875 ; 1.1042633056640625 + (-1.125) = -0.0207366943359375
    r = onp.w4a8_linear_residual(x, qw, sw, z, group, bits_bf16([[10.0, -1.125]]))
    assert r["lin"][0].tolist() == g["ref"]
    assert r["ref"][0].tolist() == [0.1580810546875, -0.0207366943359375]
    # rounded once: 0.15808... = 1.2646484375 * 2^-3 -> mantissa 0.2646484375 * 128 = 33.875 -> 34 -> 0x3E22;
    # 0.02073669... = 1.3271484375 * 2^-6 -> 41.875 -> 42 -> 0xBCAA   (rounding the projection first would give
    # bf16(-9.8125 + 10) = 0.1875 = 0x3E40: the two orders differ, and the definition is the single rounding)
    assert onp.f64_to_bf16_bits(r["ref"])[0].tolist() == [0x3E22, 0xBCAA]
    # zero residual: the projection; codes equal to zero points: the residual itself, bit for bit
    rng = np.random.default_rng(31)
    c = wl.random_codes(rng, 3, 8, 256)
    rb = wl.f32_to_bf16_bits(rng.standard_normal((3, 8)).astype(np.float32))
    r0 = onp.w4a8_linear_residual(c["x"], c["qw"], c["sw"], c["z"], 128, np.zeros((3, 8), dtype=np.uint16))
    assert np.array_equal(r0["ref"], onp.w4a8_linear(c["x"], c["qw"], c["sw"], c["z"], 128)["ref"])
    qz = np.repeat(c["z"].T, 128, axis=1).astype(np.uint8)
    rz = onp.w4a8_linear_residual(c["x"], qz, c["sw"], c["z"], 128, rb)
    assert np.array_equal(onp.f64_to_bf16_bits(rz["ref"]), rb)
    # the band never falls below the projection's own
    rr = onp.w4a8_linear_residual(c["x"], c["qw"], c["sw"], c["z"], 128, rb)
    assert np.all(onp.residual_tolerance(rr["lin"], rr["ref"]) >= onp.tolerance(rr["lin"]))
