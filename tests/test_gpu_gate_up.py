"""GPU parity of the step after the fused gate+up projection (Sec. 3.5, "Kernel Fusion"): h = bf16(SiLU(gate) * up)
and the activation quantisation of h for the down projection, alone (w4a8_silu_mul_quantize) and fused into the
projection (w4a8_gate_up_silu_quantize: one kernel with a grid-wide barrier where the strip kernel runs).

What is compared with what:
  * h against the oracle's h computed from the SAME bf16 gate/up values: the kernel evaluates SiLU in fp32 with the fast
    exponential, the oracle in fp64, so a rounded h may be the oracle's bf16 neighbour (never further), and only rarely;
  * codes, token scales and group sums against the oracle's quantiser applied to the kernel's h: bit-exact (a
    floating-point value that decides an integer is taken in the same precision on both sides);
  * the whole chain against the oracle's chain on the unfused gate and up matrices, within a band derived from the
    linear layer's tolerance (below), which also pins the channel order of the fused layer;
  * the one-kernel form against the two-kernel form: identical bits.
"""
import numpy as np
import pytest
import torch

from oracle import cfast
from oracle import w4a8_oracle as onp
from paper_2608_12932_b200 import binding as B
from paper_2608_12932_b200 import workload as wl
from tests.gpu_util import bits, t_u16

pytestmark = pytest.mark.gpu


def ordered(b):
    """bf16 bit patterns -> integers that order like the values (neighbouring values differ by 1; +0 and -0 coincide)."""
    b = b.astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)


def check_h(h_gpu_bits, gate_bits, up_bits):
    _, h_ref_bits = onp.silu_mul(gate_bits, up_bits)
    d = np.abs(ordered(h_gpu_bits) - ordered(h_ref_bits))
    # far out on the negative side (gate below -87, where e^-gate leaves fp32) the kernel returns a signed zero for
    # values whose magnitude is below 1e-30: not a matter of bf16 steps
    tiny = np.abs(onp.bf16_bits_to_f64(h_gpu_bits) - onp.bf16_bits_to_f64(h_ref_bits)) <= 1e-30
    d = np.where(tiny, 0, d)
    assert d.max(initial=0) <= 1, f"h is {d.max()} bf16 steps from the oracle's"
    assert np.count_nonzero(d) <= 0.01 * d.size + 2, f"{np.count_nonzero(d)} of {d.size} h values differ"


def check_codes(h_gpu_bits, qa_h, sa_h, asum_h, group=128):
    qa, sa, asum = onp.quantize_act(h_gpu_bits, group)
    assert np.array_equal(qa_h.cpu().numpy(), qa)
    assert np.array_equal(bits(sa_h), sa)
    assert np.array_equal(asum_h.cpu().numpy(), asum)


def split_fused(y_bits, I):
    """Columns of a fused-layout [M, 2 I] array back to (gate [M,I], up [M,I])."""
    order = B.gate_up_row_order(I)
    cat = np.empty_like(y_bits)
    cat[:, order] = y_bits
    return cat[:, :I], cat[:, I:]


@pytest.mark.parametrize("M,I", [(1, 128), (5, 384), (8, 4096), (16, 12288), (70, 1024), (130, 256), (600, 4096), (3, 12416)])
def test_silu_mul_quantize_alone(M, I):
    rng = np.random.default_rng(100 + M)
    gate = wl.f32_to_bf16_bits((rng.standard_normal((M, I)) * 3).astype(np.float32))
    up = wl.f32_to_bf16_bits((rng.standard_normal((M, I)) * 2).astype(np.float32))
    if M >= 3:
        gate[1] = 0                                            # h = 0 for a whole token: scale 0, codes 0
        gate[2, :8] = wl.f32_to_bf16_bits(np.array([-200, -95, -88, -87, 60, 200, 1e30, -1e30], dtype=np.float32))
    order = B.gate_up_row_order(I)
    y = np.concatenate([gate, up], axis=1)[:, order]
    h, qa_h, sa_h, asum_h = B.w4a8_silu_mul_quantize(t_u16(y, torch.bfloat16))
    torch.cuda.synchronize()
    hb = bits(h)
    check_h(hb, gate, up)
    check_codes(hb, qa_h, sa_h, asum_h)
    if M >= 3:
        assert not (hb[1] & 0x7FFF).any() and not qa_h[1].any().item()


def fused_layer(K, I, seed, M):
    """Separate gate and up matrices (the first and second I rows of one synthetic layer), and the same layer with its
    rows in the fused order, packed."""
    c = wl.make_layer(K, 2 * I, seed, M)
    order = B.gate_up_row_order(I)
    qw = torch.from_numpy(np.ascontiguousarray(c["qw"][order])).cuda()
    sw = t_u16(np.ascontiguousarray(c["sw"][:, order]), torch.float16)
    z = torch.from_numpy(np.ascontiguousarray(c["z"][:, order])).cuda()
    return c, B.w4a8_pack_weights(qw, sw, z)


def chain_band(ref, I):
    """Band for h of the whole chain.  The linear layer's outputs may be off by e(v) = 2^-7 |v| + 1e-3 rms(y) each;
    |SiLU'| <= 1.1 and |SiLU(g)| <= |g|, so |dh| <= 1.1 |u| e(g) + (|g| + e(g)) e(u), plus the final bf16 rounding and
    the one-step freedom of h (2^-7 |h| together)."""
    rms = float(np.sqrt(np.mean(ref * ref)))
    g, u = onp.bf16_bits_to_f64(onp.f64_to_bf16_bits(ref[:, :I])), onp.bf16_bits_to_f64(onp.f64_to_bf16_bits(ref[:, I:]))
    eg, eu = 2.0 ** -7 * np.abs(g) + 1e-3 * rms, 2.0 ** -7 * np.abs(u) + 1e-3 * rms
    h, _ = onp.silu_mul(onp.f64_to_bf16_bits(ref[:, :I]), onp.f64_to_bf16_bits(ref[:, I:]))
    return h, 1.1 * np.abs(u) * eg + (np.abs(g) + eg) * eu + 2.0 ** -7 * np.abs(h) + 1e-6


SHAPES = [(1, 256, 128), (4, 512, 256), (8, 1024, 384), (8, 4096, 12288), (3, 384, 1152), (13, 4096, 12288), (16, 512, 2432),
          (8, 12288, 256), (24, 1024, 384), (40, 512, 1024), (200, 256, 256)]


@pytest.mark.parametrize("M,K,I", SHAPES)
def test_gate_up_forms_against_oracle_and_one_another(M, K, I):
    N = 2 * I
    c, packed = fused_layer(K, I, 900 + M, M)
    ws = B.new_workspace(max(M, 16), N, K)
    x = t_u16(c["x"], torch.bfloat16)
    qa, sa, asum = B.w4a8_quantize_act(x)
    auto = B.w4a8_gate_up_form(M, N, K)
    strip = B.w4a8_plan(M, N, K)["family"] == B.PATH_STRIP
    assert auto == (B.GATE_UP_EPILOGUE if strip else B.GATE_UP_SEPARATE)
    forms = [B.GATE_UP_AUTO, B.GATE_UP_SEPARATE] + ([B.GATE_UP_EPILOGUE, B.GATE_UP_ONE_KERNEL] if M <= 16 else [])
    # Forms that multiply in the same GEMM kernel must agree bit for bit: the two epilogue forms always run the strip
    # kernel, AUTO and SEPARATE run whatever w4a8_gemm takes for the shape.
    groups = {}
    for form in forms:
        in_strip = form in (B.GATE_UP_EPILOGUE, B.GATE_UP_ONE_KERNEL) or strip
        for rep in range(3):                                   # the workspace words must come back to zero each time
            h, qa_h, sa_h, asum_h = B.w4a8_gate_up_silu_quantize(qa, sa, asum, packed, N, ws, form=form)
            torch.cuda.synchronize()
            B.w4a8_check_status(ws)
            groups.setdefault(in_strip, []).append((form, bits(h), qa_h.cpu().numpy(), bits(sa_h), asum_h.cpu().numpy()))
    ref = cfast.w4a8_linear(c["x"], c["qw"], c["sw"], c["z"], 128)["ref"]      # unfused matrices: rows 0..I-1 gate, I..2I-1 up
    h_ref, band = chain_band(ref, I)
    for in_strip, outs in groups.items():
        first = outs[0]
        for o in outs[1:]:
            assert all(np.array_equal(a, b) for a, b in zip(o[1:], first[1:])), f"forms {first[0]} and {o[0]} differ"
        hb, qa_hb, sa_hb, asum_hb = first[1:]
        # the projection by itself in the same kernel family, and the step applied to its output: the same bits
        y = B.w4a8_gemm(qa, sa, asum, packed, N, ws, path=B.PATH_STRIP if in_strip else B.PATH_AUTO)
        B.w4a8_check_status(ws)
        h2, qa2, sa2, asum2 = B.w4a8_silu_mul_quantize(y)
        torch.cuda.synchronize()
        assert np.array_equal(bits(h2), hb) and np.array_equal(qa2.cpu().numpy(), qa_hb)
        assert np.array_equal(bits(sa2), sa_hb) and np.array_equal(asum2.cpu().numpy(), asum_hb)
        # h against the oracle on the kernel's own y; codes against the oracle's quantiser on the kernel's h
        gate_b, up_b = split_fused(bits(y), I)
        check_h(hb, gate_b, up_b)
        qa_o, sa_o, asum_o = onp.quantize_act(hb, 128)
        assert np.array_equal(qa_hb, qa_o) and np.array_equal(sa_hb, sa_o) and np.array_equal(asum_hb, asum_o)
        # the whole chain against the oracle's chain
        err = np.abs(onp.bf16_bits_to_f64(hb) - h_ref)
        assert np.all(err <= band), f"worst err/band {float((err / band).max()):.3f}"
        # and the down projection's operands work as such: the scale reproduces h within half a step
        sa_f = onp.fp16_bits_to_f64(sa_hb)
        assert np.all(np.abs(onp.bf16_bits_to_f64(hb) - sa_f[:, None] * qa_hb) <= sa_f[:, None] / 2 + 1e-12)


def test_form_chosen_for_the_layer_shapes():
    assert B.w4a8_gate_up_form(8, 24576, 4096) == B.GATE_UP_EPILOGUE
    assert B.w4a8_gate_up_form(16, 24576, 4096) == B.GATE_UP_EPILOGUE
    assert B.w4a8_gate_up_form(64, 24576, 4096) == B.GATE_UP_SEPARATE
    assert B.w4a8_gate_up_form(8, 24576 + 128, 4096) == 0               # I not a multiple of 128


def test_separate_form_needs_its_scratch_and_shapes_are_checked():
    M, K, I = 64, 256, 256
    c, packed = fused_layer(K, I, 5, M)
    ws = B.new_workspace(M, 2 * I, K)
    qa, sa, asum = B.w4a8_quantize_act(t_u16(c["x"], torch.bfloat16))
    h = torch.empty((M, I), dtype=torch.bfloat16, device="cuda")
    qa_h = torch.empty((M, I), dtype=torch.int8, device="cuda")
    sa_h = torch.empty((M,), dtype=torch.float16, device="cuda")
    asum_h = torch.empty((M, I // 128), dtype=torch.int32, device="cuda")
    L = B.lib()
    args = [B.GATE_UP_AUTO, B._ptr(qa), B._ptr(sa), B._ptr(asum), B._ptr(packed), M, 2 * I, K, 128, B._ptr(h), B._ptr(qa_h),
            B._ptr(sa_h), B._ptr(asum_h), None, B._ptr(ws), ws.numel(), None]
    assert L.w4a8_gate_up_silu_quantize(*args) == B.ERR_NULL
    args[0] = B.GATE_UP_ONE_KERNEL                              # no strip kernel at 64 tokens
    assert L.w4a8_gate_up_silu_quantize(*args) == B.ERR_SHAPE
    args[0] = 7
    assert L.w4a8_gate_up_silu_quantize(*args) == B.ERR_SHAPE
    args[0] = B.GATE_UP_AUTO
    args[6] = 2 * I + 128                                       # N / 2 not a multiple of 128
    assert L.w4a8_gate_up_silu_quantize(*args) == B.ERR_SHAPE
    torch.cuda.synchronize()
