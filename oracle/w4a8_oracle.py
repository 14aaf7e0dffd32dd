"""numpy statement of the W4A8 linear (Sec. 3.4): test infrastructure only.

Integer stages in int64 (exact), scaling in fp64, one group at a time in the
order the definition is written; no blocking, fusion or reordering.  Consumes
the UNPACKED codes ``qw[N,K]`` - the packed device layout is unknown here.

Notation: M tokens, K in-features, N out-features, group size g, G = K/g.
  x   [M,K]  bf16, passed as uint16 bit patterns
  qa  [M,K]  int8      sa [M] fp16 bit patterns     asum [M,G] int32
  qw  [N,K]  uint8 codes 0..15    sw [G,N] fp16 bit patterns    z [G,N] uint8 0..15
  D   [M,G,N] int32    ref [M,N] fp64
"""
import numpy as np

FP16_MAX = 65504.0


# ---- storage formats (bit patterns <-> fp64), no arithmetic of the method -------------
def bf16_bits_to_f64(bits):
    bits = np.asarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def fp16_bits_to_f64(bits):
    return np.asarray(bits, dtype=np.uint16).view(np.float16).astype(np.float64)


def f64_to_fp16_bits(v):
    return np.asarray(v, dtype=np.float64).astype(np.float16).view(np.uint16)


def f64_to_bf16_bits(v):
    """fp64 -> bf16 bit pattern, round to nearest even (reporting only; finite inputs).

    fp64 -> fp32 first would double-round, so the rounding is done on the fp64
    value directly: scale to the bf16 ulp of its binade and use rint.
    """
    v = np.asarray(v, dtype=np.float64)
    out = np.zeros(v.shape, dtype=np.uint16)
    nz = v != 0
    a = np.abs(v[nz])
    e = np.floor(np.log2(a))
    e = np.where(np.ldexp(1.0, e.astype(np.int64)) > a, e - 1, e)          # guard log2 rounding
    e = np.where(np.ldexp(1.0, (e + 1).astype(np.int64)) <= a, e + 1, e)
    ulp = np.ldexp(1.0, (e - 7).astype(np.int64))
    r = np.rint(a / ulp) * ulp                                              # exact: power-of-two scaling
    r32 = r.astype(np.float32)                                              # r has <= 8 significant bits
    b = (r32.view(np.uint32) >> np.uint32(16)).astype(np.uint16)
    b = b | (np.signbit(v[nz]).astype(np.uint16) << np.uint16(15))
    out[nz] = b
    out[~nz] = np.signbit(v[~nz]).astype(np.uint16) << np.uint16(15)
    return out


# ---- O1: per-token activation quantisation --------------------------------------------
def quantize_act(x_bits, group):
    """bf16 activations -> (qa int8 [M,K], sa fp16 bits [M], asum int32 [M,G]).

    s_a = fp16_rne(amax/127) (saturating at 65504); q_a = clamp(rne(x/s_a), +-127);
    a row whose scale is 0 quantises to all zeros.  Quotients are fp64 divisions:
    a bf16 value over an fp16 value is never closer than 2^-12 to a half-integer
    unless it is exactly one, so fp64 rounding cannot change the integer.
    """
    x = bf16_bits_to_f64(x_bits)
    M, K = x.shape
    assert K % group == 0
    amax = np.max(np.abs(x), axis=1) if K else np.zeros(M)
    sa_bits = f64_to_fp16_bits(np.minimum(amax / 127.0, FP16_MAX))
    sa = fp16_bits_to_f64(sa_bits)
    qa = np.zeros((M, K), dtype=np.int8)
    for m in range(M):
        if sa[m] != 0.0:
            qa[m] = np.clip(np.rint(x[m] / sa[m]), -127, 127).astype(np.int8)
    asum = qa.astype(np.int64).reshape(M, K // group, group).sum(axis=2).astype(np.int32)
    return qa, sa_bits, asum


# ---- O2: per-group integer partials ---------------------------------------------------
def group_partials(qa, qw, z, group):
    """D[m,g,n] = sum_{k in g} qw[n,k] qa[m,k] - z[g,n] sum_{k in g} qa[m,k]   (int32, exact)."""
    qa = np.asarray(qa).astype(np.int64)
    qw = np.asarray(qw).astype(np.int64)
    z = np.asarray(z).astype(np.int64)
    M, K = qa.shape
    N = qw.shape[0]
    G = K // group
    D = np.empty((M, G, N), dtype=np.int64)
    for g in range(G):
        ks = slice(g * group, (g + 1) * group)
        P = qa[:, ks] @ qw[:, ks].T                      # [M,N] int64, no BLAS involved
        A = qa[:, ks].sum(axis=1)                        # [M]
        D[:, g, :] = P - A[:, None] * z[g][None, :]
    assert np.abs(D).max(initial=0) <= group * 15 * 127
    return D.astype(np.int32)


# ---- O3: scales ----------------------------------------------------------------------
def scale_partials(D, sa_bits, sw_bits):
    """ref[m,n] = s_a[m] * sum_g s_w[g,n] * D[m,g,n] in fp64, g ascending."""
    sa = fp16_bits_to_f64(sa_bits)
    sw = fp16_bits_to_f64(sw_bits)
    M, G, N = D.shape
    acc = np.zeros((M, N), dtype=np.float64)
    for g in range(G):
        acc += sw[g][None, :] * D[:, g, :].astype(np.float64)
    return sa[:, None] * acc


def w4a8_linear(x_bits, qw, sw_bits, z, group):
    """The whole path.  Returns dict(qa, sa, asum, D, ref)."""
    qa, sa_bits, asum = quantize_act(x_bits, group)
    D = group_partials(qa, qw, z, group)
    ref = scale_partials(D, sa_bits, sw_bits)
    return dict(qa=qa, sa=sa_bits, asum=asum, D=D, ref=ref)


# ---- a projection whose output is added to the residual stream (Sec. 3.5, "Kernel Fusion") ----
def w4a8_linear_residual(x_bits, qw, sw_bits, z, group, residual_bits):
    """ref[m,n] = s_a[m] sum_g s_w[g,n] D[m,g,n] + r[m,n]: the O and down projections of a decoder layer feed
    the residual stream, and Sec. 3.5 merges such element-wise steps into their neighbours.  r is bf16 (bit
    patterns); the sum is formed in fp64 and rounded once by whoever stores it.  Returns dict(lin, ref): the
    projection alone and the sum (a kernel's band is taken on `lin`, see residual_tolerance)."""
    lin = w4a8_linear(x_bits, qw, sw_bits, z, group)["ref"]
    return dict(lin=lin, ref=lin + bf16_bits_to_f64(residual_bits))


def residual_tolerance(lin, ref):
    """Band for a kernel that adds the residual before its one rounding: the projection's own band (its error does
    not shrink when the sum cancels) plus half a bf16 step of the sum."""
    return tolerance(lin) + 2.0 ** -8 * np.abs(ref)


# ---- the step after the fused gate+up projection (Sec. 3.5, "Kernel Fusion") -----------------
def silu_mul(y_gate_bits, y_up_bits):
    """h[m,c] = bf16_rne( SiLU(gate[m,c]) * up[m,c] ),  SiLU(v) = v / (1 + exp(-v)),  in fp64.

    gate and up are the two halves of the fused gate+up projection's bf16 output (Sec. 3.5 fuses
    the two projections into one GEMM and merges the element-wise operations that follow), given
    here as two separate [M,I] arrays of bf16 bit patterns: how a kernel lays the two halves out
    in one buffer is not this function's business.  Returns (h fp64 before the rounding, h bf16 bits).
    """
    g = bf16_bits_to_f64(y_gate_bits)
    u = bf16_bits_to_f64(y_up_bits)
    with np.errstate(over="ignore"):
        h = g / (1.0 + np.exp(-g)) * u
    return h, f64_to_bf16_bits(h)


def silu_mul_quantize(y_gate_bits, y_up_bits, group):
    """The down projection's quantised input from the gate+up projection's output:
    quantize_act(silu_mul(gate, up)).  Returns dict(h, h_bits, qa, sa, asum)."""
    h, h_bits = silu_mul(y_gate_bits, y_up_bits)
    qa, sa_bits, asum = quantize_act(h_bits, group)
    return dict(h=h, h_bits=h_bits, qa=qa, sa=sa_bits, asum=asum)


# ---- the weight-only variant the paper argues against (Sec. 3.4, first paragraph) ------------------
def dequantize_weights(qw, sw_bits, z, group):
    """w[n,k] = s_w[g(k),n] * (q_w[n,k] - z[g(k),n]) in fp64 (exact: an 11-bit by a 5-bit factor), and its bf16 rounding.
    Returns (w fp64 [N,K], bf16 bits [N,K])."""
    qw = np.asarray(qw).astype(np.int64)
    N, K = qw.shape
    sw = fp16_bits_to_f64(sw_bits)
    zz = np.asarray(z).astype(np.int64)
    w = np.empty((N, K), dtype=np.float64)
    for g in range(K // group):
        ks = slice(g * group, (g + 1) * group)
        w[:, ks] = sw[g][:, None] * (qw[:, ks] - zz[g][:, None]).astype(np.float64)
    return w, f64_to_bf16_bits(w)


def w4a16_linear(x_bits, qw, sw_bits, z, group):
    """W4A16: the same 4-bit weights against UNQUANTISED bf16 activations (the AWQ-style weight-only scheme the
    paper contrasts W4A8 with: it shrinks the weights, which helps the memory-bound decode, and leaves the
    multiplications in 16-bit floating point).  ref[m,n] = sum_g s_w[g,n] * sum_{k in g} x[m,k] (q_w[n,k] - z[g,n])
    in fp64, group by group.  Returns ref [M,N] fp64; a kernel's bf16 result is judged with the band below."""
    x = bf16_bits_to_f64(x_bits)
    qw = np.asarray(qw).astype(np.int64)
    zz = np.asarray(z).astype(np.int64)
    sw = fp16_bits_to_f64(sw_bits)
    M, K = x.shape
    N = qw.shape[0]
    ref = np.zeros((M, N), dtype=np.float64)
    for g in range(K // group):
        ks = slice(g * group, (g + 1) * group)
        P = x[:, ks] @ (qw[:, ks] - zz[g][:, None]).astype(np.float64).T          # [M,N]
        ref += sw[g][None, :] * P
    return ref


# ---- acceptance band for a bf16 result ------------------------------------------------
def tolerance(ref):
    """Per-element bound 2^-7 |ref| + 1e-3 rms(ref), rms over the whole [M,N] result."""
    ref = np.asarray(ref, dtype=np.float64)
    rms = float(np.sqrt(np.mean(ref * ref))) if ref.size else 0.0
    return np.abs(ref) * 2.0 ** -7 + 1e-3 * rms


def within_tolerance(y_bits, ref, rms_ref=None):
    """(ok, worst ratio |y-ref|/bound).  rms_ref overrides the rms when ref is a sample."""
    ref = np.asarray(ref, dtype=np.float64)
    y = bf16_bits_to_f64(y_bits)
    if rms_ref is None:
        bound = tolerance(ref)
    else:
        bound = np.abs(ref) * 2.0 ** -7 + 1e-3 * rms_ref
    err = np.abs(y - ref)
    ok = bool(np.all(err <= bound))
    with np.errstate(divide="ignore", invalid="ignore"):
        ratio = np.where(bound > 0, err / bound, np.where(err > 0, np.inf, 0.0))
    return ok, float(ratio.max(initial=0.0))
