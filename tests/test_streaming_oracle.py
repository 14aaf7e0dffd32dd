"""Pins for the streaming-prefill oracle (rotary embedding of cached pre-rotation keys at shifted positions, streaming
attention mask): a hand-worked example, identities that the rotation must satisfy, and the mask's defining properties."""
import numpy as np

from oracle import streaming as so
from oracle import w4a8_oracle as onp
from paper_2608_12932_b200 import workload as wl


def test_rope_hand_worked_example(golden):
    g = golden("rope_examples.txt")
    D = g["D"][0]
    k = wl.f32_to_bf16_bits(np.array(g["k"], dtype=np.float32)).reshape(1, 1, D)
    out, bits = so.rope_shifted_keys(k, np.array(g["pos"]), g["delta"][0], float(g["base"][0]))
    assert np.allclose(out[0, 0], g["out"], rtol=0, atol=6e-11)
    assert bits[0, 0].tolist() == g["out_bits"]


def test_rope_identities():
    rng = np.random.default_rng(41)
    T, H, D, base = 9, 3, 128, 1.0e6
    k = wl.f32_to_bf16_bits(rng.standard_normal((T, H, D)).astype(np.float32))
    kf = onp.bf16_bits_to_f64(k)
    pos = rng.integers(0, 5000, size=T)
    out, bits = so.rope_shifted_keys(k, pos, 7, base)
    # a rotation of every (i, i + D/2) pair: norms of pairs are kept
    half = D // 2
    assert np.allclose(out[:, :, :half] ** 2 + out[:, :, half:] ** 2, kf[:, :, :half] ** 2 + kf[:, :, half:] ** 2, rtol=1e-12)
    # position 0 is the identity, and only pos - delta matters
    same, same_bits = so.rope_shifted_keys(k, np.full(T, 11), 11, base)
    assert np.array_equal(same, kf) and np.array_equal(same_bits, k)
    again, _ = so.rope_shifted_keys(k, pos + 100, 107, base)
    assert np.array_equal(again, out)
    # the defining property of a rotary embedding: <R(p) q, R(p') k> depends on p - p' only
    q = wl.f32_to_bf16_bits(rng.standard_normal((T, H, D)).astype(np.float32))
    d1 = np.einsum("thd,thd->th", so.rope_shifted_keys(q, pos, 0, base)[0], so.rope_shifted_keys(k, pos - 3, 0, base)[0])
    d2 = np.einsum("thd,thd->th", so.rope_shifted_keys(q, pos + 50, 0, base)[0], so.rope_shifted_keys(k, pos + 47, 0, base)[0])
    assert np.allclose(d1, d2, rtol=1e-9, atol=1e-9)
    # against complex multiplication, the textbook form: (a + i b) e^{i phi}
    theta = base ** (-2.0 * np.arange(half) / D)
    zc = (kf[:, :, :half] + 1j * kf[:, :, half:]) * np.exp(1j * (pos - 7)[:, None, None] * theta[None, None, :])
    assert np.allclose(out[:, :, :half], zc.real, rtol=1e-12, atol=1e-12) and np.allclose(out[:, :, half:], zc.imag, rtol=1e-12, atol=1e-12)
    assert np.array_equal(bits, onp.f64_to_bf16_bits(out))


def test_streaming_mask_properties():
    V, F, n = 3, 4, 5
    m = so.streaming_mask(V, F, n)
    assert m.shape == (V * n, V * F * n)
    for v in range(V):
        for i in range(n):
            q = v * n + i
            p = (v * F + F - 1) * n + i                      # the query's own place in the view-major sequence
            assert m[q, p] == 1                               # a token sees itself
            assert m[q, : p + 1].all() and not m[q, p + 1:].any()      # causal: everything up to itself, nothing after
            # every frame of every earlier view is visible, no token of a later view is
            assert m[q, : v * F * n].all() and not m[q, (v + 1) * F * n:].any()
    # rows are nested: a later query sees at least what an earlier one sees
    assert np.all(m[1:] >= m[:-1])
    # one view, one frame: the plain causal mask
    assert np.array_equal(so.streaming_mask(1, 1, 6), np.tril(np.ones((6, 6), dtype=np.uint8)))
