"""Seeded synthetic inputs for the W4A8 linear: shapes, distributions, storage casts.

This module only MAKES inputs (for the CUDA library and for the CPU checker
alike); it contains none of the arithmetic of the path itself.  The inputs stand
in for the activations and ParoQuant-quantised weights of the paper's VLM
backbone (Sec. 3.4), which are not available: shapes are those of an 8B-class
decoder layer with fused QKV and fused gate+up projections (Sec. 3.5, "Kernel
Fusion"), M = 8 is one speculative draft block (Sec. 3.2) and M = 1024 a
streaming-prefill chunk of new-frame tokens (Sec. 3.1).

Recipe (draw order fixed: weights, outlier channels, activations):
  W   = 0.02 * standard_normal((N, K), float32)       -> asymmetric uint4, group 128
  idx = choice(K, max(1, round(0.01 K)), replace=False)   outlier channels, same for all tokens
  X   = standard_normal((M, K), float32); X[:, idx] *= 20 -> bf16 (round to nearest even)
"""
import numpy as np

GROUP = 128

# (K, N) of the four linear layers of one 8B-class decoder layer
LAYERS = {
    "qkv": (4096, 6144),        # 32 query heads + 2 x 8 KV heads, head dim 128
    "o": (4096, 4096),
    "gate_up": (4096, 24576),   # fused gate + up, intermediate 12288
    "down": (12288, 4096),
}
LAYER_SEEDS = {"qkv": 0, "o": 1, "gate_up": 2, "down": 3}
SWEEP_M = (1, 4, 8, 16, 64, 256, 1024, 4096)

CONFIGS = {
    "tiny": dict(M=16, K=256, N=256, seed=0),                  # checker runs it in well under a second
    "spec_verify": dict(M=8, K=4096, N=6144, seed=0),          # memory-bound, HBM GB/s
    "prefill_gate_up": dict(M=1024, K=4096, N=24576, seed=0),  # compute-bound, INT8 TOPS
    "prefill_down": dict(M=1024, K=12288, N=4096, seed=0),     # long K, 96 groups
}


def f32_to_bf16_bits(x):
    """float32 array -> bf16 bit patterns (uint16), round to nearest even; finite inputs."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits):
    return (np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def quantize_weights_uint4(W, group=GROUP):
    """Synthetic-weight quantiser: fp32 [N,K] -> (qw uint8 [N,K] in 0..15, sw fp16 bits [G,N], z uint8 [G,N]).

    Per (output channel, group): lo = min(w, 0), hi = max(w, 0); sw = fp16((hi - lo)/15);
    a zero range gets sw = 1, z = 0; z = clamp(rne(-lo/sw), 0, 15);
    qw = clamp(rne(w/sw) + z, 0, 15).  Stands in for the paper's offline quantiser.
    """
    W = np.ascontiguousarray(W, dtype=np.float32)
    N, K = W.shape
    assert K % group == 0
    G = K // group
    Wg = W.reshape(N, G, group)
    lo = np.minimum(Wg.min(axis=2), np.float32(0))
    hi = np.maximum(Wg.max(axis=2), np.float32(0))
    sw16 = ((hi - lo) / np.float32(15)).astype(np.float16)
    flat = sw16 == 0
    sw16 = np.where(flat, np.float16(1), sw16)
    sw = sw16.astype(np.float32)
    z = np.clip(np.rint(-lo / sw), 0, 15)
    z = np.where(flat, 0, z).astype(np.float32)
    q = np.clip(np.rint(Wg / sw[:, :, None]) + z[:, :, None], 0, 15).astype(np.uint8)
    return (q.reshape(N, K),
            np.ascontiguousarray(sw16.T).view(np.uint16),
            np.ascontiguousarray(z.T).astype(np.uint8))


def make_layer(K, N, seed, M, group=GROUP):
    """One synthetic layer: dict(qw, sw, z, x) with x = bf16 bits [M,K]; M may be 0."""
    rng = np.random.default_rng(seed)
    W = np.float32(0.02) * rng.standard_normal((N, K), dtype=np.float32)
    qw, sw, z = quantize_weights_uint4(W, group)
    del W
    idx = rng.choice(K, max(1, int(round(0.01 * K))), replace=False)
    X = rng.standard_normal((M, K), dtype=np.float32)
    X[:, idx] *= np.float32(20)
    return dict(qw=qw, sw=sw, z=z, x=f32_to_bf16_bits(X), outlier_channels=np.sort(idx),
                M=M, N=N, K=K, group=group, seed=seed)


def make_config(name):
    c = CONFIGS[name]
    return make_layer(c["K"], c["N"], c["seed"], c["M"])


def make_sweep_layer(layer, m_max=max(SWEEP_M)):
    """A decoder layer's linear for the M sweep: m_max rows drawn once; smaller M use the first M rows."""
    K, N = LAYERS[layer]
    return make_layer(K, N, LAYER_SEEDS[layer], m_max)


def random_codes(rng, M, N, K, group=GROUP):
    """Uniform random codes/zeros/scales/activations for layout and edge-case tests."""
    G = K // group
    qw = rng.integers(0, 16, size=(N, K), dtype=np.uint8)
    z = rng.integers(0, 16, size=(G, N), dtype=np.uint8)
    sw = rng.uniform(1e-3, 2e-2, size=(G, N)).astype(np.float16).view(np.uint16)
    x = f32_to_bf16_bits(rng.standard_normal((M, K), dtype=np.float32))
    return dict(qw=qw, sw=sw, z=z, x=x, M=M, N=N, K=K, group=group)


def algorithmic_bytes_gemm(M, N, K, group=GROUP):
    """Bytes one GEMM call must move: nibbles + scales/zeros + int8 acts + token scales/sums + bf16 out."""
    G = K // group
    return N * K // 2 + (G * N * 5) // 2 + M * K + 2 * M + 4 * M * G + 2 * M * N


def algorithmic_bytes_quantize(M, K, group=GROUP):
    G = K // group
    return 2 * M * K + M * K + 2 * M + 4 * M * G


def algorithmic_ops(M, N, K):
    return 2 * M * N * K
