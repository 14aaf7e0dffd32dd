"""numpy statement of the two pieces of streaming prefill that sit beside the quantised linears (Sec. 3.1,
"Streaming design"): test infrastructure only, like the rest of this package.

Keys are cached BEFORE the rotary embedding, because a cached token's position changes when the window slides
(a token that was at position p is now at p - delta); the rotation is applied when the keys are used, at the
shifted positions.  The new frame's tokens are inserted at the last-frame place of each camera view (the sequence
is view-major), only they are queries, and attention stays causal in that order.
"""
import numpy as np

from oracle.w4a8_oracle import bf16_bits_to_f64, f64_to_bf16_bits


def rope_shifted_keys(k_pre_bits, pos, delta, base):
    """k_rot[t,h,:] = R(pos[t] - delta) k_pre[t,h,:], the rotary embedding in its rotate-half form:
    with i < D/2, theta_i = base^(-2i/D), phi = (pos[t] - delta) theta_i,
        out[i]       = k[i] cos(phi) - k[i + D/2] sin(phi)
        out[i + D/2] = k[i + D/2] cos(phi) + k[i] sin(phi)
    in fp64, rounded to bf16 once.  k_pre_bits: [T,H,D] bf16 bit patterns; pos: [T] integers.
    Returns (fp64 [T,H,D], bf16 bits)."""
    k = bf16_bits_to_f64(k_pre_bits)
    T, H, D = k.shape
    half = D // 2
    theta = np.float64(base) ** (-2.0 * np.arange(half, dtype=np.float64) / D)
    phi = (np.asarray(pos, dtype=np.int64) - int(delta)).astype(np.float64)[:, None] * theta[None, :]      # [T, D/2]
    c, s = np.cos(phi)[:, None, :], np.sin(phi)[:, None, :]
    a, b = k[:, :, :half], k[:, :, half:]
    out = np.concatenate([a * c - b * s, b * c + a * s], axis=2)
    return out, f64_to_bf16_bits(out)


def streaming_mask(views, frames, tokens_per_frame):
    """mask[q, j] = 1 where query q may attend key j.  Keys: all views x frames x tokens_per_frame tokens in view-major
    order (position ((v * frames + f) * n + i).  Queries: the tokens of the newest frame (f = frames - 1) of every
    view, in view order.  Attention is causal in the view-major order: a key is visible iff its position is not after
    the query's.  (The paper's figure of the mask is not available; this is its caption written out.)"""
    n = tokens_per_frame
    kv = views * frames * n
    q_pos = np.array([((v * frames + frames - 1) * n + i) for v in range(views) for i in range(n)], dtype=np.int64)
    mask = np.zeros((views * n, kv), dtype=np.uint8)
    for q in range(views * n):
        for j in range(kv):
            mask[q, j] = 1 if j <= q_pos[q] else 0
    return mask
