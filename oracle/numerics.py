"""Elementary operators of the looped LM, float64.

Readings of points the paper leaves to "the model as given" (Sec. 3.1):
Llama-style blocks -- RMSNorm with eps inside the square root, rotary
embedding with rotate-half pairing (i, i + d/2) and inverse frequencies
theta^(-2i/d), attention scale 1/sqrt(head_dim), SwiGLU MLP, no biases.
"""
import numpy as np


def round_bf16(a):
    """Nearest-bf16 rounding (ties to even) of float64 values; result float64.

    The value is first rounded to float32 (as a float32 store would), then its
    low 16 bits are rounded away.
    """
    f = np.asarray(a, dtype=np.float64).astype(np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    r = ((u + np.uint64(0x7FFF) + lsb) >> np.uint64(16)) << np.uint64(16)
    return r.astype(np.uint32).view(np.float32).astype(np.float64)


def rmsnorm(x, gain, eps):
    """x / sqrt(mean(x^2) + eps) * gain over the last axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain


def rope_angles(pos, head_dim, theta):
    """cos, sin of pos * theta^(-2i/d), i = 0..d/2-1.  pos: int array [...]."""
    i = np.arange(head_dim // 2, dtype=np.float64)
    inv_freq = theta ** (-2.0 * i / head_dim)
    ang = np.asarray(pos, dtype=np.float64)[..., None] * inv_freq
    return np.cos(ang), np.sin(ang)


def rope(x, pos, theta):
    """Rotate x[..., n_heads, head_dim] at integer positions pos[...]."""
    d = x.shape[-1]
    cos, sin = rope_angles(pos, d, theta)
    cos, sin = cos[..., None, :], sin[..., None, :]
    x1, x2 = x[..., : d // 2], x[..., d // 2:]
    return np.concatenate([x1 * cos - x2 * sin, x2 * cos + x1 * sin], axis=-1)


def silu(x):
    return x / (1.0 + np.exp(-x))


def softmax(z, axis=-1):
    z = z - np.max(z, axis=axis, keepdims=True)
    e = np.exp(z)
    return e / np.sum(e, axis=axis, keepdims=True)


def attend(q, K, V):
    """One query against its keys.  q [n_q_heads, d]; K, V [ctx, n_kv_heads, d].

    Query head h uses kv head h // (n_q_heads // n_kv_heads).  Returns [n_q_heads, d].
    """
    nq, d = q.shape
    nkv = K.shape[1]
    g = nq // nkv
    out = np.empty_like(q)
    for h in range(nq):
        kh, vh = K[:, h // g, :], V[:, h // g, :]
        w = softmax(kh @ q[h] / np.sqrt(d))
        out[h] = w @ vh
    return out
