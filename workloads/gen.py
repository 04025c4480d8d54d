"""Seeded generators of weights and prompts (numpy only, no model arithmetic).

Weights: every matrix is drawn N(0, std) in float32 from numpy's default_rng
(PCG64) seeded with `seed`, one tensor after another in the fixed order
`weight_order` returns; W_o and W_down are multiplied by `out_scale` after
drawing; for bf16 models every matrix is then rounded to the nearest bf16
value (ties to even) and returned as float32 holding that value exactly.
Norm gains are ones (optionally jittered for tests).  Linear weights are laid
out [out_features, in_features].
"""
import numpy as np


def bf16_round(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result is float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return rounded.view(np.float32)


def weight_order(shape):
    """Names and shapes of all tensors, in generation order."""
    h, f, d = shape.hidden, shape.ffn, shape.head_dim
    nq, nkv = shape.n_q_heads * d, shape.n_kv_heads * d
    out = [("embed", (shape.vocab, h))]
    if not shape.tied:
        out.append(("lm_head", (shape.vocab, h)))
    out.append(("final_norm", (h,)))
    stacks = [("layers", shape.n_recurrent)]
    if shape.n_prelude or shape.n_coda:   # Raven layout: adapter on [state; prelude output], then prelude, recurrent, coda blocks
        out.append(("adapter", (h, 2 * h)))
        stacks = [("prelude", shape.n_prelude), ("layers", shape.n_recurrent), ("coda", shape.n_coda)]
    for prefix, n in stacks:
        for l in range(n):
            out += [(f"{prefix}.{l}.norm1", (h,)), (f"{prefix}.{l}.wqkv", (nq + 2 * nkv, h)),
                    (f"{prefix}.{l}.wo", (h, nq)), (f"{prefix}.{l}.norm2", (h,)),
                    (f"{prefix}.{l}.wgateup", (2 * f, h)), (f"{prefix}.{l}.wdown", (h, f))]
    return out


def make_weights(shape, seed: int = 0, gain_jitter: float = 0.0, out_scale=None, only=None):
    """Return {name: float32 array}.  `only` (a set of names) skips materialising the others
    while still consuming the generator identically, so a subset equals the same slice of the
    full draw."""
    rng = np.random.default_rng(seed)
    scale = shape.out_scale if out_scale is None else out_scale
    w = {}
    for name, shp in weight_order(shape):
        if len(shp) == 1:
            g = np.ones(shp, dtype=np.float32)
            if gain_jitter:
                g = g + gain_jitter * rng.standard_normal(shp, dtype=np.float32)
            if only is None or name in only:
                w[name] = g
            continue
        a = rng.standard_normal(shp, dtype=np.float32)
        if only is not None and name not in only:
            continue
        a *= np.float32(shape.std)
        if name.endswith(".wo") or name.endswith(".wdown"):
            a *= np.float32(scale)
        if shape.weight_dtype == "bf16":
            a = bf16_round(a)
        w[name] = a
    return w


def make_prompt(vocab: int, n: int, seed: int = 1, seq: int = 0) -> np.ndarray:
    """Uniform-random prompt ids (int32) for sequence `seq`."""
    rng = np.random.default_rng([seed, seq])
    return rng.integers(0, vocab, size=n, dtype=np.int32)
