"""Looped transformer of Sec. 3.1 (Eq. 1): H0 = P(X), Hr = B(H(r-1)), p_r = C(Hr).

Ouro layout: P is the embedding lookup, B is the whole stack of pre-norm
blocks (shared by every recurrence), C is final RMSNorm -> lm_head ->
temperature -> softmax, applied identically at every depth.

KV is depth indexed (App. B, "KV Cache Management"): a token at recurrence r
attends to the keys/values its prefix produced *at the same recurrence r*.
Keys (after RoPE) and values are rounded to bf16 when cached if `kv_bf16`
is set -- a quantisation point of the bf16 model definition, not of the paper.
"""
import numpy as np

from . import numerics as nm


class LoopedLM:
    def __init__(self, shape, weights, kv_bf16=True):
        self.s = shape
        self.kv_bf16 = kv_bf16
        f64 = lambda a: np.asarray(a, dtype=np.float64)
        self.embed = f64(weights["embed"])
        self.lm_head = self.embed if shape.tied else f64(weights["lm_head"])
        self.final_norm = f64(weights["final_norm"])
        self.layers = []
        for l in range(shape.n_recurrent):
            g = lambda k: f64(weights[f"layers.{l}.{k}"])
            self.layers.append(dict(norm1=g("norm1"), wqkv=g("wqkv"), wo=g("wo"),
                                    norm2=g("norm2"), wgateup=g("wgateup"), wdown=g("wdown")))

    # ---- P ------------------------------------------------------------------------------
    def embed_tokens(self, ids):
        return self.embed[np.asarray(ids)]

    # ---- B, the rows of one step (Sec. 4.2 step 1: one batched call to B) ---------------
    def advance_rows(self, X, pos, prefix_kv):
        """Apply B once to every row.  A row is one token position at one recurrence.

        X [m, H]; pos [m] position of each row's token; prefix_kv(i, layer) -> (K, V) arrays
        [ctx_i, nkv, d] holding, *for row i's recurrence*, the cached keys/values of every
        earlier position of row i's prefix.  The linear maps are applied to all rows at once;
        attention is per row.  Returns the new hidden states [m, H] and own[i][layer] = (k, v),
        row i's keys/values to be cached at (layer, its recurrence, its position).
        """
        s = self.s
        X = np.array(X, dtype=np.float64)
        m = X.shape[0]
        pos = np.asarray(pos)
        nq, nkv, d = s.n_q_heads, s.n_kv_heads, s.head_dim
        own = [[] for _ in range(m)]
        for l, w in enumerate(self.layers):
            Y = nm.rmsnorm(X, w["norm1"], s.rms_eps) @ w["wqkv"].T
            q = nm.rope(Y[:, : nq * d].reshape(m, nq, d), pos, s.rope_theta)
            k = nm.rope(Y[:, nq * d: (nq + nkv) * d].reshape(m, nkv, d), pos, s.rope_theta)
            v = Y[:, (nq + nkv) * d:].reshape(m, nkv, d)
            if self.kv_bf16:
                k, v = nm.round_bf16(k), nm.round_bf16(v)
            A = np.empty((m, nq, d))
            for i in range(m):
                Kp, Vp = prefix_kv(i, l)
                K = np.concatenate([Kp, k[i][None]], axis=0)
                V = np.concatenate([Vp, v[i][None]], axis=0)
                A[i] = nm.attend(q[i], K, V)
                own[i].append((k[i], v[i]))
            X = X + A.reshape(m, -1) @ w["wo"].T
            GU = nm.rmsnorm(X, w["norm2"], s.rms_eps) @ w["wgateup"].T
            X = X + (nm.silu(GU[:, : s.ffn]) * GU[:, s.ffn:]) @ w["wdown"].T
        return X, own

    # ---- B, a whole prompt at one recurrence (prefill; causal) ---------------------------
    def advance_prompt(self, X):
        """X [n, H] hidden states of positions 0..n-1, all at the same recurrence.

        Returns the new hidden states and per-layer (K, V) [n, nkv, d] for that recurrence.
        """
        s = self.s
        n = X.shape[0]
        pos = np.arange(n)
        nq, nkv, d = s.n_q_heads, s.n_kv_heads, s.head_dim
        kv = []
        for w in self.layers:
            N1 = nm.rmsnorm(X, w["norm1"], s.rms_eps)
            Y = N1 @ w["wqkv"].T
            q = nm.rope(Y[:, : nq * d].reshape(n, nq, d), pos, s.rope_theta)
            k = nm.rope(Y[:, nq * d: (nq + nkv) * d].reshape(n, nkv, d), pos, s.rope_theta)
            v = Y[:, (nq + nkv) * d:].reshape(n, nkv, d)
            if self.kv_bf16:
                k, v = nm.round_bf16(k), nm.round_bf16(v)
            A = np.empty((n, nq, d))
            for i in range(n):
                A[i] = nm.attend(q[i], k[: i + 1], v[: i + 1])
            X = X + A.reshape(n, -1) @ w["wo"].T
            N2 = nm.rmsnorm(X, w["norm2"], s.rms_eps)
            GU = N2 @ w["wgateup"].T
            X = X + (nm.silu(GU[:, : s.ffn]) * GU[:, s.ffn:]) @ w["wdown"].T
            kv.append((k, v))
        return X, kv

    # ---- C ------------------------------------------------------------------------------
    def logits(self, x):
        """Final norm + lm_head (no temperature)."""
        return self.lm_head @ nm.rmsnorm(x, self.final_norm, self.s.rms_eps)
