"""Looped transformer of Sec. 3.1 (Eq. 1): H0 = P(X), Hr = B(H(r-1)), p_r = C(Hr).

Ouro layout: P is the embedding lookup, B is the whole stack of pre-norm
blocks (shared by every recurrence), C is final RMSNorm -> lm_head ->
temperature -> softmax, applied identically at every depth.

Raven layout (Sec. 3.1: P and C hold transformer blocks too; n_prelude, n_coda > 0):
P = embedding -> prelude blocks, giving e; H0 = e; one application of B is
  Hr = RecurrentBlocks(W_a [H(r-1); e])        (the adapter W_a is [H, 2H])
and C = coda blocks -> final RMSNorm -> lm_head.  The prelude blocks have an ordinary
KV cache; the coda blocks have ONE CACHE PER READOUT DEPTH (App. B "KV Cache Management":
"separate caches for C at each proposal and verification depth"): a readout at depth d
attends to the coda keys/values that the earlier positions produced at THEIR depth-d readout.

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
        def stack(prefix, n):
            out = []
            for l in range(n):
                g = lambda k: f64(weights[f"{prefix}.{l}.{k}"])
                out.append(dict(norm1=g("norm1"), wqkv=g("wqkv"), wo=g("wo"),
                                norm2=g("norm2"), wgateup=g("wgateup"), wdown=g("wdown")))
            return out
        self.layers = stack("layers", shape.n_recurrent)
        self.raven = shape.n_prelude > 0 or shape.n_coda > 0
        self.prelude = stack("prelude", shape.n_prelude)
        self.coda = stack("coda", shape.n_coda)
        self.adapter = f64(weights["adapter"]) if self.raven else None

    # ---- P ------------------------------------------------------------------------------
    def embed_tokens(self, ids):
        return self.embed[np.asarray(ids)]

    # ---- B, the rows of one step (Sec. 4.2 step 1: one batched call to B) ---------------
    def advance_rows(self, X, pos, prefix_kv, E=None):
        """Apply B once to every row.  A row is one token position at one recurrence.  Raven layout: E [m, H] holds
        the rows' prelude outputs and the recurrent blocks start from the adapter's W_a [X; E].

        X [m, H]; pos [m] position of each row's token; prefix_kv(i, layer) -> (K, V) arrays
        [ctx_i, nkv, d] holding, *for row i's recurrence*, the cached keys/values of every
        earlier position of row i's prefix.  The linear maps are applied to all rows at once;
        attention is per row.  Returns the new hidden states [m, H] and own[i][layer] = (k, v),
        row i's keys/values to be cached at (layer, its recurrence, its position).
        """
        X = np.array(X, dtype=np.float64)
        if self.raven:
            X = np.concatenate([X, np.asarray(E, dtype=np.float64)], axis=1) @ self.adapter.T
        return self._blocks_rows(self.layers, X, pos, prefix_kv)

    def prelude_rows(self, X, pos, prefix_kv):
        """The transformer blocks of P on embedded rows X [m, H]: returns e [m, H] and own[i][layer] = (k, v)."""
        return self._blocks_rows(self.prelude, np.array(X, dtype=np.float64), pos, prefix_kv)

    def coda_rows(self, X, pos, prefix_kv):
        """The transformer blocks of C on states X [m, H] (all read out at the same depth class): returns the hidden
        states the final norm + lm_head (`logits`) take, and own[i][layer] = (k, v) for that depth's coda cache."""
        return self._blocks_rows(self.coda, np.array(X, dtype=np.float64), pos, prefix_kv)

    def _blocks_rows(self, layers, X, pos, prefix_kv):
        s = self.s
        m = X.shape[0]
        pos = np.asarray(pos)
        nq, nkv, d = s.n_q_heads, s.n_kv_heads, s.head_dim
        own = [[] for _ in range(m)]
        for l, w in enumerate(layers):
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
    def advance_prompt(self, X, E=None):
        """X [n, H] hidden states of positions 0..n-1, all at the same recurrence (Raven layout: E = their prelude
        outputs, fed through the adapter first).

        Returns the new hidden states and per-layer (K, V) [n, nkv, d] for that recurrence.
        """
        X = np.array(X, dtype=np.float64)
        if self.raven:
            X = np.concatenate([X, np.asarray(E, dtype=np.float64)], axis=1) @ self.adapter.T
        return self._blocks_prompt(self.layers, X)

    def prelude_prompt(self, X):
        return self._blocks_prompt(self.prelude, np.array(X, dtype=np.float64))

    def coda_prompt(self, X):
        return self._blocks_prompt(self.coda, np.array(X, dtype=np.float64))

    def _blocks_prompt(self, layers, X):
        s = self.s
        n = X.shape[0]
        pos = np.arange(n)
        nq, nkv, d = s.n_q_heads, s.n_kv_heads, s.head_dim
        kv = []
        for w in layers:
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
