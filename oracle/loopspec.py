"""Vanilla decoding and LoopSpec (Algorithm 1, App. H; Sec. 4.2-4.3), float64, one sequence.

`Decoder` holds the committed prefix and its depth-indexed KV.  `vanilla` finishes all R
recurrences of a token before the next (Fig. 1a).  `loopspec` follows Algorithm 1 in its
printed order: snapshot the active set, advance every branch once, first proposal at d1,
gated residual second proposal at d2, then cascade verification of the branch at depth R
and Reroot.  Every decision is logged with its margin (distance to the opposite outcome).
"""
from dataclasses import dataclass, field

import numpy as np

from . import numerics as nm
from . import sampling as sp


@dataclass
class Record:                      # one entry of Q_b: (candidate token, proposal distribution, child)
    token: int
    q: object                      # probability vector (None under greedy decoding)
    child: "Branch"


@dataclass
class Branch:                      # Algorithm 1: prefix X(b), hidden H_b, depth r_b, records Q_b
    parent: "Branch"               # None for the root (its whole prefix is committed)
    token: int                     # last token of the prefix
    pos: int                       # position of that token = len(prefix) - 1
    H: np.ndarray
    r: int = 0
    records: list = field(default_factory=list)
    kv: dict = field(default_factory=dict)      # recurrence -> [per layer (k, v)] while speculative
    e: object = None               # Raven layout: prelude output of the last token (constant over the recurrences)
    pre_kv: object = None          # ... its prelude keys/values [per layer (k, v)] while speculative
    coda_kv: dict = field(default_factory=dict)  # ... readout depth -> [per coda layer (k, v)] while speculative
    q1_logits: object = None       # kept for inspection
    q2_logits: object = None

    def is_descendant_of(self, other):
        b = self
        while b is not None:
            if b is other:
                return True
            b = b.parent
        return False


class Decoder:
    def __init__(self, model, temperature=0.0, seed=0, seq=0, max_ctx=None, top_k=0, top_p=1.0):
        self.m = model
        self.T = float(temperature)
        self.top_k, self.top_p = int(top_k), float(top_p)   # the optional filters of C (Sec. 3.1)
        self.seed, self.seq = seed, seq
        self.ids = []              # committed tokens (prompt + decoded)
        self.n_prompt = 0
        self.max_ctx = max_ctx
        self.K = self.V = None     # [R+1][layer] arrays [max_ctx, nkv, d]; index by recurrence 1..R
        self.log = []              # decision log
        self.rows_per_step = []
        self.tv_log = []           # per verification (sampling): TV(p_d1, p_R) and TV(p_d2, p_R) or None (Sec. 4.1)

    # ---- committed, depth-indexed KV ---------------------------------------------------------
    def _alloc(self, n_total):
        s = self.m.s
        shp = (n_total, s.n_kv_heads, s.head_dim)
        self.K = [[np.zeros(shp) for _ in range(s.n_recurrent)] for _ in range(s.R + 1)]
        self.V = [[np.zeros(shp) for _ in range(s.n_recurrent)] for _ in range(s.R + 1)]
        if getattr(self.m, "raven", False):   # prelude cache, and one coda cache per readout depth (App. B)
            self.PK = [np.zeros(shp) for _ in range(s.n_prelude)]
            self.PV = [np.zeros(shp) for _ in range(s.n_prelude)]
            self.CK = {d: [np.zeros(shp) for _ in range(s.n_coda)] for d in self.readout_depths}
            self.CV = {d: [np.zeros(shp) for _ in range(s.n_coda)] for d in self.readout_depths}

    @property
    def raven(self):
        return getattr(self.m, "raven", False)

    def _store_prelude(self, pos, per_layer_kv):
        for l, (k, v) in enumerate(per_layer_kv):
            self.PK[l][pos], self.PV[l][pos] = k, v

    def _store_coda(self, d, pos, per_layer_kv):
        for l, (k, v) in enumerate(per_layer_kv):
            self.CK[d][l][pos], self.CV[d][l][pos] = k, v

    def _store_committed(self, r, pos, per_layer_kv):
        for l, (k, v) in enumerate(per_layer_kv):
            self.K[r][l][pos] = k
            self.V[r][l][pos] = v

    # ---- readout C -----------------------------------------------------------------------------
    def probs(self, logits):
        """C after the lm_head: temperature, optional top-k / top-p filtering, normalisation (Sec. 3.1)."""
        p = nm.softmax(logits / self.T)
        if self.top_k or self.top_p < 1.0:
            p, margin = sp.top_k_top_p(p, self.top_k, self.top_p)
            self.log.append(dict(kind="filter", margin=margin))
        return p

    def _draw(self, weights, position, purpose):
        g = sp.gumbel(self.seed, self.seq, position, purpose, len(weights))
        idx, margin = sp.race(weights, g)
        return int(idx), float(margin)

    def _argmax(self, logits):
        i = int(np.argmax(logits))             # lowest index on ties
        rest = np.delete(logits, i)
        return i, float(logits[i] - rest.max()) if rest.size else np.inf

    def _sample_target(self, logits, position, purpose):
        """x ~ C(H) (argmax when T = 0)."""
        if self.T == 0.0:
            return self._argmax(logits)
        return self._draw(self.probs(logits), position, purpose)

    # ---- prefill: all R recurrences over the prompt, first token from C(H^R) -------------------
    def prefill(self, prompt, n_decode, depths=None):
        """depths = (d1, d2) of the LoopSpec run that follows (Raven layout only: the prompt must fill the coda cache of
        every readout depth; None: only depth R, which is all vanilla decoding needs)."""
        s = self.m.s
        self.ids = [int(t) for t in prompt]
        self.n_prompt = n = len(self.ids)
        self.readout_depths = sorted({s.R} | {d for d in (depths or ()) if d})
        self._alloc(self.max_ctx or (n + n_decode + 1))
        X = self.m.embed_tokens(self.ids)
        E = None
        if self.raven:
            X, kv = self.m.prelude_prompt(X)
            E = X
            for l, (k, v) in enumerate(kv):
                self.PK[l][:n], self.PV[l][:n] = k, v
        for r in range(1, s.R + 1):
            X, kv = self.m.advance_prompt(X, E)
            for l, (k, v) in enumerate(kv):
                self.K[r][l][:n] = k
                self.V[r][l][:n] = v
            if self.raven and r in self.readout_depths:
                Xc, ckv = self.m.coda_prompt(X)
                for l, (k, v) in enumerate(ckv):
                    self.CK[r][l][:n], self.CV[r][l][:n] = k, v
        z = self.m.logits(Xc[-1] if self.raven else X[-1])
        self.first_logits = z
        tok, margin = self._sample_target(z, n, sp.VANILLA)
        self.log.append(dict(kind="first", pos=n, token=tok, margin=margin))
        self.ids.append(tok)
        return tok

    # ---- vanilla: R recurrences per token ------------------------------------------------------
    def vanilla(self, n_tokens, keep_logits=False):
        s = self.m.s
        out, all_logits = [], []
        for _ in range(n_tokens):
            pos = len(self.ids) - 1
            x = self.m.embed_tokens([self.ids[-1]])
            e = None
            if self.raven:
                x, own = self.m.prelude_rows(x, [pos], lambda i, l: (self.PK[l][:pos], self.PV[l][:pos]))
                self._store_prelude(pos, own[0])
                e = x
            for r in range(1, s.R + 1):
                x, own = self.m.advance_rows(
                    x, [pos], lambda i, l, r=r: (self.K[r][l][:pos], self.V[r][l][:pos]), e)
                self._store_committed(r, pos, own[0])
            if self.raven:
                x, own = self.m.coda_rows(x, [pos], lambda i, l: (self.CK[s.R][l][:pos], self.CV[s.R][l][:pos]))
                self._store_coda(s.R, pos, own[0])
            z = self.m.logits(x[0])
            tok, margin = self._sample_target(z, pos + 1, sp.VANILLA)
            self.log.append(dict(kind="vanilla", pos=pos + 1, token=tok, margin=margin))
            self.ids.append(tok)
            out.append(tok)
            if keep_logits:
                all_logits.append(z)
        return (out, all_logits) if keep_logits else out

    # ---- LoopSpec ------------------------------------------------------------------------------
    def _spawn(self, parent, token, pos):
        """Spawn(X || token): a branch at depth 0 with H0 = P(X || token) (Eq. 1; for the Raven layout the prelude blocks
        run here, over the prelude keys/values of the branch's prefix)."""
        b = Branch(parent=parent, token=int(token), pos=pos, H=self.m.embed_tokens([token])[0])
        if self.raven:
            e, own = self.m.prelude_rows(b.H[None], [pos], lambda i, l: self._prefix_generic(
                b, l, self.PK, self.PV, lambda a: a.pre_kv))
            b.H = b.e = e[0]
            if parent is None:
                self._store_prelude(pos, own[0])
            else:
                b.pre_kv = own[0]
        self.active.append(b)
        return b

    def _prefix_generic(self, b, layer, Kc, Vc, branch_kv):
        """Keys/values of every position before b's own in b's prefix, for a cache with committed arrays Kc/Vc [layer] and
        per-branch entries branch_kv(a) -> [per layer (k, v)] for the uncommitted ancestors."""
        chain = []
        a = b.parent
        while a is not None:
            chain.append(a)
            a = a.parent
        chain.reverse()
        n_committed = b.pos if not chain else chain[0].pos
        Ks, Vs = [Kc[layer][:n_committed]], [Vc[layer][:n_committed]]
        for a in chain:
            if a.parent is None:
                Ks.append(Kc[layer][a.pos][None])
                Vs.append(Vc[layer][a.pos][None])
            else:
                k, v = branch_kv(a)[layer]
                Ks.append(k[None])
                Vs.append(v[None])
        return np.concatenate(Ks, axis=0), np.concatenate(Vs, axis=0)

    def _readout_logits(self, b, depth):
        """p_r = C(H^r) before temperature (Sec. 3.1): final norm + lm_head; for the Raven layout the coda blocks first, over
        the coda cache of this readout depth (App. B), whose entry for b's own position is produced here."""
        if not self.raven:
            return self.m.logits(b.H)
        x, own = self.m.coda_rows(b.H[None], [b.pos], lambda i, l: self._prefix_generic(
            b, l, self.CK[depth], self.CV[depth], lambda a: a.coda_kv[depth]))
        if b.parent is None:
            self._store_coda(depth, b.pos, own[0])
        else:
            b.coda_kv[depth] = own[0]
        return self.m.logits(x[0])

    def _prefix_kv(self, b, r, layer):
        """Keys/values, at recurrence r, of every position before b's own in b's prefix."""
        chain = []
        a = b.parent
        while a is not None:
            chain.append(a)
            a = a.parent
        chain.reverse()                          # chain[0] is the root when b is speculative
        n_committed = b.pos if not chain else chain[0].pos
        Ks = [self.K[r][layer][:n_committed]]
        Vs = [self.V[r][layer][:n_committed]]
        for a in chain:
            if a.parent is None:                 # the root's KV already lives in the committed arrays
                Ks.append(self.K[r][layer][a.pos][None])
                Vs.append(self.V[r][layer][a.pos][None])
            else:
                k, v = a.kv[r][layer]
                Ks.append(k[None])
                Vs.append(v[None])
        return np.concatenate(Ks, axis=0), np.concatenate(Vs, axis=0)

    def _verify(self, b, p_logits):
        """Algorithm 1 Verify(b, p): returns (token, child or None, source) with source 1, 2 or 3 (resampled)."""
        pos = b.pos + 1                          # the position being decided
        if self.T == 0.0:                        # greedy form (end of Sec. 4.3)
            top, margin = self._argmax(p_logits)
            for j, rec in enumerate(b.records):
                if rec.token == top:
                    self.log.append(dict(kind="verify", pos=pos, source=j + 1, token=top, margin=margin))
                    return top, rec.child, j + 1
            self.log.append(dict(kind="verify", pos=pos, source=3, token=top, margin=margin))
            return top, None, 3
        rho = self.probs(p_logits)
        # the empirical profile of Sec. 4.1: total variation between the early readouts and the target
        if b.records:
            tv1 = 0.5 * float(np.abs(b.records[0].q - rho).sum())
            tv2 = None
            if len(b.records) > 1 and b.q2_logits is not None:
                tv2 = 0.5 * float(np.abs(self.probs(b.q2_logits) - rho).sum())
            self.tv_log.append((tv1, tv2))
        for j, rec in enumerate(b.records):
            U = float(sp.uniform(self.seed, self.seq, pos, sp.ACCEPT1 + j))
            a = sp.accept_prob(rho, rec.q, rec.token)
            self.log.append(dict(kind=f"accept{j + 1}", pos=pos, token=rec.token, accepted=U < a,
                                 margin=abs(U - a)))
            if U < a:
                return rec.token, rec.child, j + 1
            rho = sp.residual(rho, rec.q)
        tok, margin = self._draw(rho, pos, sp.RESAMPLE)
        self.log.append(dict(kind="resample", pos=pos, token=tok, margin=margin))
        return tok, None, 3

    def loopspec(self, n_tokens, d1, d2=0, gate=True, residual_q2=True, keep_logits=False, mask_first=False):
        """Commit exactly n_tokens more tokens.  d2 = 0 disables the second proposal.

        Returns the committed tokens; `self.commits` lists, per token, its source and flags;
        `self.rows_per_step` the number of branches advanced by each batched call.
        """
        s = self.m.s
        R = s.R
        assert 1 <= d1 < R and (d2 == 0 or d1 < d2 < R)
        if self.raven:
            assert {d for d in (d1, d2, R) if d} <= set(self.readout_depths), "prefill(..., depths=(d1, d2)) first"
        self.active = []
        self.commits, self.verify_logits = [], []
        self.stats = dict(steps=0, n_decode=0, n_accept1=0, n_accept2=0, n_restart=0,
                          gate_evals=0, gate_opens=0, rows_total=0, rows_max=0, readout_rows_total=0)
        out = []
        self._spawn(None, self.ids[-1], len(self.ids) - 1)
        while len(out) < n_tokens:
            cur = list(self.active)
            X = np.stack([b.H for b in cur])
            Xn, own = self.m.advance_rows(
                X, [b.pos for b in cur], lambda i, l: self._prefix_kv(cur[i], cur[i].r + 1, l),
                np.stack([b.e for b in cur]) if self.raven else None)
            self.stats["steps"] += 1
            self.stats["rows_total"] += len(cur)
            self.stats["rows_max"] = max(self.stats["rows_max"], len(cur))
            self.rows_per_step.append(len(cur))
            for i, b in enumerate(cur):
                b.H = Xn[i]
                b.r += 1
                if b.parent is None:
                    self._store_committed(b.r, b.pos, own[i])
                else:
                    b.kv[b.r] = own[i]
            for b in cur:
                pos = b.pos + 1                  # position this branch proposes for
                if b.r == d1:                    # first proposal
                    z1 = self._readout_logits(b, d1)
                    self.stats["readout_rows_total"] += 1
                    b.q1_logits = z1
                    if self.T == 0.0:
                        x1, margin = self._argmax(z1)
                        q1 = None
                    else:
                        q1 = self.probs(z1)
                        x1, margin = self._draw(q1, pos, sp.DRAFT1)
                    self.log.append(dict(kind="draft1", pos=pos, token=x1, margin=margin))
                    c1 = self._spawn(b, x1, pos)
                    b.records.append(Record(x1, q1, c1))
                elif d2 and b.r == d2:           # gated residual second proposal
                    z2 = self._readout_logits(b, d2)
                    self.stats["readout_rows_total"] += 1
                    b.q2_logits = z2
                    x1 = b.records[0].token
                    self.stats["gate_evals"] += 1
                    if self.T == 0.0:
                        top, margin = self._argmax(z2)
                        is_open = (top != x1) or not gate
                        self.log.append(dict(kind="gate", pos=pos, open=is_open, token=top, margin=margin))
                        if is_open:
                            # residual of two one-hot distributions: the deeper argmax; without the
                            # gate the two may coincide and the residual falls back to q2~ itself
                            x2 = top
                            if mask_first and top == x1:   # second-proposal ablation (Sec. 6): the first candidate is masked out
                                x2, margin = self._argmax(np.where(np.arange(len(z2)) == x1, -np.inf, z2))
                                self.log.append(dict(kind="draft2", pos=pos, token=x2, margin=margin))
                            self.stats["gate_opens"] += 1
                            c2 = self._spawn(b, x2, pos)
                            b.records.append(Record(x2, None, c2))
                    else:
                        q1 = b.records[0].q
                        q2t = self.probs(z2)
                        is_open = (q2t[x1] < q1[x1]) or not gate
                        with np.errstate(divide="ignore"):   # a filtered q2~ may give the candidate no mass
                            gm = abs(np.log(q2t[x1]) - np.log(q1[x1]))
                        self.log.append(dict(kind="gate", pos=pos, open=is_open, margin=gm))
                        if is_open and mask_first:
                            # second-proposal ablation (Sec. 6): the first candidate is masked out of the proposal
                            q2 = sp.masked_second_proposal(q2t, q1, x1, residual_q2)
                            is_open = q2 is not None      # q2~ puts all its mass on the first candidate: no proposal
                        elif is_open:
                            q2 = sp.residual(q2t, q1) if residual_q2 else q2t
                        if is_open:
                            x2, margin = self._draw(q2, pos, sp.DRAFT2)
                            self.log.append(dict(kind="draft2", pos=pos, token=x2, margin=margin))
                            self.stats["gate_opens"] += 1
                            c2 = self._spawn(b, x2, pos)
                            b.records.append(Record(x2, q2, c2))
            bmax = max(self.active, key=lambda b: b.r)
            if bmax.r == R:
                assert bmax.parent is None
                p_logits = self._readout_logits(bmax, R)
                self.stats["readout_rows_total"] += 1
                tok, child, source = self._verify(bmax, p_logits)
                if keep_logits:
                    self.verify_logits.append(p_logits)
                gate_open = len(bmax.records) > 1
                self.ids.append(tok)
                out.append(tok)
                self.commits.append(dict(token=tok, source=source, accepted1=int(source == 1),
                                         accepted2=int(source == 2), gate_open=int(gate_open),
                                         step=self.stats["steps"]))
                self.stats["n_decode"] += 1
                self.stats["n_accept1"] += source == 1
                self.stats["n_accept2"] += source == 2
                self.stats["n_restart"] += source == 3
                if child is None:                # restart: fresh branch on the verified prefix
                    self.active = []
                    self._spawn(None, tok, bmax.pos + 1)
                else:                            # Reroot: keep the chosen child and its descendants
                    self.active = [b for b in self.active if b.is_descendant_of(child)]
                    child.parent = None
                    for r, per_layer in child.kv.items():
                        self._store_committed(r, child.pos, per_layer)
                    child.kv = {}
                    if self.raven:
                        self._store_prelude(child.pos, child.pre_kv)
                        for d, per_layer in child.coda_kv.items():
                            self._store_coda(d, child.pos, per_layer)
                        child.pre_kv, child.coda_kv = None, {}
        st = self.stats
        den = st["n_accept1"] * d1 + st["n_accept2"] * d2 + st["n_restart"] * R
        st["gamma"] = st["n_decode"] * R / den if den else float("nan")
        return out
