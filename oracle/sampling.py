"""Random draws and the rejection rule (Sec. 3.2 Eq. 2-4, Sec. 4.3, Algorithm 1 Verify).

The paper only says "x ~ q" and "U ~ U(0,1)".  Readings fixed here (any exact
sampler is lossless, Sec. 3.2):
  * random bits: the counter-based generator Philox4x32-10 with key = the two
    32-bit halves of the seed and counter = (block, position, sequence, purpose),
    so a draw depends only on what is being decided, never on which branches
    were pruned before it;
  * uniform from a 32-bit word x: u = ((x >> 9) + 0.5) * 2^-23, in (0, 1);
  * categorical draw: exponential race / Gumbel-max, x = argmax_v log w_v + g_v,
    g_v = -log(-log u_v), u_v = word (v mod 4) of block v div 4; ties -> lowest v;
  * acceptance uniforms: word 0 of block 0;
  * the optional top-k / top-p filters of the post-layers C (Sec. 3.1): tokens are ranked by
    decreasing probability (ties: lower index first); top-k keeps the first k and renormalises;
    top-p then keeps the shortest prefix of that ranking whose mass reaches top_p and
    renormalises.  The filtered distribution IS p_r, at every depth r.
"""
import numpy as np

DRAFT1, DRAFT2, ACCEPT1, ACCEPT2, RESAMPLE, VANILLA = 1, 2, 3, 4, 5, 6

_M0, _M1 = 0xD2511F53, 0xCD9E8D57
_W0, _W1 = 0x9E3779B9, 0xBB67AE85
_MASK = 0xFFFFFFFF


def philox4x32_10(counter, key):
    """Philox4x32 with 10 rounds.  counter: 4 arrays (or ints) of uint32 values, key: 2 ints.

    Returns 4 uint64 arrays holding 32-bit words.
    """
    c = [np.asarray(x, dtype=np.uint64) & np.uint64(_MASK) for x in counter]
    c = list(np.broadcast_arrays(*c))
    k0, k1 = int(key[0]) & _MASK, int(key[1]) & _MASK
    for _ in range(10):
        p0 = np.uint64(_M0) * c[0]
        p1 = np.uint64(_M1) * c[2]
        hi0, lo0 = p0 >> np.uint64(32), p0 & np.uint64(_MASK)
        hi1, lo1 = p1 >> np.uint64(32), p1 & np.uint64(_MASK)
        c = [hi1 ^ c[1] ^ np.uint64(k0), lo1, hi0 ^ c[3] ^ np.uint64(k1), lo0]
        k0, k1 = (k0 + _W0) & _MASK, (k1 + _W1) & _MASK
    return c


def _u01(words):
    return ((words >> np.uint64(9)).astype(np.float64) + 0.5) * 2.0 ** -23


def _key(seed):
    return (seed & _MASK, (seed >> 32) & _MASK)


def uniform(seed, seq, position, purpose):
    """One U(0,1) draw for (sequence, position, purpose).  position may be an array."""
    w = philox4x32_10((0, position, seq, purpose), _key(seed))
    return _u01(w[0])


def gumbel(seed, seq, position, purpose, vocab):
    """Gumbel(0,1) noise for every vocabulary index: shape [..., vocab] (position may be an array)."""
    nblk = (vocab + 3) // 4
    blk = np.arange(nblk, dtype=np.uint64)
    pos = np.asarray(position, dtype=np.uint64)[..., None]
    w = philox4x32_10((blk, pos, seq, purpose), _key(seed))
    words = np.stack(w, axis=-1).reshape(pos.shape[:-1] + (nblk * 4,))[..., :vocab]
    return -np.log(-np.log(_u01(words)))


def race(weights, g):
    """Exponential-race draw from unnormalised weights (last axis): argmax of log w + g over w > 0.

    Returns (index, margin) where margin is the gap between the best and second-best score.
    """
    with np.errstate(divide="ignore"):
        score = np.where(weights > 0, np.log(np.where(weights > 0, weights, 1.0)) + g, -np.inf)
    idx = np.argmax(score, axis=-1)
    if score.shape[-1] > 1:
        top2 = np.partition(score, -2, axis=-1)[..., -2:]
        margin = top2[..., 1] - top2[..., 0]
    else:
        margin = np.full(idx.shape, np.inf)
    return idx, margin


def positive_part_diff(mu, nu):
    """[mu - nu]_+ of Sec. 3.2."""
    return np.maximum(mu - nu, 0.0)


def residual(mu, nu):
    """(mu (-) nu) of Eq. 2: [mu - nu]_+ normalised.  If the positive part has no mass (mu == nu,
    excluded by the paper's "distinct distributions") mu itself is returned."""
    d = positive_part_diff(mu, nu)
    s = np.sum(d, axis=-1, keepdims=True)
    return np.where(s > 0, d / np.where(s > 0, s, 1.0), mu)


def masked_second_proposal(q2t, q1, x1, residual_q2=True):
    """Second proposal with the first candidate x1 masked out (the variant of the second-proposal ablation, Sec. 6):
    x1's mass is removed from the residual proposal norm([q2~ - q1]_+) if that leaves mass elsewhere (or if
    residual_q2 is off, from q2~ directly), else from q2~, and the rest renormalised.  None when q2~ has all its mass
    on x1: there is nothing else to propose."""
    for base in ([positive_part_diff(q2t, q1)] if residual_q2 else []) + [np.asarray(q2t, dtype=np.float64)]:
        base = base.copy()
        base[x1] = 0.0
        if base.sum() > 0:
            return base / base.sum()
    return None


def accept_prob(rho, q, x):
    """min{1, rho(x)/q(x)} of Eq. 3 for a candidate x drawn from q (so q(x) > 0)."""
    return min(1.0, rho[x] / q[x])


def top_k_top_p(p, top_k=0, top_p=1.0):
    """The filters inside C (Sec. 3.1) applied to one probability vector.

    Returns (filtered distribution, margin): margin is how far the decision "keep exactly this many
    tokens" is from flipping - the smaller of the distance of the cumulative mass from top_p on
    either side of the last kept token and, in probability units, the gap between the last kept
    and the first dropped token (their order decides who is kept).
    """
    p = np.asarray(p, dtype=np.float64)
    V = len(p)
    order = np.lexsort((np.arange(V), -p))          # decreasing probability, then increasing index
    margin = np.inf
    m = V
    if top_k and top_k < V:
        m = int(top_k)
        margin = min(margin, p[order[m - 1]] - p[order[m]])
    kept = order[:m]
    pk = p[kept] / p[kept].sum()
    if top_p < 1.0:
        cum = np.cumsum(pk)
        j = int(np.searchsorted(cum, top_p, side="left")) + 1   # first prefix whose mass reaches top_p
        j = min(j, m)
        margin = min(margin, cum[j - 1] - top_p)
        if j >= 2:
            margin = min(margin, top_p - cum[j - 2])
        if j < m:
            margin = min(margin, pk[j - 1] - pk[j])
        kept, pk = kept[:j], pk[:j] / pk[:j].sum()
    out = np.zeros(V)
    out[kept] = pk
    return out, float(margin)
