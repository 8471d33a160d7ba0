"""CPU oracle for the ActQKV per-window retrieval path (arXiv 2502.13542).

TEST INFRASTRUCTURE ONLY.  A plain, slow, fp64 NumPy statement of what the
paper defines, used to check the CUDA library and as the timed CPU baseline.
It shares no code with the CUDA path and imports nothing from it; only the
tests, the smoke check and the benchmark's cpu-baseline / reference legs may
import this module.  The product never routes through it.

Every function cites the passage of the paper it follows.  Where the paper is
silent the reading taken is stated next to the code; the pieces the paper does
not pin at all are marked PARITY UNPINNED:

  * PARITY UNPINNED  kv_head_probe      (how G query heads share one KV head)
  * PARITY UNPINNED  build_representatives / block aggregation (how a block of
                     keys is turned into one score)
  * PARITY UNPINNED  BudgetChain's theta-bar (history mean) and integer rounding

Shapes: W window tokens, Hq query heads, Hkv KV heads, G = Hq // Hkv,
D head dim, B tokens per block, r representatives per block, n candidate blocks.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# ----------------------------------------------------------------------------
# storage rounding (an encoding, restated here independently of any other code)
# ----------------------------------------------------------------------------
def round_to_bf16(x) -> np.ndarray:
    """Nearest-even rounding of real values to bfloat16 (8-bit significand,
    fp32 exponent range); returns float64 holding the rounded values."""
    x32 = np.asarray(x, dtype=F64).astype(np.float32)          # fp64 -> fp32 (RNE)
    bits = x32.view(np.uint32).astype(np.uint64)
    keep = bits >> np.uint64(16)
    rem = bits & np.uint64(0xFFFF)
    up = (rem > 0x8000) | ((rem == 0x8000) & ((keep & np.uint64(1)) == 1))
    keep = keep + up.astype(np.uint64)
    out = (keep << np.uint64(16)).astype(np.uint32).view(np.float32)
    return out.astype(F64)


def round_to_storage(x, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return round_to_bf16(x)
    if dtype == "f32":
        return np.asarray(x, dtype=F64).astype(np.float32).astype(F64)
    raise ValueError(dtype)


# ----------------------------------------------------------------------------
# Step 1: query statistics (Eq. 8) and Activation Bias (Eq. 7)
# ----------------------------------------------------------------------------
def query_stats_two_pass(q_history) -> tuple[np.ndarray, np.ndarray]:
    """Eq. 8 written out: per (head, channel) mean over ALL m*t queries seen so
    far and the unbiased variance about that mean (divisor m*t - 1).

    q_history: [m*t, Hq, D] (all windows 1..t concatenated)."""
    q = np.asarray(q_history, dtype=F64)
    mt = q.shape[0]
    zbar = q.sum(axis=0) / mt
    dev = q - zbar[None]
    sigma2 = (dev * dev).sum(axis=0) / (mt - 1) if mt > 1 else np.zeros_like(zbar)
    return zbar, sigma2


class RunningStats:
    """Streaming form of Eq. 8: each window's (count, mean, sum of squared
    deviations) is computed two-pass and merged into the running triple with the
    pairwise-merge identity, so the result after window t equals
    query_stats_two_pass over windows 1..t."""

    def __init__(self, n_heads: int, head_dim: int):
        self.count = 0
        self.mean = np.zeros((n_heads, head_dim), F64)
        self.m2 = np.zeros((n_heads, head_dim), F64)

    def update(self, q_window) -> None:
        q = np.asarray(q_window, dtype=F64)
        nb = q.shape[0]
        if nb == 0:
            return
        mean_b = q.sum(axis=0) / nb
        m2_b = ((q - mean_b[None]) ** 2).sum(axis=0)
        na = self.count
        n = na + nb
        delta = mean_b - self.mean
        self.mean = self.mean + delta * (nb / n)
        self.m2 = self.m2 + m2_b + delta * delta * (na * nb / n)
        self.count = n

    def variance(self) -> np.ndarray:
        return self.m2 / (self.count - 1) if self.count > 1 else np.zeros_like(self.m2)

    def copy(self) -> "RunningStats":
        c = RunningStats(*self.mean.shape)
        c.count, c.mean, c.m2 = self.count, self.mean.copy(), self.m2.copy()
        return c


def activation_bias(q_window, zbar, sigma2, var_eps: float = 1e-12):
    """Eq. 7: phi_j = (q_j - zbar)^2 / sigma^2, element-wise per head and channel.
    sigma^2 is floored at var_eps (the paper does not treat sigma^2 = 0).

    Returns (Phi [W, Hq, D], a [W, Hq]) with a_j = ||phi_j||_1 (phi >= 0)."""
    q = np.asarray(q_window, dtype=F64)
    var = np.maximum(np.asarray(sigma2, dtype=F64), var_eps)
    phi = (q - np.asarray(zbar, F64)[None]) ** 2 / var[None]
    return phi, phi.sum(axis=2)


# ----------------------------------------------------------------------------
# Step 2: activation-aware probe-query (Eq. 9)
# ----------------------------------------------------------------------------
def probe_weights(a) -> np.ndarray:
    """Eq. 9 weights ||phi_j||_1 / ||Phi||_1 with ||Phi||_1 the entry-wise L1
    norm, so each head's weights sum to 1.  If every a_j is 0 the weights are
    uniform (case not treated by the paper).  a: [W, Hq] -> [W, Hq]."""
    a = np.asarray(a, dtype=F64)
    tot = a.sum(axis=0)
    w = np.empty_like(a)
    for h in range(a.shape[1]):
        w[:, h] = a[:, h] / tot[h] if tot[h] > 0 else 1.0 / a.shape[0]
    return w


def probe_query(q_window, a) -> np.ndarray:
    """Eq. 9: Q_probe = sum_j w_j q_j, per query head.  -> [Hq, D]."""
    q = np.asarray(q_window, dtype=F64)
    w = probe_weights(a)
    return np.einsum("jh,jhd->hd", w, q)


def mean_pool_probe(q_window) -> np.ndarray:
    """The mean-pooling probe the paper compares against (Sec. 1): uniform weights."""
    return np.asarray(q_window, dtype=F64).mean(axis=0)


def kv_head_probe(probe_qh, n_kv_heads: int) -> np.ndarray:
    """PARITY UNPINNED (the paper never mentions grouped-query attention):
    the probe of a KV head is the arithmetic mean of the probes of its G query
    heads.  Reduces to Eq. 9 when G = 1.  [Hq, D] -> [Hkv, D]."""
    p = np.asarray(probe_qh, dtype=F64)
    hq, d = p.shape
    return p.reshape(n_kv_heads, hq // n_kv_heads, d).mean(axis=1)


# ----------------------------------------------------------------------------
# Step 6 (needed by step 3): cache append and block representatives (Eq. 4)
# ----------------------------------------------------------------------------
def build_representatives(k_block, n_repr: int, dtype: str, mode: str = "chunk_mean"):
    """PARITY UNPINNED (the paper only says a score is taken per chunk of 32 KV
    pairs).  Representative i of a block of B keys is

      chunk_mean:    the mean of the keys of tokens [i*B/r, (i+1)*B/r),
      strided_token: the key of token i*B/r + B/(2r),

    rounded to the cache's storage type.  k_block: [B, D] -> [r, D]."""
    kb = np.asarray(k_block, dtype=F64)
    b = kb.shape[0]
    seg = b // n_repr
    reps = np.empty((n_repr, kb.shape[1]), F64)
    for i in range(n_repr):
        if mode == "chunk_mean":
            reps[i] = kb[i * seg:(i + 1) * seg].sum(axis=0) / seg
        elif mode == "strided_token":
            reps[i] = kb[i * seg + seg // 2]
        else:
            raise ValueError(mode)
    return round_to_storage(reps, dtype)


def n_candidate_blocks(p0: int, n_init: int, block: int, n_local_prev: int = 0) -> int:
    """Blocks tile the past after the initial tokens: block b holds tokens
    [n_init + b*B, n_init + (b+1)*B).  Candidates are the complete blocks that
    end at or before p0 - n_local_prev."""
    return max(0, (p0 - n_local_prev - n_init) // block)


def representative_table(k_cache, n_blocks: int, n_init: int, block: int, n_repr: int,
                         dtype: str, mode: str = "chunk_mean") -> np.ndarray:
    """Representatives of blocks 0..n_blocks-1 of a token-major key cache
    [N, Hkv, D] -> [Hkv, n_blocks, r, D]."""
    kc = np.asarray(k_cache)
    hkv, d = kc.shape[1], kc.shape[2]
    tab = np.zeros((hkv, n_blocks, n_repr, d), F64)
    for g in range(hkv):
        for b in range(n_blocks):
            lo = n_init + b * block
            tab[g, b] = build_representatives(kc[lo:lo + block, g, :], n_repr, dtype, mode)
    return tab


def append_window(k_cache, v_cache, k_window, v_window):
    """Eq. 4: the cache after step t is the concatenation of the cache after
    step t-1 and the step's keys / values."""
    return (np.concatenate([k_cache, k_window], axis=0),
            np.concatenate([v_cache, v_window], axis=0))


# ----------------------------------------------------------------------------
# Step 3: cosine scores (Eq. 10) and information density (Eq. 11)
# ----------------------------------------------------------------------------
def cosine_scores(probe_kv, repr_table) -> np.ndarray:
    """Eq. 10 for every representative key:
    s = <probe, key> / (||probe|| * ||key||).  [Hkv, D], [Hkv, n, r, D] -> [Hkv, n, r].
    A zero-norm probe or key gives score 0."""
    p = np.asarray(probe_kv, dtype=F64)
    t = np.asarray(repr_table, dtype=F64)
    dots = np.einsum("gd,gnrd->gnr", p, t)
    pn = np.sqrt((p * p).sum(axis=1))
    tn = np.sqrt((t * t).sum(axis=3))
    den = pn[:, None, None] * tn
    return np.divide(dots, den, out=np.zeros_like(dots), where=den > 0)


def block_scores(probe_kv, repr_table, agg: str = "mean") -> np.ndarray:
    """PARITY UNPINNED aggregation: one score per block = mean (or max) of the
    cosines of its r representatives.  -> [Hkv, n]."""
    s = cosine_scores(probe_kv, repr_table)
    return s.mean(axis=2) if agg == "mean" else s.max(axis=2)


def information_density(scores, beta: float = 1.0) -> np.ndarray:
    """Eq. 11: entropy (natural log) of softmax(beta * s) over the n scores of
    one head; beta = 1 is the paper.  [Hkv, n] -> [Hkv].  n = 0 gives 0."""
    s = np.asarray(scores, dtype=F64)
    out = np.zeros(s.shape[0], F64)
    for g in range(s.shape[0]):
        if s.shape[1] == 0:
            continue
        e = np.exp(beta * s[g])
        p = e / e.sum()
        out[g] = -(p * np.log(p)).sum()
    return out


# ----------------------------------------------------------------------------
# Step 4: dynamic KV cut-off (Eq. 12) and top-c selection (Algorithm 1)
# ----------------------------------------------------------------------------
def round_half_up(x: float) -> int:
    return int(np.floor(x + 0.5))


class BudgetChain:
    """Eq. 12 processed shallow -> deep for one sequence.

    B^l = Theta^l / (Theta^l + sum_{j>l} ThetaBar^j) * B_kv,  B_kv <- B_kv - (granted),
    B_kv initialised to L*k at the first layer of every step.

    PARITY UNPINNED readings:
      * ThetaBar^j ("streaming"): the mean of layer j's Theta over the previous
        steps of this sequence; with no history yet, ThetaBar^j := Theta^l.
        ("alg1"): ThetaBar^j := Theta^j of the same step (Algorithm 1 computes
        every layer's Theta before any budget).
      * the granted count c^l is B^l rounded half up and clamped to
        [min(1, n), min(cap, n)]; the integer c^l is what is subtracted.
      * a non-positive denominator splits the remainder evenly over the
        remaining layers; a layer with n = 0 takes nothing.
    Theta values are taken as stored in fp32 (the precision they are handed
    over in); the chain itself is fp64.
    """

    def __init__(self, n_layers: int, k_blocks: int, cap_blocks: int, mode: str = "streaming"):
        self.L, self.k, self.cap, self.mode = n_layers, k_blocks, cap_blocks, mode
        self.b_rem = float(n_layers * k_blocks)
        self.theta_sum = np.zeros(n_layers, F64)
        self.theta_cnt = np.zeros(n_layers, np.int64)

    def real_budget(self, layer: int, theta_layer: float, theta_all=None) -> float:
        """Un-rounded B^l of Eq. 12 for 0-based `layer` given the remaining B_kv."""
        rest = 0.0
        for j in range(layer + 1, self.L):
            if self.mode == "alg1":
                rest += float(theta_all[j])
            elif self.theta_cnt[j] > 0:
                rest += self.theta_sum[j] / self.theta_cnt[j]
            else:
                rest += theta_layer
        den = theta_layer + rest
        if den > 0:
            return theta_layer / den * self.b_rem
        return self.b_rem / (self.L - layer)

    def grant(self, layer: int, theta_heads, n: int, theta_all=None):
        """Process one layer.  theta_heads: per-KV-head Theta (Eq. 11); the
        layer's density is their mean.  Returns (c, B_real, fragile) where
        fragile flags a rounding decision within 1e-4 of a boundary."""
        if layer == 0:
            self.b_rem = float(self.L * self.k)
        th = np.asarray(theta_heads, dtype=np.float32).astype(F64)
        theta_layer = float(th.mean()) if th.size else 0.0
        if n <= 0:
            return 0, 0.0, False
        b_real = self.real_budget(layer, theta_layer, theta_all)
        c = round_half_up(b_real)
        frac = (b_real + 0.5) - np.floor(b_real + 0.5)
        fragile = bool(min(frac, 1.0 - frac) < 1e-4)
        c = max(min(1, n), min(c, min(self.cap, n)))
        self.b_rem -= c
        self.theta_sum[layer] += theta_layer
        self.theta_cnt[layer] += 1
        return c, b_real, fragile


def select_blocks(scores_head, c: int, near_rel: float = 1e-3):
    """Algorithm 1, last loop, for one head: sort by score descending (softmax
    is monotone, so sorting by P equals sorting by s), keep the first c; equal
    scores keep the lower block index first; NaN sorts last.

    Returns (idx ascending int32 [c], tau = c-th largest score,
             near = blocks with |s - tau| <= near_rel * |tau|)."""
    s = np.asarray(scores_head, dtype=F64)
    n = s.shape[0]
    c = min(c, n)
    if c <= 0:
        return np.zeros(0, np.int32), np.nan, np.zeros(0, np.int32)
    key = np.where(np.isnan(s), -np.inf, s)
    order = np.argsort(-key, kind="stable")
    idx = np.sort(order[:c]).astype(np.int32)
    tau = key[order[c - 1]]
    with np.errstate(invalid="ignore"):
        near = np.nonzero(np.abs(key - tau) <= near_rel * abs(tau))[0].astype(np.int32)
    return idx, float(tau), near


# ----------------------------------------------------------------------------
# Step 5: attention over [initial | selected blocks | local] (Eq. 2 / Eq. 3)
# ----------------------------------------------------------------------------
def key_layout(p0: int, n_init: int, block: int, n_local_prev: int = 0):
    """(init_len, n, local_start): the past splits into initial tokens
    [0, init_len), n candidate blocks, and a local segment [local_start, p0).
    While p0 <= n_init there is no separate initial segment."""
    if p0 <= n_init:
        return 0, 0, 0
    n = n_candidate_blocks(p0, n_init, block, n_local_prev)
    return n_init, n, n_init + n * block


def past_key_positions(p0: int, sel_idx, n_init: int, block: int, n_local_prev: int = 0):
    """Absolute positions of the past tokens one KV head attends to."""
    init_len, _, local_start = key_layout(p0, n_init, block, n_local_prev)
    parts = [np.arange(init_len)]
    for b in np.asarray(sel_idx, dtype=np.int64):
        parts.append(n_init + b * block + np.arange(block))
    parts.append(np.arange(local_start, p0))
    return np.concatenate(parts).astype(np.int64)


def retrieval_attention(q_window, k_window, v_window, k_cache, v_cache, p0: int, sel_idx_per_head,
                        n_init: int, block: int, n_local_prev: int = 0, sm_scale=None):
    """Eq. 2 (Eq. 3 when the step has one token): softmax(q k^T / sqrt(D)) v of
    every query of the step over
        [initial tokens | selected blocks of its KV head | local past | step tokens <= itself]
    with one normalisation over the union.

    q_window [n, Hq, D]; k_window, v_window [n, Hkv, D]; k_cache, v_cache
    token-major [>=p0, Hkv, D]; sel_idx_per_head: list of Hkv index arrays.
    Returns (O [n, Hq, D], lse [Hq, n])."""
    q = np.asarray(q_window, dtype=F64)
    kw = np.asarray(k_window, dtype=F64)
    vw = np.asarray(v_window, dtype=F64)
    nt, hq, d = q.shape
    hkv = kw.shape[1]
    grp = hq // hkv
    scale = 1.0 / np.sqrt(d) if not sm_scale else sm_scale
    out = np.zeros((nt, hq, d), F64)
    lse = np.zeros((hq, nt), F64)
    causal = np.tril(np.ones((nt, nt), bool))
    for g in range(hkv):
        pos = past_key_positions(p0, sel_idx_per_head[g], n_init, block, n_local_prev)
        kp = np.asarray(k_cache[pos, g, :], dtype=F64)
        vp = np.asarray(v_cache[pos, g, :], dtype=F64)
        keys = np.concatenate([kp, kw[:, g, :]], axis=0)
        vals = np.concatenate([vp, vw[:, g, :]], axis=0)
        mask = np.concatenate([np.ones((nt, pos.shape[0]), bool), causal], axis=1)
        for h in range(g * grp, (g + 1) * grp):
            s = (q[:, h, :] @ keys.T) * scale
            s = np.where(mask, s, -np.inf)
            m = s.max(axis=1, keepdims=True)
            e = np.exp(s - m)
            z = e.sum(axis=1, keepdims=True)
            out[:, h, :] = (e / z) @ vals
            lse[h] = (m + np.log(z))[:, 0]
    return out, lse


def full_causal_attention(q_window, k_all, v_all, p0: int, sm_scale=None) -> np.ndarray:
    """Eq. 1 by brute force, one query at a time: the query at absolute position
    p attends to every token 0..p of the full cache.  k_all, v_all: [>= p0+n, Hkv, D]."""
    q = np.asarray(q_window, dtype=F64)
    nt, hq, d = q.shape
    hkv = k_all.shape[1]
    grp = hq // hkv
    scale = 1.0 / np.sqrt(d) if not sm_scale else sm_scale
    out = np.zeros((nt, hq, d), F64)
    for j in range(nt):
        p = p0 + j
        for h in range(hq):
            g = h // grp
            logits = np.asarray(k_all[:p + 1, g, :], F64) @ q[j, h] * scale
            w = np.exp(logits - logits.max())
            w /= w.sum()
            out[j, h] = w @ np.asarray(v_all[:p + 1, g, :], F64)
    return out


# ----------------------------------------------------------------------------
# the whole per-window path, in the paper's order, for one (sequence, layer)
# ----------------------------------------------------------------------------
class LayerState:
    """Oracle-side state of one (sequence, layer): running query statistics and
    the token-major cache."""

    def __init__(self, n_q_heads, n_kv_heads, head_dim):
        self.stats = RunningStats(n_q_heads, head_dim)
        self.k_cache = np.zeros((0, n_kv_heads, head_dim), np.float32)
        self.v_cache = np.zeros((0, n_kv_heads, head_dim), np.float32)


def window_retrieval(state: LayerState, chain: BudgetChain, layer: int, q, k, v, *, n_init, block,
                     n_repr, dtype, n_local_prev=0, beta=1.0, var_eps=1e-12, repr_mode="chunk_mean",
                     agg="mean", attention=True, stats_mode="cumulative", theta_all=None,
                     repr_table=None, probe_mode="activation"):
    """One step of the path for one layer: bias -> probe -> score -> cut-off /
    select -> attention -> append.  Returns a dict of every intermediate.

    probe_mode "activation" is Eq. 9; "mean_pool" is the uniform-weight probe the
    paper compares against (Sec. 1, and the ablation of Sec. 5.3)."""
    p0 = state.k_cache.shape[0]
    hkv = k.shape[1]
    if stats_mode == "cumulative":
        state.stats.update(q)
        zbar, sigma2 = state.stats.mean, state.stats.variance()
    else:
        zbar, sigma2 = query_stats_two_pass(q)
    phi, a = activation_bias(q, zbar, sigma2, var_eps)
    if probe_mode == "activation":
        pq = probe_query(q, a)
    elif probe_mode == "mean_pool":
        pq = mean_pool_probe(q)
    else:
        raise ValueError(probe_mode)
    pkv = kv_head_probe(pq, hkv)
    n = n_candidate_blocks(p0, n_init, block, n_local_prev) if p0 > n_init else 0
    if repr_table is None:
        repr_table = representative_table(state.k_cache, n, n_init, block, n_repr, dtype, repr_mode)
    s = block_scores(pkv, repr_table[:, :n], agg)
    theta = information_density(s, beta)
    c, b_real, fragile = chain.grant(layer, theta, n, theta_all)
    sel, taus, nears = [], [], []
    for g in range(hkv):
        idx, tau, near = select_blocks(s[g], c)
        sel.append(idx)
        taus.append(tau)
        nears.append(near)
    res = dict(p0=p0, n=n, zbar=zbar, sigma2=sigma2, phi=phi, phi_l1=a, probe_qh=pq, probe_kv=pkv,
               scores=s, theta=theta, c=c, b_real=b_real, fragile=fragile, sel=sel, tau=taus,
               near=nears, repr_table=repr_table)
    if attention:
        o, lse = retrieval_attention(q, k, v, state.k_cache, state.v_cache, p0, sel, n_init, block,
                                     n_local_prev)
        res["out"], res["lse"] = o, lse
    state.k_cache, state.v_cache = append_window(state.k_cache, state.v_cache, k, v)
    return res
