"""Pins for the CPU oracle: every function is checked against something other
than itself -- library routines, closed forms that follow from the paper's
equations, brute force on tiny inputs, and the constants the paper prints."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import actqkv_oracle as orc
from paper_2502_13542_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")


def golden():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                k, v = line.split()
                out[k] = float(v)
    return out


def rng(seed=0):
    return np.random.default_rng(seed)


# ---------------------------------------------------------------- storage rounding
def test_bf16_rounding_matches_torch():
    import torch
    x = rng(1).standard_normal(20000).astype(np.float32) * np.float32(7.0)
    x[:6] = [0.0, 1.0, 1.00390625, 1.01171875, -3.0e-5, 65504.0]   # incl. exact ties
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(orc.round_to_bf16(x).astype(np.float32), want)
    assert np.array_equal(wl.bf16_grid(x), want)


# ---------------------------------------------------------------- Eq. 8 statistics
def test_stats_equal_numpy_mean_var_over_concatenation():
    g = rng(2)
    wins = [g.standard_normal((37, 3, 5)) * 3 + 1.5 for _ in range(4)]
    allq = np.concatenate(wins)
    zbar, s2 = orc.query_stats_two_pass(allq)
    assert np.allclose(zbar, np.mean(allq, axis=0), rtol=1e-13, atol=1e-13)
    assert np.allclose(s2, np.var(allq, axis=0, ddof=1), rtol=1e-12)
    # the divisor is m*t - 1 (unbiased), not m*t
    assert not np.allclose(s2, np.var(allq, axis=0, ddof=0), rtol=1e-4)


def test_running_stats_equal_two_pass_at_every_window():
    g = rng(3)
    st = orc.RunningStats(2, 4)
    hist = []
    for t in range(6):
        w = g.standard_normal((16 + t, 2, 4)) * (1 + t) + 100.0     # large offset: cancellation trap
        hist.append(w)
        st.update(w)
        zbar, s2 = orc.query_stats_two_pass(np.concatenate(hist))
        assert st.count == sum(h.shape[0] for h in hist)
        assert np.allclose(st.mean, zbar, rtol=1e-13)
        assert np.allclose(st.variance(), s2, rtol=1e-11)


# ---------------------------------------------------------------- Eq. 7 activation bias
def test_bias_closed_form_first_window():
    """At t = 1 the statistics are the window's own, so for each channel
    sum_j phi_j = sum_j (q_j - mean)^2 / (sum_j (q_j - mean)^2 / (m-1)) = m - 1,
    hence ||Phi||_1 = D * (m - 1)."""
    m, hq, d = 64, 3, 8
    q = rng(4).standard_normal((m, hq, d)) * 5 - 2
    zbar, s2 = orc.query_stats_two_pass(q)
    phi, a = orc.activation_bias(q, zbar, s2)
    assert np.all(phi >= 0)
    assert np.allclose(phi.sum(axis=0), m - 1, rtol=1e-12)
    assert np.allclose(a.sum(axis=0), d * (m - 1), rtol=1e-12)


def test_bias_matches_scalar_loops():
    m, hq, d = 5, 2, 3
    g = rng(5)
    hist = g.standard_normal((2 * m, hq, d))
    q = hist[m:]
    zbar, s2 = orc.query_stats_two_pass(hist)
    phi, a = orc.activation_bias(q, zbar, s2)
    for j in range(m):
        for h in range(hq):
            tot = 0.0
            for c in range(d):
                mean = sum(hist[i, h, c] for i in range(2 * m)) / (2 * m)
                var = sum((hist[i, h, c] - mean) ** 2 for i in range(2 * m)) / (2 * m - 1)
                want = (q[j, h, c] - mean) ** 2 / var
                assert math.isclose(phi[j, h, c], want, rel_tol=1e-12)
                tot += want
            assert math.isclose(a[j, h], tot, rel_tol=1e-12)


def test_bias_and_weights_invariant_to_per_channel_affine_map():
    """phi is a squared z-score, so q_c -> alpha_c q_c + beta_c leaves phi and the
    Eq. 9 weights unchanged: scaling outlier channels must not change the weights."""
    m, hq, d = 40, 2, 6
    g = rng(6)
    q = g.standard_normal((m, hq, d))
    alpha = g.uniform(0.5, 10.0, (hq, d)) * g.choice([-1, 1], (hq, d))
    beta = g.standard_normal((hq, d)) * 4
    q2 = q * alpha[None] + beta[None]
    p1, a1 = orc.activation_bias(q, *orc.query_stats_two_pass(q))
    p2, a2 = orc.activation_bias(q2, *orc.query_stats_two_pass(q2))
    assert np.allclose(p1, p2, rtol=1e-9, atol=1e-12)
    assert np.allclose(orc.probe_weights(a1), orc.probe_weights(a2), rtol=1e-9)


def test_bias_variance_floor_and_zero_total():
    q = np.ones((4, 1, 2))
    zbar, s2 = orc.query_stats_two_pass(q)
    phi, a = orc.activation_bias(q, zbar, s2)
    assert np.all(phi == 0) and np.all(a == 0)
    assert np.allclose(orc.probe_weights(a), 0.25)          # uniform fallback


# ---------------------------------------------------------------- Eq. 9 probe-query
def test_probe_weights_sum_to_one_and_probe_in_box():
    m, hq, d = 50, 4, 8
    q = rng(7).standard_normal((m, hq, d)) * 3
    _, a = orc.activation_bias(q, *orc.query_stats_two_pass(q))
    w = orc.probe_weights(a)
    assert np.all(w >= 0) and np.allclose(w.sum(axis=0), 1.0, rtol=1e-13)
    p = orc.probe_query(q, a)
    assert np.all(p <= q.max(axis=0) + 1e-12) and np.all(p >= q.min(axis=0) - 1e-12)
    # scalar restatement of Eq. 9
    for h in range(hq):
        norm_phi = sum(a[j, h] for j in range(m))
        want = sum(a[j, h] / norm_phi * q[j, h] for j in range(m))
        assert np.allclose(p[h], want, rtol=1e-12)


def test_probe_two_tokens_is_plain_mean():
    """m = 2, t = 1: both tokens are equally far from their mean, phi_1 = phi_2."""
    q = rng(8).standard_normal((2, 3, 5))
    _, a = orc.activation_bias(q, *orc.query_stats_two_pass(q))
    assert np.allclose(orc.probe_query(q, a), q.mean(axis=0), rtol=1e-12)
    assert np.allclose(orc.probe_query(q, a), orc.mean_pool_probe(q), rtol=1e-12)


def test_probe_concentrates_on_the_anchor_token():
    """Identical queries except one: the odd token is the farthest from the mean
    (the anchor-token criterion, Eq. 6) and takes most of the weight."""
    m, d = 32, 8
    q = np.tile(rng(9).standard_normal((1, 1, d)), (m, 1, 1))
    q[5, 0] += 3.0
    _, a = orc.activation_bias(q, *orc.query_stats_two_pass(q))
    w = orc.probe_weights(a)[:, 0]
    # closed form: deviation of the odd one is (m-1)/m * delta, others delta/m
    want_odd = (m - 1) ** 2 / ((m - 1) ** 2 + (m - 1))
    assert math.isclose(w[5], want_odd, rel_tol=1e-9)
    assert np.argmax(w) == 5 and w[5] > 0.9
    mean_cos = lambda p: p @ q[5, 0] / np.linalg.norm(p) / np.linalg.norm(q[5, 0])
    assert mean_cos(orc.probe_query(q, a)[0]) > mean_cos(orc.mean_pool_probe(q)[0])


def test_kv_head_probe_groups_consecutive_heads():
    p = np.arange(8 * 3, dtype=float).reshape(8, 3)
    kv = orc.kv_head_probe(p, 2)
    assert np.allclose(kv[0], p[0:4].mean(axis=0)) and np.allclose(kv[1], p[4:8].mean(axis=0))
    assert np.allclose(orc.kv_head_probe(p, 8), p)             # G = 1: Eq. 9 itself


# ---------------------------------------------------------------- Eq. 10 cosine scores
def test_cosine_known_values_and_invariances():
    probe = np.array([[1.0, 0.0], [0.0, 2.0]])
    tab = np.zeros((2, 3, 1, 2))
    tab[0, :, 0] = [[1, 1], [0, 5], [-2, 0]]
    tab[1, :, 0] = [[1, 1], [0, 5], [3, -4]]
    s = orc.cosine_scores(probe, tab)[:, :, 0]
    want = np.array([[1 / math.sqrt(2), 0.0, -1.0], [1 / math.sqrt(2), 1.0, -0.8]])
    assert np.allclose(s, want, rtol=1e-14, atol=1e-15)
    g = rng(10)
    p = g.standard_normal((2, 16))
    t = g.standard_normal((2, 7, 4, 16))
    s0 = orc.cosine_scores(p, t)
    assert np.all(np.abs(s0) <= 1 + 1e-12)
    assert np.allclose(orc.cosine_scores(3.7 * p, 0.2 * t), s0, rtol=1e-12)
    t[1, 3, 2] = 5.0 * p[1]
    assert math.isclose(orc.cosine_scores(p, t)[1, 3, 2], 1.0, rel_tol=1e-12)
    # scipy's cosine distance as the library routine
    from scipy.spatial.distance import cosine
    assert math.isclose(s0[0, 4, 1], 1.0 - cosine(p[0], t[0, 4, 1]), rel_tol=1e-10)
    assert np.allclose(orc.block_scores(p, t, "mean"), orc.cosine_scores(p, t).mean(axis=2))
    assert np.allclose(orc.block_scores(p, t, "max"), orc.cosine_scores(p, t).max(axis=2))


# ---------------------------------------------------------------- Eq. 11 information density
def test_density_uniform_bounds_library_and_paper_perplexity():
    gold = golden()
    n = int(gold["chunks"])
    th = orc.information_density(np.full((1, n), 0.37))
    assert math.isclose(th[0], math.log(n), rel_tol=1e-13)       # uniform -> ln n (the maximum)
    assert math.isclose(math.exp(th[0]), gold["uniform_perplexity"], rel_tol=1e-12)
    from scipy.special import softmax
    from scipy.stats import entropy
    s = rng(11).uniform(-1, 1, (3, n))
    th = orc.information_density(s)
    for g in range(3):
        assert math.isclose(th[g], entropy(softmax(s[g])), rel_tol=1e-12)
        assert 0 <= th[g] <= math.log(n)
        # cosines live in [-1, 1]: the softmax stays close to uniform, perplexity near 46
        assert 0.8 * n < math.exp(th[g]) < n
    sharp = np.zeros((1, n)); sharp[0, 3] = 60.0
    assert orc.information_density(sharp)[0] < 1e-20 + 1e-10
    assert math.isclose(orc.information_density(s, beta=0.0)[0], math.log(n), rel_tol=1e-13)
    assert orc.information_density(s, beta=32.0)[0] < th[0]


# ---------------------------------------------------------------- Eq. 12 budget
def test_paper_budget_constants():
    g = golden()
    assert g["sinks"] + g["local"] + g["retrieved_k"] == g["reused_kv"]
    assert g["chunks"] * g["pairs_per_chunk"] == g["retrieved_k"]


def test_budget_single_layer_and_equal_density():
    ch = orc.BudgetChain(1, 32, 32)
    assert ch.grant(0, [5.1, 5.2], 251)[0] == 32                # L = 1: B^1 = B_kv = k
    ch = orc.BudgetChain(8, 10, 20)
    for step in range(3):
        cs = [ch.grant(l, [4.0, 4.0], 500)[0] for l in range(8)]
        assert cs == [10] * 8                                     # equal density: k each


def test_budget_telescopes_to_L_times_k():
    g = rng(12)
    L, k = 12, 16
    ch = orc.BudgetChain(L, k, 10_000)
    for step in range(5):
        cs = [ch.grant(l, g.uniform(1.0, 6.0, 4), 100_000)[0] for l in range(L)]
        assert sum(cs) == L * k                                  # last layer's ratio is 1
        assert ch.b_rem == 0


def test_budget_alg1_closed_form_and_log_base():
    """With every layer's Theta known (Algorithm 1) and real-valued subtraction,
    Eq. 12 telescopes to B^l = L*k*Theta^l / sum_j Theta^j; the ratio does not
    depend on the log base."""
    g = rng(13)
    L, k = 6, 20
    theta = g.uniform(2.0, 5.0, L)
    for base_scale in (1.0, 1.0 / math.log(2.0)):
        th = theta * base_scale
        ch = orc.BudgetChain(L, k, 10_000, mode="alg1")
        for l in range(L):
            b = ch.real_budget(l, th[l], th)
            assert math.isclose(b, L * k * theta[l] / theta.sum(), rel_tol=1e-12)
            ch.b_rem -= b                                          # the paper's real-valued update
        assert abs(ch.b_rem) < 1e-9


def test_budget_streaming_uses_history_mean_and_clamps():
    L, k, cap = 3, 10, 12
    ch = orc.BudgetChain(L, k, cap)
    first = [ch.grant(l, [t], 100)[0] for l, t in enumerate([1.0, 4.0, 7.0])]
    # no history: ThetaBar := current Theta -> B = B_rem / (layers left)
    assert first == [10, 10, 10]
    # second step: history means are (1, 4, 7)
    c0, real0, _ = ch.grant(0, [1.0], 100)
    assert math.isclose(real0, 1.0 / (1.0 + 4.0 + 7.0) * 30) and c0 == 3     # 2.5 rounds half up
    c1, real1, _ = ch.grant(1, [4.0], 100)
    assert math.isclose(real1, 4.0 / (4.0 + 7.0) * 27) and c1 == 10
    c2, real2, _ = ch.grant(2, [7.0], 100)
    assert math.isclose(real2, 17.0) and c2 == cap                            # cap binds
    # third step: history means are still (1, 4, 7); a denser first layer takes more
    c0, real0, _ = ch.grant(0, [3.0], 100)
    assert math.isclose(real0, 3.0 / (3.0 + 4.0 + 7.0) * 30) and c0 == 6
    assert orc.BudgetChain(2, 5, 9).grant(0, [3.0], 0)[0] == 0   # n = 0 takes nothing
    assert orc.BudgetChain(2, 5, 9).grant(0, [3.0], 2)[0] == 2   # n < budget
    assert orc.BudgetChain(2, 5, 9).grant(0, [0.0], 1)[0] == 1   # zero density, n = 1
    assert orc.round_half_up(2.5) == 3 and orc.round_half_up(2.4999) == 2


# ---------------------------------------------------------------- Eq. 5 / Alg. 1 selection
def test_selection_is_the_argmax_subset_of_eq5():
    g = rng(14)
    for n in range(1, 9):
        s = g.standard_normal(n)
        for c in range(1, n + 1):
            idx, tau, _ = orc.select_blocks(s, c)
            best = max(itertools.combinations(range(n), c), key=lambda I: sum(s[list(I)]))
            assert list(idx) == sorted(best)
            assert tau == sorted(s)[::-1][c - 1]


def test_selection_ties_nan_and_overflow():
    s = np.array([0.5, 0.9, 0.5, 0.5, np.nan, 0.1])
    idx, tau, near = orc.select_blocks(s, 3)
    assert list(idx) == [0, 1, 2] and tau == 0.5                # equal scores: lower index first
    assert list(near) == [0, 2, 3]
    assert list(orc.select_blocks(s, 99)[0]) == [0, 1, 2, 3, 4, 5]
    assert list(orc.select_blocks(s, 5)[0]) == [0, 1, 2, 3, 5]  # NaN last
    assert orc.select_blocks(s, 0)[0].size == 0
    big = rng(15).standard_normal(1000)
    idx, _, _ = orc.select_blocks(big, 37)
    assert list(idx) == sorted(np.argsort(-big, kind="stable")[:37])


# ---------------------------------------------------------------- Eq. 4 append / representatives
def test_representatives_and_table():
    g = rng(16)
    kb = g.standard_normal((128, 16))
    reps = orc.build_representatives(kb, 4, "f32")
    want = kb.reshape(4, 32, 16).mean(axis=1).astype(np.float32)
    assert np.array_equal(reps.astype(np.float32), want)
    import torch
    want16 = torch.from_numpy(kb.reshape(4, 32, 16).mean(axis=1)).to(torch.bfloat16).double().numpy()
    assert np.array_equal(orc.build_representatives(kb, 4, "bf16"), want16)
    st = orc.build_representatives(kb, 4, "f32", "strided_token")
    assert np.array_equal(st.astype(np.float32), kb[[16, 48, 80, 112]].astype(np.float32))
    cache = g.standard_normal((64 + 3 * 128 + 17, 2, 16))
    tab = orc.representative_table(cache, 3, 64, 128, 4, "f32")
    assert tab.shape == (2, 3, 4, 16)
    assert np.allclose(tab[1, 2, 3], cache[64 + 2 * 128 + 96: 64 + 3 * 128, 1].mean(axis=0), atol=1e-6)
    assert orc.n_candidate_blocks(3840, 64, 128) == 29
    assert orc.n_candidate_blocks(32256, 128, 128) == 251
    assert orc.n_candidate_blocks(130560, 128, 128) == 1019
    assert orc.n_candidate_blocks(100, 128, 128) == 0
    assert orc.n_candidate_blocks(32768, 128, 128, 512) == 251
    k2, v2 = orc.append_window(cache, cache * 2, cache[:5] + 1, cache[:5] + 2)
    assert k2.shape[0] == cache.shape[0] + 5 and np.array_equal(k2[-5:], cache[:5] + 1)
    assert np.array_equal(v2[:-5], cache * 2) and np.array_equal(v2[-5:], cache[:5] + 2)


# ---------------------------------------------------------------- Eq. 2 / Eq. 3 attention
def _tiny_attention_case(seed, p0, nt, n_init=8, block=4, hq=4, hkv=2, d=8, n_local_prev=0):
    g = rng(seed)
    q = g.standard_normal((nt, hq, d))
    k = g.standard_normal((p0 + nt, hkv, d))
    v = g.standard_normal((p0 + nt, hkv, d))
    n = orc.n_candidate_blocks(p0, n_init, block, n_local_prev) if p0 > n_init else 0
    return q, k, v, n


@pytest.mark.parametrize("p0,nt,nlp", [(0, 6, 0), (5, 6, 0), (8, 6, 0), (30, 6, 0), (31, 1, 0), (40, 3, 7)])
def test_attention_with_all_blocks_equals_full_causal_attention(p0, nt, nlp):
    """When the selection covers every candidate block the key set is the whole
    past, so Eq. 2 must equal Eq. 1 (brute force over the full cache)."""
    q, k, v, n = _tiny_attention_case(20 + p0, p0, nt, n_local_prev=nlp)
    sel = [np.arange(n), np.arange(n)[::-1].copy()]             # order of blocks is irrelevant
    o, lse = orc.retrieval_attention(q, k[p0:], v[p0:], k[:p0], v[:p0], p0, sel, 8, 4, nlp)
    want = orc.full_causal_attention(q, k, v, p0)
    assert np.allclose(o, want, rtol=1e-11, atol=1e-13)
    # softmax rows sum to one: exp(logit - lse) over the key set
    for h in range(4):
        for j in range(nt):
            logits = k[:p0 + j + 1, h // 2] @ q[j, h] / math.sqrt(8)
            assert math.isclose(np.exp(logits - lse[h, j]).sum(), 1.0, rel_tol=1e-11)


def test_attention_subset_matches_loop_over_explicit_key_set():
    p0, nt, n_init, block = 45, 4, 8, 4
    q, k, v, n = _tiny_attention_case(31, p0, nt)
    assert n == 9
    sel = [np.array([1, 4, 7]), np.array([0, 8])]
    o, _ = orc.retrieval_attention(q, k[p0:], v[p0:], k[:p0], v[:p0], p0, sel, n_init, block)
    for j in range(nt):
        for h in range(4):
            g = h // 2
            keys = set(range(n_init)) | set(range(n_init + n * block, p0 + j + 1))
            for b in sel[g]:
                keys |= set(range(n_init + b * block, n_init + (b + 1) * block))
            keys = sorted(keys)
            lg = np.array([k[t, g] @ q[j, h] for t in keys]) / math.sqrt(8)
            w = np.exp(lg - lg.max()); w /= w.sum()
            want = sum(wi * v[t, g] for wi, t in zip(w, keys))
            assert np.allclose(o[j, h], want, rtol=1e-11, atol=1e-13)
            assert np.all(o[j, h] <= v[keys, g].max(axis=0) + 1e-12)
            assert np.all(o[j, h] >= v[keys, g].min(axis=0) - 1e-12)


def test_attention_single_key_returns_its_value():
    g = rng(33)
    q = g.standard_normal((1, 2, 4)); k = g.standard_normal((1, 1, 4)); v = g.standard_normal((1, 1, 4))
    o, _ = orc.retrieval_attention(q, k, v, k[:0], v[:0], 0, [np.zeros(0, int)], 8, 4)
    assert np.allclose(o[0, 0], v[0, 0]) and np.allclose(o[0, 1], v[0, 0])


# ---------------------------------------------------------------- the generator and the whole path
def test_workload_generator_is_seeded_and_windowed():
    sp = wl.tiny_pr1()
    assert np.array_equal(wl.gen_q(sp, 0, 3), wl.gen_q(sp, 0, 3))
    assert not np.array_equal(wl.gen_q(sp, 0, 3), wl.gen_q(sp, 0, 4))
    cq, ck = wl.outlier_channels(sp, 0)
    q = wl.gen_q(sp, 0, 1)
    for h in range(sp.n_q_heads):
        std = q[:, h].std(axis=0)
        assert set(np.argsort(-std)[:sp.n_outlier]) == set(cq[h])
    pb = wl.planted_blocks(sp, 0)
    assert pb.shape == (2, 3) and pb.max() < 29
    sp2 = wl.llama3_8b_layer()
    q2 = wl.gen_q(sp2, 0, 0)
    assert np.array_equal(q2, wl.bf16_grid(q2))                  # already on the bf16 grid
    pt = wl.shuffled_page_table(sp2, 4096)
    assert sorted(pt) == list(range(256)) and list(pt) != list(range(256))
    x = rng(40).standard_normal((100, 8, 128)).astype(np.float32)
    pages = wl.to_pages(sp2, x, pt, 256)
    assert np.array_equal(pages[pt[3], 5, 7], x[3 * 16 + 7, 5])
    ctx = wl.decode_contexts(wl.decode_batch16())
    assert ctx.shape == (16,) and ctx.min() >= 32768 and ctx.max() <= 131072


def test_planted_block_recall_tiny_config():
    """End to end on the tiny config: at the target (last) window the planted
    blocks are all retrieved under chunk-mean representatives, and the path with
    a budget covering every block equals full causal attention."""
    sp = wl.tiny_pr1()
    st = orc.LayerState(sp.n_q_heads, sp.n_kv_heads, sp.head_dim)
    ch = orc.BudgetChain(1, sp.k_blocks, sp.cap_blocks)
    res = None
    for t in range(sp.n_windows):
        q = wl.gen_q(sp, 0, t)
        k, v = wl.gen_kv(sp, 0, t)
        last = t == sp.n_windows - 1
        res = orc.window_retrieval(st, ch, 0, q, k, v, n_init=sp.n_init, block=sp.block,
                                   n_repr=sp.n_repr, dtype=sp.dtype, attention=last)
        assert res["n"] == wl.n_candidates(sp, t * sp.window)
        assert res["c"] == min(sp.k_blocks, res["n"])
    assert res["n"] == 29
    pb = wl.planted_blocks(sp, 0)
    for g in range(sp.n_kv_heads):
        assert set(pb[g]) <= set(res["sel"][g]), (pb[g], res["sel"][g], res["scores"][g])
        planted_min = res["scores"][g][pb[g]].min()
        others = np.delete(res["scores"][g], pb[g])
        assert planted_min > others.max()
    # budget covering all blocks == brute-force causal attention over the whole context
    p0 = res["p0"]
    q = wl.gen_q(sp, 0, sp.n_windows - 1)[:24]
    k, v = wl.gen_kv(sp, 0, sp.n_windows - 1)
    allsel = [np.arange(29)] * sp.n_kv_heads
    o, _ = orc.retrieval_attention(q, k[:24], v[:24], st.k_cache[:p0], st.v_cache[:p0], p0, allsel,
                                   sp.n_init, sp.block)
    want = orc.full_causal_attention(q, st.k_cache, st.v_cache, p0)
    assert np.allclose(o, want, rtol=1e-10, atol=1e-12)


def test_window_retrieval_variant_switches_reduce_to_library_routines():
    """The switches of the whole-path function: window-only statistics are numpy's mean and
    unbiased variance of the CURRENT window alone (no history), and the mean-pooling probe
    (Sec. 1 of the paper: the probe its baselines use) is numpy's mean over the window's tokens
    followed by the mean over each KV head's group of query heads."""
    sp = wl.tiny_pr1()
    for stats_mode, probe_mode in (("window_only", "activation"), ("cumulative", "mean_pool")):
        st = orc.LayerState(sp.n_q_heads, sp.n_kv_heads, sp.head_dim)
        ch = orc.BudgetChain(1, sp.k_blocks, sp.cap_blocks)
        for t in range(3):
            q = wl.gen_q(sp, 0, t)
            k, v = wl.gen_kv(sp, 0, t)
            res = orc.window_retrieval(st, ch, 0, q, k, v, n_init=sp.n_init, block=sp.block, n_repr=sp.n_repr,
                                       dtype=sp.dtype, attention=False, stats_mode=stats_mode,
                                       probe_mode=probe_mode)
        q64 = q.astype(np.float64)
        if stats_mode == "window_only":
            assert np.allclose(res["zbar"], q64.mean(axis=0), rtol=1e-12, atol=1e-14)
            assert np.allclose(res["sigma2"], q64.var(axis=0, ddof=1), rtol=1e-12)
            assert st.stats.count == 0                      # the running statistics are left alone
        else:
            hist = np.concatenate([wl.gen_q(sp, 0, i) for i in range(3)]).astype(np.float64)
            assert np.allclose(res["sigma2"], hist.var(axis=0, ddof=1), rtol=1e-12)
        if probe_mode == "mean_pool":
            want_qh = q64.mean(axis=0)
            assert np.allclose(res["probe_qh"], want_qh, rtol=1e-12, atol=1e-14)
            want_kv = want_qh.reshape(sp.n_kv_heads, sp.group, sp.head_dim).mean(axis=1)
            assert np.allclose(res["probe_kv"], want_kv, rtol=1e-12, atol=1e-14)
        else:
            assert not np.allclose(res["probe_qh"], q64.mean(axis=0), rtol=1e-3)   # Eq. 9 is not a plain mean here


def test_one_token_probe_is_the_query_itself():
    """Decode (Sec. 4.2): with a single token Eq. 9 has one term of weight 1, whatever phi is."""
    q = rng(3).standard_normal((1, 4, 8))
    for a in (np.ones((1, 4)), np.full((1, 4), 7.5), np.zeros((1, 4))):
        assert np.allclose(orc.probe_query(q, a), q[0], rtol=0, atol=0)
