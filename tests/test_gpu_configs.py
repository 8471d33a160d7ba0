"""GPU parity on the larger workload shapes: the 32-layer stack with the budget chain running over
real scores, the 131072-token sweep, and batched single-token decode with fixed probes.  Every
intermediate that is cheap for the oracle is compared at every step; attention on stated samples."""
import numpy as np
import pytest

from oracle import actqkv_oracle as orc
from paper_2502_13542_b200 import workloads as wl
from tests import parity_utils as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import torch
    assert torch.cuda.is_available()
    from paper_2502_13542_b200 import binding
    return binding


def _stack(B, spec, beta, attention_layers, check_windows=None):
    """All layers of `spec` batched in one call per stage (n_seq = 1, n_layers = L): layer l's
    budget depends on what the shallower layers were granted (Eq. 12)."""
    import torch
    L = spec.n_layers
    cfg = B.make_config(spec, beta=beta, out_dtype=B.F32)
    pt = wl.shuffled_page_table(spec, spec.context)
    st = B.RetrievalState(cfg, n_seq=1, n_layers=L, page_table=pt[None, :])
    chain = orc.BudgetChain(L, spec.k_blocks, spec.cap_blocks, "streaming")
    runners = [pu.OracleRunner(spec, layer=l, chain=chain, beta=beta) for l in range(L)]
    out = torch.zeros(L, spec.window, spec.n_q_heads, spec.head_dim, dtype=torch.float32, device="cuda")
    counts = []
    for t in range(spec.n_windows):
        qs, ks, vs, res = [], [], [], []
        last = t == spec.n_windows - 1
        for l in range(L):
            q = wl.gen_q(spec, l, t)
            k, v = wl.gen_kv(spec, l, t)
            qs.append(q); ks.append(k); vs.append(v)
            res.append(runners[l].step(q, k, v, attention=last and l in attention_layers))
        st.step(pu.to_device(np.stack(qs), spec), pu.to_device(np.stack(ks), spec),
                pu.to_device(np.stack(vs), spec), out)
        torch.cuda.synchronize()
        assert int(st.status.item()) == 0
        if check_windows is not None and t not in check_windows:
            continue
        got_c = st.sel_count.cpu().numpy().tolist()
        want_c = [r["c"] for r in res]
        fragile = [r["fragile"] for r in res]
        tag = f"{spec.name} beta={beta} window {t}"
        n = res[0]["n"]
        if n:
            for l in range(L):
                pu.assert_rel(pu.to_numpy(st.scores[l, :, :n]), res[l]["scores"], 1.0, f"{tag} layer {l} scores")
                pu.assert_rel(pu.to_numpy(st.theta[l]), res[l]["theta"], 1e-30, f"{tag} layer {l} theta")
        if not any(fragile):
            assert got_c == want_c, tag
            for l in range(L):
                assert pu.compare_selection(pu.to_numpy(st.sel_idx[l]).astype(np.int64), got_c[l], res[l],
                                            f"{tag} layer {l}") >= 0
                if last and l in attention_layers:
                    pu.assert_attention(pu.to_numpy(out[l]), res[l]["out"], f"{tag} layer {l} attention")
        counts.append((n, want_c))
    assert abs(float(st.budget_state[0, 0]) - chain.b_rem) < 1e-9
    return counts


def test_tiny_stack32_paper_temperature(B):
    """32 layers of the tiny shape at beta = 1 (the paper): the densities of the layers are close,
    the counts stay near k, and they add up to L * k whenever no clamp binds."""
    spec = wl.tiny_stack32()
    counts = _stack(B, spec, 1.0, attention_layers={0, 31})
    unclamped = [c for n, c in counts if n >= spec.cap_blocks and max(c) < spec.cap_blocks]
    assert unclamped and all(sum(c) == spec.n_layers * spec.k_blocks for c in unclamped)
    print("tiny stack, beta = 1: per-layer counts at the last window", counts[-1][1])


def test_llama_stack32_32k_paper_and_sharpened_temperature(B):
    """The 32-layer stack at its stated size: LLaMA3-8B shape, context 32768 (64 windows), k = 32,
    cap 64, all layers batched per call, at beta = 1 (the paper's softmax) AND beta = 32 (counts
    vary by layer and hit the cap).  Both temperatures share the bias / probe / score stages (they
    do not depend on beta); the beta = 32 cut-off runs on a second set of selection buffers.
    Scores and densities at every checked window (every 4th, the first two and the last), counts
    at every window, block sets at the checked ones, tensor-core attention of the last window on
    layers {0, 13, 31} for both temperatures."""
    import torch
    spec = wl.llama3_8b_stack32()
    L, Hkv = spec.n_layers, spec.n_kv_heads
    att_layers = {0, 13, 31}
    cfg1 = B.make_config(spec, beta=1.0, out_dtype=B.F32)
    cfg32 = B.make_config(spec, beta=32.0, out_dtype=B.F32)
    pt = wl.shuffled_page_table(spec, spec.context)
    st = B.RetrievalState(cfg1, n_seq=1, n_layers=L, page_table=pt[None, :])
    budget32 = torch.zeros_like(st.budget_state)
    scores32, theta32 = torch.zeros_like(st.scores), torch.zeros_like(st.theta)
    sel_idx32, sel_count32, real32 = torch.full_like(st.sel_idx, -1), torch.zeros_like(st.sel_count), torch.zeros_like(st.budget_real)
    chain1 = orc.BudgetChain(L, spec.k_blocks, spec.cap_blocks, "streaming")
    chain32 = orc.BudgetChain(L, spec.k_blocks, spec.cap_blocks, "streaming")
    runners = [pu.OracleRunner(spec, layer=l, chain=chain1, beta=1.0) for l in range(L)]
    out = torch.zeros(L, spec.window, spec.n_q_heads, spec.head_dim, dtype=torch.float32, device="cuda")
    out32 = torch.zeros_like(out)
    T = spec.n_windows
    tally = dict(windows=0, sets=0, near=0, fragile=0, att=0, worst_att=0.0)
    last_counts = None
    for t in range(T):
        last = t == T - 1
        check = last or t < 2 or t % 4 == 3
        qs, ks, vs, res, res32 = [], [], [], [], []
        for l in range(L):
            q = wl.gen_q(spec, l, t)
            k, v = wl.gen_kv(spec, l, t)
            qs.append(q); ks.append(k); vs.append(v)
            r = runners[l].step(q, k, v, attention=last and l in att_layers)
            res.append(r)
            th = orc.information_density(r["scores"], 32.0)
            c, b_real, fragile = chain32.grant(l, th, r["n"])
            r32 = dict(c=c, b_real=b_real, fragile=fragile, theta=th)
            if check:
                picks = [orc.select_blocks(r["scores"][g], c) for g in range(Hkv)]
                r32.update(sel=[x[0] for x in picks], tau=[x[1] for x in picks], near=[x[2] for x in picks])
                if last and l in att_layers:
                    state = runners[l].state
                    r32["out"], _ = orc.retrieval_attention(q, k, v, state.k_cache, state.v_cache, r["p0"], r32["sel"],
                                                            spec.n_init, spec.block, spec.n_local_prev)
            res32.append(r32)
        dq, dk, dv = (pu.to_device(np.stack(x), spec) for x in (qs, ks, vs))
        st.step(dq, dk, dv, out, advance=False)
        B.score_select(cfg32, st.batch, st.probe_kv, st.repr_k, st.repr_inv_norm, st.n_cand, budget32, scores32,
                       theta32, sel_idx32, sel_count32, real32, st.status)
        if last:
            B.retrieval_attention(cfg32, st.batch, dq, dk, dv, spec.window, st.k_pages, st.v_pages, st.page_table,
                                  st.pos0, sel_idx32, sel_count32, out32, None, st.status)
        st.set_positions([(t + 1) * spec.window])
        torch.cuda.synchronize()
        assert int(st.status.item()) == 0
        n = res[0]["n"]
        for beta, rr, cnt, idx, th_gpu, o_gpu in ((1.0, res, st.sel_count, st.sel_idx, st.theta, out),
                                                  (32.0, res32, sel_count32, sel_idx32, theta32, out32)):
            tag = f"{spec.name} beta={beta} window {t}"
            got_c = cnt.cpu().numpy().tolist()
            want_c = [r["c"] for r in rr]
            if any(r["fragile"] for r in rr):
                tally["fragile"] += 1
                # a rounding decision on the boundary: the later layers of this step inherit the
                # difference, so follow the device from here on
                assert sum(abs(a - b) for a, b in zip(got_c, want_c)) <= 2 * sum(r["fragile"] for r in rr), tag
                chain = chain1 if beta == 1.0 else chain32
                chain.b_rem = float(budget32[0, 0] if beta == 32.0 else st.budget_state[0, 0])
                continue
            assert got_c == want_c, tag
            if not (check and n):
                continue
            th = pu.to_numpy(th_gpu)
            for l in range(L):
                if beta == 1.0:
                    pu.assert_rel(pu.to_numpy(st.scores[l, :, :n]), res[l]["scores"], 1.0, f"{tag} layer {l} scores")
                pu.assert_rel(th[l], rr[l]["theta"], 1e-30, f"{tag} layer {l} theta", tol=2e-4 if beta > 1 else pu.REL_TOL)
                r_full = dict(res[l], **rr[l]) if beta != 1.0 else rr[l]
                nd = pu.compare_selection(pu.to_numpy(idx[l]).astype(np.int64), got_c[l], r_full, f"{tag} layer {l}")
                assert nd >= 0
                tally["sets"] += 1
                tally["near"] += nd
                if last and l in att_layers and nd == 0:
                    mx, _ = pu.assert_attention(pu.to_numpy(o_gpu[l]), rr[l]["out"], f"{tag} layer {l} attention")
                    tally["att"] += 1
                    tally["worst_att"] = max(tally["worst_att"], mx)
            if last:
                last_counts = (last_counts or {})
                last_counts[beta] = want_c
        tally["windows"] += 1
    print("stack32 at 32k:", tally)
    last_counts = last_counts or {}
    print("  counts at the last window, beta = 1 :", last_counts.get(1.0))
    print("  counts at the last window, beta = 32:", last_counts.get(32.0))
    print("  exp(theta) per layer at the last window (beta = 1):",
          [round(float(np.exp(np.mean(r["theta"]))), 2) for r in res])
    assert tally["att"] >= 5                                   # of 6 (3 layers x 2 temperatures)
    assert abs(float(st.budget_state[0, 0]) - chain1.b_rem) < 1e-9
    c32 = last_counts.get(32.0) or sel_count32.cpu().numpy().tolist()
    assert len(set(c32)) > 2 and max(c32) == spec.cap_blocks   # counts vary by layer, the cap binds


def test_long_131k_sweep(B):
    """131072-token prefill, one layer, cut-off capped at 128 blocks: steps 1-4 and 6 at every
    window (n grows to 1019 candidate blocks), attention at windows {0, 1, 31, 32, 33, 127, 255}."""
    import torch
    spec = wl.long_131k()
    cfg = B.make_config(spec, out_dtype=B.F32)
    pt = wl.shuffled_page_table(spec, spec.context)
    st = B.RetrievalState(cfg, page_table=pt[None, :])
    run = pu.OracleRunner(spec)
    out = torch.zeros(spec.window, spec.n_q_heads, spec.head_dim, dtype=torch.float32, device="cuda")
    att = {0, 1, 31, 32, 33, 127, 255}
    near = att_checked = 0
    for t in range(spec.n_windows):
        q = wl.gen_q(spec, 0, t)
        k, v = wl.gen_kv(spec, 0, t)
        res = run.step(q, k, v, attention=t in att)
        assert int(st.n_cand.item()) == res["n"]
        st.step(pu.to_device(q[None], spec), pu.to_device(k[None], spec), pu.to_device(v[None], spec), out)
        if t % 8 and t not in att:
            continue
        torch.cuda.synchronize()
        assert int(st.status.item()) == 0
        tag = f"{spec.name} window {t}"
        n = res["n"]
        if n:
            pu.assert_rel(pu.to_numpy(st.scores[0, :, :n]), res["scores"], 1.0, tag + " scores")
        nd = pu.compare_selection(pu.to_numpy(st.sel_idx[0]).astype(np.int64), int(st.sel_count.item()), res, tag)
        assert nd >= 0
        near += nd
        if t in att and nd == 0:
            pu.assert_attention(pu.to_numpy(out), res["out"], tag + " attention")
            att_checked += 1
    assert att_checked >= len(att) - 1, f"attention compared at only {att_checked} of {len(att)} sampled windows"
    sel = pu.to_numpy(st.sel_idx[0]).astype(int)
    for g in range(spec.n_kv_heads):
        assert set(wl.planted_blocks(spec, 0)[g]) <= set(sel[g])
    print("131k sweep: near-tie differences", near)


def test_decode_batch_fixed_probes(B):
    """Batched decode (Eq. 3): sequences of different lengths, one token per step, 512 recent
    tokens kept local, probes fixed from each sequence's last prefill window, two layers with
    the budget chain between them.  Reduced sizes of the 16-sequence workload."""
    import torch
    base = wl.decode_batch16()
    spec = base.replace(n_layers=2, n_seq=3, decode_steps=6, ctx_lo=2048, ctx_hi=6144, context=8192,
                        k_blocks=8, cap_blocks=16, n_planted=0)
    L, S = spec.n_layers, spec.n_seq
    ctx = (wl.decode_contexts(spec) // spec.window) * spec.window          # whole prefill windows
    cfg = B.make_config(spec, out_dtype=B.F32, max_context=int(ctx.max()) + spec.decode_steps + spec.window,
                        n_phys_pages=S * (-(-(int(ctx.max()) + spec.decode_steps + 16) // 16)))
    # one pool of pages per layer shared by the sequences, disjoint seeded page tables
    per_seq = cfg.n_phys_pages // S
    rng = np.random.default_rng(5)
    perm = rng.permutation(cfg.n_phys_pages).astype(np.int32)
    table = np.zeros((S, cfg.max_pages), np.int32)
    for s in range(S):
        table[s, :per_seq] = perm[s * per_seq:(s + 1) * per_seq][: cfg.max_pages][:per_seq]
    st = B.RetrievalState(cfg, n_seq=S, n_layers=L, page_table=table)
    # prefill (n_local_prev = 0 during prefill, as in the paper's prefill stage) sequence by sequence
    # through per-sequence states that alias the shared buffers
    pre_spec = spec.replace(n_local_prev=0)
    pre_cfg = B.make_config(pre_spec, out_dtype=B.F32, max_context=cfg.max_pages * 16, n_phys_pages=cfg.n_phys_pages)
    pre_cfg.n_cap, pre_cfg.max_pages = cfg.n_cap, cfg.max_pages
    chains = [orc.BudgetChain(L, spec.k_blocks, spec.cap_blocks, "streaming") for _ in range(S)]
    runners = [[pu.OracleRunner(pre_spec, layer=l, chain=chains[s]) for l in range(L)] for s in range(S)]
    out_w = torch.zeros(L, spec.window, spec.n_q_heads, spec.head_dim, dtype=torch.float32, device="cuda")
    probes = np.zeros((S, L, spec.n_kv_heads, spec.head_dim))
    for s in range(S):
        ps = B.RetrievalState(pre_cfg, n_seq=1, n_layers=L, page_table=table[s:s + 1], shared_pages=(st.k_pages, st.v_pages))
        sspec = pre_spec.replace(seed=spec.seed + 100 * s)
        for t in range(int(ctx[s]) // spec.window):
            qs, ks, vs = [], [], []
            for l in range(L):
                q = wl.gen_q(sspec, l, t); k, v = wl.gen_kv(sspec, l, t)
                qs.append(q); ks.append(k); vs.append(v)
                r = runners[s][l].step(q, k, v, attention=False)
                probes[s, l] = r["probe_kv"]
            ps.step(pu.to_device(np.stack(qs), spec), pu.to_device(np.stack(ks), spec),
                    pu.to_device(np.stack(vs), spec), out_w)
        torch.cuda.synchronize()
        assert int(ps.status.item()) == 0
        # hand the sequence's state over to the batched decode state (unit = s * L + l)
        for name in ("repr_k", "repr_inv_norm", "probe_kv", "probe_qh", "stats_mean", "stats_m2", "stats_count"):
            getattr(st, name)[s * L:(s + 1) * L].copy_(getattr(ps, name))
        st.budget_state[s].copy_(ps.budget_state[0])
        assert np.allclose(pu.to_numpy(ps.probe_kv), probes[s], rtol=1e-3, atol=1e-4)
    st.set_positions([int(c) for c in ctx])
    # ---- decode: one token per sequence per step, probes fixed
    for l in range(L):
        for s in range(S):
            runners[s][l].spec = spec                      # 512 local tokens from here on
    out = torch.zeros(S * L, 1, spec.n_q_heads, spec.head_dim, dtype=torch.float32, device="cuda")
    rs = np.random.default_rng(9)
    for step in range(spec.decode_steps):
        q = wl.bf16_grid(rs.standard_normal((S * L, 1, spec.n_q_heads, spec.head_dim)).astype(np.float32))
        k = wl.bf16_grid(rs.standard_normal((S * L, 1, spec.n_kv_heads, spec.head_dim)).astype(np.float32))
        v = wl.bf16_grid(rs.standard_normal((S * L, 1, spec.n_kv_heads, spec.head_dim)).astype(np.float32))
        st.step(pu.to_device(q, spec), pu.to_device(k, spec), pu.to_device(v, spec), out, n_tokens=1,
                update_probe=False)
        torch.cuda.synchronize()
        assert int(st.status.item()) == 0
        for s in range(S):
            for l in range(L):
                u = s * L + l
                run = runners[s][l]
                state = run.state
                p0 = state.k_cache.shape[0]
                n = orc.n_candidate_blocks(p0, spec.n_init, spec.block, spec.n_local_prev)
                run._extend_table(run.complete_blocks())
                sc = orc.block_scores(probes[s, l], run.table[:, :n])
                theta = orc.information_density(sc)
                c, b_real, fragile = chains[s].grant(l, theta, n)
                sel = [orc.select_blocks(sc[g], c)[0] for g in range(spec.n_kv_heads)]
                o, _ = orc.retrieval_attention(q[u], k[u], v[u], state.k_cache, state.v_cache, p0, sel, spec.n_init,
                                               spec.block, spec.n_local_prev)
                state.k_cache, state.v_cache = orc.append_window(state.k_cache, state.v_cache, k[u], v[u])
                tag = f"decode step {step} seq {s} layer {l}"
                if fragile:
                    continue
                assert int(st.sel_count[u].item()) == c, tag
                got = pu.to_numpy(st.sel_idx[u]).astype(np.int64)
                for g in range(spec.n_kv_heads):
                    _, tau, near = orc.select_blocks(sc[g], c)
                    diff = set(got[g][:c].tolist()) ^ set(sel[g].tolist())
                    assert diff <= set(near.tolist()), tag
                    if diff:
                        break
                else:
                    pu.assert_attention(pu.to_numpy(out[u]), o, tag + " attention")


@pytest.mark.parametrize("n_new", [1, 5, 32])
def test_decode_attention_splits_match_general_kernel(B, n_new):
    """The tensor-core decode kernel, unsplit and with the key stream cut into 2, 5, 16 and the
    automatic number of shares (workspace + merge kernel), against the general fp32 kernel on the
    same state: ragged position (the last cache page partly filled), 512 local tokens, steps of
    1, 5 and 32 = 128 / G new tokens."""
    import torch
    spec = wl.llama3_8b_layer().replace(context=4096, n_local_prev=512, k_blocks=16, cap_blocks=16)
    cfg = B.make_config(spec, out_dtype=B.F32, max_context=8192)
    st = B.RetrievalState(cfg, page_table=wl.shuffled_page_table(spec, 8192)[None, :])
    out_w = torch.zeros(spec.window, spec.n_q_heads, spec.head_dim, dtype=torch.float32, device="cuda")
    for t in range(spec.n_windows):
        q = pu.to_device(wl.gen_q(spec, 0, t)[None], spec)
        k, v = wl.gen_kv(spec, 0, t)
        st.step(q, pu.to_device(k[None], spec), pu.to_device(v[None], spec), out_w)
    g = torch.Generator(device="cuda").manual_seed(3)
    def rnd(n, h):
        return torch.randn(1, n, h, spec.head_dim, device="cuda", generator=g).to(torch.bfloat16)
    o1 = torch.zeros(1, 1, spec.n_q_heads, spec.head_dim, device="cuda")
    for _ in range(19):                                   # leaves p0 = 4096 + 19: not on a page boundary
        st.step(rnd(1, spec.n_q_heads), rnd(1, spec.n_kv_heads), rnd(1, spec.n_kv_heads), o1, n_tokens=1,
                update_probe=False)
    q, k, v = rnd(n_new, spec.n_q_heads), rnd(n_new, spec.n_kv_heads), rnd(n_new, spec.n_kv_heads)
    B.score_select(cfg, st.batch, st.probe_kv, st.repr_k, st.repr_inv_norm, st.n_cand, st.budget_state, st.scores,
                   st.theta, st.sel_idx, st.sel_count, st.budget_real, st.status)
    shape = (1, n_new, spec.n_q_heads, spec.head_dim)
    ref, ref_lse = torch.zeros(shape, device="cuda"), torch.zeros(spec.n_q_heads, n_new, device="cuda")
    cfg_gen = B.make_config(spec, out_dtype=B.F32, max_context=8192, attention_kernel=B.ATTN_GENERAL)
    B.retrieval_attention(cfg_gen, st.batch, q, k, v, n_new, st.k_pages, st.v_pages, st.page_table, st.pos0, st.sel_idx,
                          st.sel_count, ref, ref_lse, st.status)
    torch.cuda.synchronize()
    auto = B.decode_splits(cfg, st.batch)
    assert auto >= 8                                      # 8 (unit, KV head) pairs on a GPU of ~148 SMs
    for splits in (1, 2, 5, 16, 0):
        ws_bytes = B.decode_workspace_bytes(cfg, st.batch, n_new, splits)
        assert (ws_bytes == 0) == (splits == 1)
        ws = torch.full((max(ws_bytes, 16) // 4,), float("nan"), device="cuda")
        got, lse = torch.full(shape, float("nan"), device="cuda"), torch.zeros_like(ref_lse)
        B.decode_attention(cfg, st.batch, q, k, v, n_new, st.k_pages, st.v_pages, st.page_table, st.pos0, st.sel_idx,
                           st.sel_count, got, lse, n_splits=splits, workspace=ws if splits != 1 else None,
                           status=st.status)
        torch.cuda.synchronize()
        assert int(st.status.item()) == 0
        assert (got - ref).abs().max().item() < 4e-3, splits
        assert (lse - ref_lse).abs().max().item() < 2e-3, splits
    # a workspace that is too small is refused on the host
    with pytest.raises(B.ActQKVError):
        B.decode_attention(cfg, st.batch, q, k, v, n_new, st.k_pages, st.v_pages, st.page_table, st.pos0, st.sel_idx,
                           st.sel_count, got, lse, n_splits=4, workspace=torch.zeros(64, device="cuda"))


@pytest.mark.gpu
@pytest.mark.parametrize("shape", ["f32_d64", "bf16_d128"])
def test_bias_probe_many_units_against_oracle(B, shape):
    """Calls with at least two (unit, head) items per SM take the persistent streaming kernel
    instead of the cluster kernel.  Two windows per unit (so the second merges into running
    statistics, Eq. 8), the second one ragged (fewer tokens than a whole number of row chunks),
    every unit with its own data, all outputs against the oracle (Eq. 7 - 9)."""
    import torch
    if shape == "f32_d64":
        spec, U = wl.tiny_pr1(), 96              # 96 units x 4 heads
    else:
        spec, U = wl.llama3_8b_layer().replace(context=4096), 12    # 12 units x 32 heads
    assert U * spec.n_q_heads >= 2 * torch.cuda.get_device_properties(0).multi_processor_count
    spec = spec.replace(n_layers=U)
    cfg = B.make_config(spec)
    batch = B.Batch(1, U, 0)
    Hq, Hkv, D, W = spec.n_q_heads, spec.n_kv_heads, spec.head_dim, spec.window
    f32 = dict(dtype=torch.float32, device="cuda")
    count = torch.zeros(U, Hq, dtype=torch.int64, device="cuda")
    mean, m2 = torch.zeros(U, Hq, D, **f32), torch.zeros(U, Hq, D, **f32)
    probe_qh, probe_kv = torch.zeros(U, Hq, D, **f32), torch.zeros(U, Hkv, D, **f32)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    runs = [orc.RunningStats(Hq, D) for _ in range(U)]
    for t, n_tok in enumerate([W, W - 37]):
        q_host = [wl.gen_q(spec, u, t)[:n_tok] for u in range(U)]
        q = pu.to_device(np.stack(q_host), spec)
        phi_l1 = torch.zeros(U, Hq, n_tok, **f32)
        phi_full = torch.zeros(U, n_tok, Hq, D, **f32)
        # the two-call form (Eq. 7-8, then Eq. 9) on copies of the statistics: same kernels, other switches
        count2, mean2, m22 = count.clone(), mean.clone(), m2.clone()
        phi_l1_b, pqh_b, pkv_b = torch.zeros_like(phi_l1), torch.zeros_like(probe_qh), torch.zeros_like(probe_kv)
        B.activation_bias(cfg, batch, q, n_tok, count2, mean2, m22, phi_l1_b, None, status)
        B.probe_query(cfg, batch, q, n_tok, phi_l1_b, pqh_b, pkv_b, status)
        B.bias_probe(cfg, batch, q, n_tok, count, mean, m2, phi_l1, phi_full, probe_qh, probe_kv, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.equal(count2, count) and torch.equal(mean2, mean) and torch.equal(m22, m2)
        assert torch.equal(phi_l1_b, phi_l1)
        for got, want, nm in ((pqh_b, probe_qh, "probe_qh"), (pkv_b, probe_kv, "probe_kv")):
            for u in range(U):
                pu.assert_probe(pu.to_numpy(got[u]), pu.to_numpy(want[u]).astype(np.float64), f"{shape} unit {u} two-call {nm}")
        for u in range(U):
            tag = f"{shape} unit {u} window {t}"
            runs[u].update(q_host[u])
            zbar, sigma2 = runs[u].mean, runs[u].variance()
            phi, a = orc.activation_bias(q_host[u], zbar, sigma2)
            pqh = orc.probe_query(q_host[u], a)
            assert int(count[u, 0].item()) == runs[u].count
            pu.assert_rel(pu.to_numpy(mean[u]), zbar, 1e-3 * np.abs(zbar).max() + 1e-30, tag + " mean")
            pu.assert_rel(pu.to_numpy(m2[u]) / (runs[u].count - 1), sigma2, 1e-30, tag + " variance")
            pu.assert_phi_like(pu.to_numpy(phi_l1[u]).T, a, tag + " phi_l1")
            pu.assert_phi_like(pu.to_numpy(phi_full[u]), phi, tag + " phi")
            pu.assert_probe(pu.to_numpy(probe_qh[u]), pqh, tag + " probe_qh")
            pu.assert_probe(pu.to_numpy(probe_kv[u]), orc.kv_head_probe(pqh, Hkv), tag + " probe_kv")
