"""GPU parity of the switches and shapes beside the default path: the probe / statistics /
representation / aggregation variants (an analogue of the paper's ablation, Sec. 5.3), the
paper's own hyper-parameters (Sec. 5.1: window 256, 64 initial tokens, chunks of 32 pairs, 46 of
them), a prefill step that does not start on a page boundary, and decode with the paper's
decode-stage probe q^t (Sec. 4.2)."""
import numpy as np
import pytest

from oracle import actqkv_oracle as orc
from paper_2502_13542_b200 import workloads as wl
from tests import parity_utils as pu
from tests.test_gpu_parity import _run_sweep

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    import torch
    assert torch.cuda.is_available()
    from paper_2502_13542_b200 import binding
    return binding


def _recall(spec, st):
    sel = pu.to_numpy(st.sel_idx[0]).astype(int)
    pb = wl.planted_blocks(spec, 0)
    hit = sum(len(set(pb[g]) & set(sel[g])) for g in range(spec.n_kv_heads))
    return hit / float(pb.size)


VARIANTS = {
    "window_only_stats": {"stats_mode": (1, "window_only")},
    "strided_token_repr": {"repr_mode": (1, "strided_token")},
    "max_aggregation": {"agg_mode": (1, "max")},
    "mean_pool_probe": {"probe_mode": (1, "mean_pool")},
    "strided_max_meanpool": {"repr_mode": (1, "strided_token"), "agg_mode": (1, "max"),
                             "probe_mode": (1, "mean_pool")},
}


@pytest.mark.parametrize("name", sorted(VARIANTS))
@pytest.mark.parametrize("fused", [True, False])
def test_variants_tiny_every_window(B, name, fused):
    """Every window of the tiny fp32 workload under each switch, all intermediates against the
    oracle run with the same switch; the planted-block recall of the CUDA path is printed (the
    oracle's selection is identical, so it is the oracle's recall too)."""
    spec = wl.tiny_pr1()
    stats, o_run, st = _run_sweep(B, spec, {0, 1, 7, 15}, fused, variant=VARIANTS[name])
    print(f"variant {name} (tiny, fused={fused}): planted recall {_recall(spec, st):.2f}, {stats}")


@pytest.mark.parametrize("name", sorted(VARIANTS))
def test_variants_llama_shape(B, name):
    """The same switches on the bf16 / D = 128 / paged shape (8 windows of a 4096-token prefill),
    attention on the tensor-core kernel at windows {1, 7}."""
    spec = wl.llama3_8b_layer().replace(context=4096, n_planted=3)
    stats, o_run, st = _run_sweep(B, spec, {1, 7}, True, variant=VARIANTS[name], also_bf16_out=True,
                                  min_attention_checked=1)
    print(f"variant {name} (llama shape, 4k): planted recall {_recall(spec, st):.2f}, {stats}")


def test_paper_shaped_config(B):
    """The paper's own hyper-parameters (Sec. 5.1): W = 256, 64 initial tokens, 256 extra local
    tokens (512 local pairs with the window), blocks of 32 tokens with one representative,
    budget 46 blocks.  One score per 256-byte table row (the general path of the score kernel),
    two pages per block in the attention gather."""
    spec = wl.paper_shaped()
    stats, o_run, st = _run_sweep(B, spec, {2, 15, 31}, True, also_bf16_out=True, min_attention_checked=2)
    n = wl.n_candidates(spec, (spec.n_windows - 1) * spec.window)
    print(f"paper-shaped: n = {n} candidate blocks at the last window, planted recall {_recall(spec, st):.2f}, {stats}")
    assert int(st.sel_count.item()) == 46


def test_prefill_step_off_the_page_boundary(B):
    """A 128-token step whose first token does not sit on a 16-token page boundary (after a
    ragged step of 37 tokens): the tensor-core kernels load the partly filled last page whole and
    mask its tail.  Both tensor-core kernels and the general kernel against the oracle."""
    import torch
    spec = wl.llama3_8b_layer().replace(context=4096, n_planted=0)
    cfg = B.make_config(spec, out_dtype=B.F32)
    st = B.RetrievalState(cfg, page_table=wl.shuffled_page_table(spec, spec.context)[None, :])
    run = pu.OracleRunner(spec)
    out = torch.zeros(spec.window, spec.n_q_heads, spec.head_dim, device="cuda")
    steps = [(0, 512), (1, 512), (2, 37), (3, 128), (4, 256)]
    for t, nt in steps:
        q = wl.gen_q(spec, 0, t)[:nt]
        k, v = wl.gen_kv(spec, 0, t)
        k, v = k[:nt], v[:nt]
        res = run.step(q, k, v, attention=t >= 3)
        o = out[:nt]
        dq, dk, dv = pu.to_device(q[None], spec), pu.to_device(k[None], spec), pu.to_device(v[None], spec)
        p0 = st.host_pos0[0]
        st.step(dq, dk, dv, o, n_tokens=nt, advance=False)
        torch.cuda.synchronize()
        assert int(st.status.item()) == 0
        if t >= 3:
            assert p0 % 16 != 0
            assert pu.compare_selection(pu.to_numpy(st.sel_idx[0]).astype(np.int64), int(st.sel_count.item()), res,
                                        f"step {t}") == 0
            pu.assert_attention(pu.to_numpy(o), res["out"], f"unaligned p0 = {p0}, pair kernel")
            for which, nm in ((B.ATTN_SINGLE_CTA, "single-CTA kernel"), (B.ATTN_CLUSTER4, "4-CTA-cluster kernel"),
                              (B.ATTN_GENERAL, "general kernel")):
                c2 = B.make_config(spec, out_dtype=B.F32, attention_kernel=which)
                o2 = torch.full_like(o, float("nan"))
                B.retrieval_attention(c2, st.batch, dq, dk, dv, nt, st.k_pages, st.v_pages, st.page_table, st.pos0,
                                      st.sel_idx, st.sel_count, o2, None, st.status)
                torch.cuda.synchronize()
                pu.assert_attention(pu.to_numpy(o2), res["out"], f"unaligned p0 = {p0}, {nm}")
        st.set_positions([p0 + nt])
    assert int(st.status.item()) == 0


@pytest.mark.parametrize("page_tokens", [32, 64, 128])
def test_larger_cache_pages(B, page_tokens):
    """Cache pages of 32, 64 and 128 tokens (the paged cache's page size is a deployment choice;
    the other workloads use 16): every stage on the LLaMA shape, 8 windows of a 4096-token prefill,
    shuffled page table, attention on the CTA-pair tensor-core kernel (one copy box per page, or
    per part of a page inside a CTA's share of a tile) at windows {1, 7}."""
    spec = wl.llama3_8b_layer().replace(context=4096, n_planted=3, page_tokens=page_tokens)
    stats, o_run, st = _run_sweep(B, spec, {1, 7}, True, also_bf16_out=True, min_attention_checked=1)
    print(f"pages of {page_tokens} tokens (llama shape, 4k): planted recall {_recall(spec, st):.2f}, {stats}")


@pytest.mark.parametrize("page_tokens", [64, 128])
def test_larger_cache_pages_off_the_page_boundary(B, page_tokens):
    """A step that starts in the middle of a 64- or 128-token page (after a ragged step of 37
    tokens): the pair kernel loads the partly filled last page whole and masks its tail; compared
    with the oracle and with the general kernel."""
    import torch
    spec = wl.llama3_8b_layer().replace(context=4096, n_planted=0, page_tokens=page_tokens)
    cfg = B.make_config(spec, out_dtype=B.F32)
    st = B.RetrievalState(cfg, page_table=wl.shuffled_page_table(spec, spec.context)[None, :])
    run = pu.OracleRunner(spec)
    out = torch.zeros(spec.window, spec.n_q_heads, spec.head_dim, device="cuda")
    for t, nt in [(0, 512), (1, 512), (2, 37), (3, 128), (4, 256)]:
        q = wl.gen_q(spec, 0, t)[:nt]
        k, v = wl.gen_kv(spec, 0, t)
        k, v = k[:nt], v[:nt]
        res = run.step(q, k, v, attention=t >= 3)
        o = out[:nt]
        dq, dk, dv = pu.to_device(q[None], spec), pu.to_device(k[None], spec), pu.to_device(v[None], spec)
        p0 = st.host_pos0[0]
        st.step(dq, dk, dv, o, n_tokens=nt, advance=False)
        torch.cuda.synchronize()
        assert int(st.status.item()) == 0
        if t >= 3:
            assert p0 % page_tokens != 0
            assert pu.compare_selection(pu.to_numpy(st.sel_idx[0]).astype(np.int64), int(st.sel_count.item()), res,
                                        f"step {t}") == 0
            pu.assert_attention(pu.to_numpy(o), res["out"], f"p0 = {p0}, pages of {page_tokens}, pair kernel")
            c2 = B.make_config(spec, out_dtype=B.F32, attention_kernel=B.ATTN_GENERAL)
            o2 = torch.full_like(o, float("nan"))
            B.retrieval_attention(c2, st.batch, dq, dk, dv, nt, st.k_pages, st.v_pages, st.page_table, st.pos0,
                                  st.sel_idx, st.sel_count, o2, None, st.status)
            torch.cuda.synchronize()
            pu.assert_attention(pu.to_numpy(o2), res["out"], f"p0 = {p0}, pages of {page_tokens}, general kernel")
        st.set_positions([p0 + nt])
    assert int(st.status.item()) == 0
