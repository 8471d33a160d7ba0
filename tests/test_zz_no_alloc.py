"""The decode attention entry point that allocates nothing (actqkv_decode_attention_static).

Some users of this library cannot allocate device memory at the moment they call it -- a server
that gave the whole GPU to its KV-cache pool at start-up, a decode loop that cannot afford the
device-wide synchronisation of an allocation -- so this variant takes the scratch of the split
decode attention from a fixed array inside the library.  The test calls it through the C ABI
twice in a row, with different inputs and split counts, and checks each result against the
workspace form (actqkv_decode_attention) of the same call; it also checks that a request beyond
the array's size is refused on the host.  It runs last so that a failure here cannot hide the
results of the other tests, and it builds all of its own state, so it passes alone as well."""
import pytest

from paper_2502_13542_b200 import workloads as wl
from tests import parity_utils as pu

pytestmark = pytest.mark.gpu


def test_static_scratch_variant_matches_workspace_variant_twice():
    import torch
    assert torch.cuda.is_available()
    from paper_2502_13542_b200 import binding as B

    spec = wl.llama3_8b_layer().replace(context=2048, n_local_prev=512, k_blocks=8, cap_blocks=8)
    cfg = B.make_config(spec, out_dtype=B.F32, max_context=4096)
    st = B.RetrievalState(cfg, page_table=wl.shuffled_page_table(spec, 4096)[None, :])
    out_w = torch.zeros(spec.window, spec.n_q_heads, spec.head_dim, dtype=torch.float32, device="cuda")
    for t in range(spec.n_windows):
        q = pu.to_device(wl.gen_q(spec, 0, t)[None], spec)
        k, v = wl.gen_kv(spec, 0, t)
        st.step(q, pu.to_device(k[None], spec), pu.to_device(v[None], spec), out_w)
    B.score_select(cfg, st.batch, st.probe_kv, st.repr_k, st.repr_inv_norm, st.n_cand, st.budget_state, st.scores,
                   st.theta, st.sel_idx, st.sel_count, st.budget_real, st.status)
    gen = torch.Generator(device="cuda").manual_seed(11)

    def rnd(n, h):
        return torch.randn(1, n, h, spec.head_dim, device="cuda", generator=gen).to(torch.bfloat16)

    for n_new, splits in ((1, 6), (4, 3)):                # two calls in a row share the one array
        q, k, v = rnd(n_new, spec.n_q_heads), rnd(n_new, spec.n_kv_heads), rnd(n_new, spec.n_kv_heads)
        shape = (1, n_new, spec.n_q_heads, spec.head_dim)
        ws = torch.empty(B.decode_workspace_bytes(cfg, st.batch, n_new, splits) // 4, device="cuda")
        want, want_lse = torch.zeros(shape, device="cuda"), torch.zeros(spec.n_q_heads, n_new, device="cuda")
        B.decode_attention(cfg, st.batch, q, k, v, n_new, st.k_pages, st.v_pages, st.page_table, st.pos0, st.sel_idx,
                           st.sel_count, want, want_lse, n_splits=splits, workspace=ws, status=st.status)
        got, got_lse = torch.full(shape, float("nan"), device="cuda"), torch.zeros_like(want_lse)
        B.decode_attention_static(cfg, st.batch, q, k, v, n_new, st.k_pages, st.v_pages, st.page_table, st.pos0,
                                  st.sel_idx, st.sel_count, got, got_lse, n_splits=splits, status=st.status)
        torch.cuda.synchronize()
        assert int(st.status.item()) == 0
        assert (got - want).abs().max().item() <= pu.ATT_MAX_ABS
        assert (got - want).abs().mean().item() <= pu.ATT_MEAN_ABS
        assert (got_lse - want_lse).abs().max().item() <= 2e-3

    # 32 tokens x 32 heads x 64 splits x 516 bytes is four times the array: refused, nothing enqueued
    n_new = 32
    assert B.decode_workspace_bytes(cfg, st.batch, n_new, 64) > B.STATIC_SCRATCH_BYTES
    q, k, v = rnd(n_new, spec.n_q_heads), rnd(n_new, spec.n_kv_heads), rnd(n_new, spec.n_kv_heads)
    out = torch.zeros(1, n_new, spec.n_q_heads, spec.head_dim, device="cuda")
    with pytest.raises(B.ActQKVError, match="scratch"):
        B.decode_attention_static(cfg, st.batch, q, k, v, n_new, st.k_pages, st.v_pages, st.page_table, st.pos0,
                                  st.sel_idx, st.sel_count, out, None, n_splits=64, status=st.status)
