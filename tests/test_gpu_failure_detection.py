"""Failure detection on the device: a bounded wait that runs out must end in a status bit, not in
a hang or a fault.  Nothing here faults or hangs the GPU: the decode attention kernel is given a
short limit for its waits and told (through the test hooks of the config) never to issue the K copy
of one tile, so the wait for that tile expires after a few thousand polls; the kernel must flag
ACTQKV_DEV_TIMEOUT, drain its copies, free its TMEM and return, and the next ordinary call on the
same context must be correct."""
import pytest

from paper_2502_13542_b200 import workloads as wl
from tests import parity_utils as pu

pytestmark = pytest.mark.gpu


def test_decode_wait_that_runs_out_sets_the_timeout_bit_and_the_context_stays_usable():
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
    gen = torch.Generator(device="cuda").manual_seed(5)
    q = torch.randn(1, 1, spec.n_q_heads, spec.head_dim, device="cuda", generator=gen).to(torch.bfloat16)
    k = torch.randn(1, 1, spec.n_kv_heads, spec.head_dim, device="cuda", generator=gen).to(torch.bfloat16)
    v = torch.randn(1, 1, spec.n_kv_heads, spec.head_dim, device="cuda", generator=gen).to(torch.bfloat16)
    shape = (1, 1, spec.n_q_heads, spec.head_dim)

    def run(c, splits, ws):
        out = torch.full(shape, float("nan"), device="cuda")
        st.status.zero_()
        B.decode_attention(c, st.batch, q, k, v, 1, st.k_pages, st.v_pages, st.page_table, st.pos0, st.sel_idx,
                           st.sel_count, out, None, n_splits=splits, workspace=ws, status=st.status)
        torch.cuda.synchronize()                      # returns: the kernel did not hang
        return out, int(st.status.item())

    ws = torch.full((B.decode_workspace_bytes(cfg, st.batch, 1, 3) // 4,), float("nan"), device="cuda")
    good1, s = run(cfg, 1, None)
    assert s == 0
    good3, s = run(cfg, 3, ws)
    assert s == 0 and (good3 - good1).abs().max().item() < 4e-3

    broken = B.make_config(spec, out_dtype=B.F32, max_context=4096)
    broken.test_wait_limit, broken.test_drop_k_tile = 2000, 1
    for splits, w in ((1, None), (3, ws)):
        _, s = run(broken, splits, w)
        assert s & B.DEV_TIMEOUT, f"{splits} split(s): status {s}"
        # the context is intact: the same call without the hooks gives the same result as before
        again, s = run(cfg, splits, w)
        assert s == 0
        assert torch.equal(again, good1 if splits == 1 else good3)
