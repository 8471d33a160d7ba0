"""A window step replayed from a CUDA graph against the same step enqueued call by call.

Enqueued from Python, a step's launches reach the GPU one at a time, so the attention kernel
hardly ever runs beside the kernels that produce its selection.  Replayed from a graph the whole
chain is resident at once (programmatic dependent launch): the attention works through its
initial / local / window tiles while bias + probe, score and cut-off are still running, takes its
dependency wait where the selected blocks begin, and the append runs on a second stream beside
it.  The result must not depend on that timing: every buffer the step writes is compared bit for
bit with the eager step, and the eager step is compared with the oracle as everywhere else."""
import numpy as np
import pytest

from paper_2502_13542_b200 import workloads as wl
from tests import parity_utils as pu

pytestmark = pytest.mark.gpu

STATE = ["stats_count", "stats_mean", "stats_m2", "repr_k", "repr_inv_norm", "budget_state", "k_pages", "v_pages",
         "probe_kv", "probe_qh", "pos0", "n_cand"]
WRITTEN = STATE + ["phi_l1", "scores", "theta", "sel_idx", "sel_count", "budget_real"]


@pytest.mark.parametrize("context", [8192, 2048 + 37])
def test_graph_replay_of_a_step_matches_the_eager_step(context):
    import torch
    assert torch.cuda.is_available()
    from paper_2502_13542_b200 import binding as B

    ragged = context % 512 != 0
    spec = wl.llama3_8b_layer().replace(context=8192, n_planted=2)
    cfg = B.make_config(spec, out_dtype=B.BF16)
    table = wl.shuffled_page_table(spec, spec.context)[None, :]
    eager = B.RetrievalState(cfg, page_table=table)
    run = pu.OracleRunner(spec)
    W = spec.window
    out = torch.zeros(W, spec.n_q_heads, spec.head_dim, dtype=torch.bfloat16, device="cuda")
    n_before = context // W if ragged else context // W - 1
    for t in range(n_before):
        q = wl.gen_q(spec, 0, t)
        k, v = wl.gen_kv(spec, 0, t)
        run.step(q, k, v, attention=False)
        eager.step(pu.to_device(q[None], spec), pu.to_device(k[None], spec), pu.to_device(v[None], spec), out)
    if ragged:                        # a short step first, so that the step under test starts off the page grid
        nt = context % W
        q = wl.gen_q(spec, 0, n_before)[:nt]
        k, v = wl.gen_kv(spec, 0, n_before)
        run.step(q, k[:nt], v[:nt], attention=False)
        p0 = eager.host_pos0[0]
        eager.step(pu.to_device(q[None], spec), pu.to_device(k[:nt][None], spec), pu.to_device(v[:nt][None], spec),
                   out[:nt], n_tokens=nt, advance=False)
        eager.set_positions([p0 + nt])
        assert eager.host_pos0[0] % 16 != 0
    torch.cuda.synchronize()

    # a second state that stands exactly where the first one does
    replay = B.RetrievalState(cfg, page_table=table)
    for name in STATE:
        getattr(replay, name).copy_(getattr(eager, name))
    replay.host_pos0 = list(eager.host_pos0)

    t = n_before + (1 if ragged else 0)
    q = wl.gen_q(spec, 0, t)
    k, v = wl.gen_kv(spec, 0, t)
    dq, dk, dv = pu.to_device(q[None], spec), pu.to_device(k[None], spec), pu.to_device(v[None], spec)
    res = run.step(q, k, v, attention=True)
    out_e = torch.zeros_like(out)
    eager.step(dq, dk, dv, out_e, advance=False)
    torch.cuda.synchronize()
    assert int(eager.status.item()) == 0
    assert pu.compare_selection(pu.to_numpy(eager.sel_idx[0]).astype(np.int64), int(eager.sel_count.item()), res,
                                "eager step") == 0
    pu.assert_attention_bf16_out(pu.to_numpy(out_e), res["out"], "eager step")

    out_g = torch.full_like(out, float("nan"))
    replay._side = torch.cuda.Stream()          # the append's stream exists before the capture begins
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        replay.step(dq, dk, dv, out_g, advance=False, overlap_append=True)
    torch.cuda.synchronize()
    assert torch.isnan(out_g.float()).all(), "capturing must not run anything"
    graph.replay()
    torch.cuda.synchronize()
    assert int(replay.status.item()) == 0
    assert torch.equal(out_g, out_e), "attention output differs between graph replay and eager calls"
    for name in WRITTEN:
        a, b = getattr(replay, name), getattr(eager, name)
        assert torch.equal(a, b), f"{name} differs between graph replay and eager calls"
