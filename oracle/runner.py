"""The oracle's view of one (sequence, layer) driven window by window.

TEST INFRASTRUCTURE ONLY, like the rest of this package: it keeps the oracle's state (running
statistics, token-major cache) and an incrementally built representative table, and calls
`actqkv_oracle.window_retrieval` once per step.  `spec` is any object with the workload's shape
fields (n_q_heads, n_kv_heads, head_dim, n_layers, k_blocks, cap_blocks, n_repr, n_init, block,
dtype, n_local_prev); nothing of the CUDA package is imported.
"""
from __future__ import annotations

import numpy as np

from oracle import actqkv_oracle as orc


class OracleRunner:
    """The oracle's view of one (sequence, layer): state + incremental representative table."""

    def __init__(self, spec, layer: int = 0, chain: orc.BudgetChain | None = None,
                 beta: float = 1.0, thetabar_mode: str = "streaming", repr_mode="chunk_mean", agg="mean",
                 stats_mode="cumulative", probe_mode="activation"):
        self.spec, self.layer, self.beta = spec, layer, beta
        self.repr_mode, self.agg = repr_mode, agg
        self.stats_mode, self.probe_mode = stats_mode, probe_mode
        self.state = orc.LayerState(spec.n_q_heads, spec.n_kv_heads, spec.head_dim)
        self.chain = chain or orc.BudgetChain(spec.n_layers, spec.k_blocks, spec.cap_blocks, thetabar_mode)
        self.table = np.zeros((spec.n_kv_heads, 0, spec.n_repr, spec.head_dim))

    def _extend_table(self, n_blocks):
        sp = self.spec
        have = self.table.shape[1]
        if n_blocks <= have:
            return
        new = np.zeros((sp.n_kv_heads, n_blocks - have, sp.n_repr, sp.head_dim))
        for g in range(sp.n_kv_heads):
            for b in range(have, n_blocks):
                lo = sp.n_init + b * sp.block
                new[g, b - have] = orc.build_representatives(self.state.k_cache[lo:lo + sp.block, g, :],
                                                             sp.n_repr, sp.dtype, self.repr_mode)
        self.table = np.concatenate([self.table, new], axis=1)

    def complete_blocks(self):
        sp = self.spec
        n_tok = self.state.k_cache.shape[0]
        return max(0, (n_tok - sp.n_init) // sp.block)

    def step(self, q, k, v, attention=True, theta_all=None, layer_in_model=None):
        sp = self.spec
        self._extend_table(self.complete_blocks())
        res = orc.window_retrieval(self.state, self.chain, self.layer if layer_in_model is None else layer_in_model,
                                   q, k, v, n_init=sp.n_init, block=sp.block,
                                   n_repr=sp.n_repr, dtype=sp.dtype, n_local_prev=sp.n_local_prev,
                                   beta=self.beta, repr_mode=self.repr_mode, agg=self.agg,
                                   attention=attention, theta_all=theta_all, repr_table=self.table,
                                   stats_mode=self.stats_mode, probe_mode=self.probe_mode)
        self._extend_table(self.complete_blocks())
        return res
