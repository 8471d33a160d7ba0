"""Seeded synthetic workloads shaped like the paper's long-context runs.

This module only *draws inputs*: query/key/value activations with outlier
channels, planted relevant blocks, shuffled page tables and decode context
lengths.  It contains none of the method's arithmetic (no activation bias, no
scoring, no selection, no attention), so both the CPU oracle's tests and the
CUDA path's tests may draw identical inputs from it.

Every tensor is a pure function of (seed, layer, tensor kind, window index):
any window of any layer can be regenerated on its own without materialising
the whole context, which is what makes parity checks at 32k / 131k context
feasible on the host.

Values are returned as float32 numpy arrays.  For bf16 workloads they are
already rounded to the bf16 grid, so converting to a bf16 device tensor is
exact and both sides see the same bits.
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass
from functools import lru_cache

import numpy as np

# Tensor kinds: one Philox stream each.
_KIND_Q, _KIND_K, _KIND_V, _KIND_OUTLIER, _KIND_PLANT_POS, _KIND_PLANT_NOISE, \
    _KIND_PAGES, _KIND_CTX, _KIND_PLANT_CFG = range(9)


@dataclass(frozen=True)
class WorkloadSpec:
    """Shapes and generator parameters of one synthetic workload."""
    name: str
    seed: int
    n_layers: int          # L
    n_q_heads: int         # Hq
    n_kv_heads: int        # Hkv
    head_dim: int          # D
    dtype: str             # "f32" | "bf16"
    context: int           # prefill tokens
    window: int            # W (the paper's m)
    block: int             # B tokens per block
    n_repr: int            # r representative keys per block
    page_tokens: int       # tokens per cache page
    n_init: int            # initial ("sink") tokens always attended
    n_local_prev: int      # extra recent past tokens kept local
    k_blocks: int          # k: average per-layer block budget
    cap_blocks: int        # per-layer cap on selected blocks
    n_outlier: int         # outlier channels per head
    outlier_scale: float
    n_planted: int         # planted relevant blocks per KV head
    planted_noise: float   # std of the noise added to the planted keys
    n_seq: int = 1
    decode_steps: int = 0
    ctx_lo: int = 0        # decode: contexts ~ U[ctx_lo, ctx_hi]
    ctx_hi: int = 0
    vary_planted_by_layer: bool = False

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def n_windows(self) -> int:
        return self.context // self.window

    def replace(self, **kw) -> "WorkloadSpec":
        return dataclasses.replace(self, **kw)


def tiny_pr1() -> WorkloadSpec:
    """Config 0: 1 layer, 4/2 heads, D=64, fp32, 4096 ctx, W=256, k=8."""
    return WorkloadSpec("tiny_pr1", 0, 1, 4, 2, 64, "f32", 4096, 256, 128, 4, 16, 64, 0,
                        8, 8, 2, 8.0, 3, 0.3)


def llama3_8b_layer() -> WorkloadSpec:
    """Config 1: LLaMA3-8B-shaped layer, bf16, 32k ctx, W=512, k=32."""
    return WorkloadSpec("llama3_8b_layer_32k", 1, 1, 32, 8, 128, "bf16", 32768, 512, 128, 4, 16,
                        128, 0, 32, 32, 4, 10.0, 8, 0.3)


def llama3_8b_stack32() -> WorkloadSpec:
    """Config 2: 32 layers of the LLaMA3-8B shape, k=32 (B_kv=1024), cap 64."""
    return llama3_8b_layer().replace(name="llama3_8b_stack32_32k", seed=2, n_layers=32,
                                     cap_blocks=64, vary_planted_by_layer=True)


def tiny_stack32() -> WorkloadSpec:
    """Cheap 32-layer variant of the tiny shape (fp32, k=8, cap 16)."""
    return tiny_pr1().replace(name="tiny_stack32", seed=2, n_layers=32, cap_blocks=16,
                              vary_planted_by_layer=True)


def long_131k() -> WorkloadSpec:
    """Config 3: 131072 ctx, LLaMA3-8B shape, k=cap=128, 16 planted blocks."""
    return llama3_8b_layer().replace(name="llama3_8b_layer_131k", seed=3, context=131072,
                                     k_blocks=128, cap_blocks=128, n_planted=16)


def decode_batch16() -> WorkloadSpec:
    """Config 4: decode, 16 sequences, contexts ~ U[32768,131072], 256 steps."""
    return llama3_8b_layer().replace(name="llama3_8b_decode_b16", seed=4, n_layers=32,
                                     context=131072, cap_blocks=64, n_local_prev=512,
                                     n_seq=16, decode_steps=256, ctx_lo=32768, ctx_hi=131072)


def paper_shaped() -> WorkloadSpec:
    """The paper's own hyper-parameters (Sec. 5.1): W=256, 64 sinks, 512 local,
    46 chunks of 32 pairs; here B=32 tokens with r=1 representative."""
    return WorkloadSpec("paper_shaped", 5, 1, 32, 8, 128, "bf16", 8192, 256, 32, 1, 16, 64, 256,
                        46, 46, 4, 10.0, 8, 0.3)


# ----------------------------------------------------------------------------
# helpers
# ----------------------------------------------------------------------------
def _rng(spec: WorkloadSpec, kind: int, layer: int = 0, index: int = 0, seq: int = 0):
    key = (np.uint64(spec.seed) << np.uint64(32)) | np.uint64(kind)
    ctr = [int(layer), int(index), int(seq), 0]
    return np.random.Generator(np.random.Philox(key=int(key), counter=ctr))


def bf16_grid(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even), keep float32 storage."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def _store(spec: WorkloadSpec, x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    return bf16_grid(x) if spec.dtype == "bf16" else x


def outlier_channels(spec: WorkloadSpec, layer: int):
    """Outlier channel indices: ([Hq, n_outlier] for Q, [Hkv, n_outlier] for K and V)."""
    g = _rng(spec, _KIND_OUTLIER, layer)
    cq = np.stack([g.choice(spec.head_dim, spec.n_outlier, replace=False)
                   for _ in range(spec.n_q_heads)])
    ck = np.stack([g.choice(spec.head_dim, spec.n_outlier, replace=False)
                   for _ in range(spec.n_kv_heads)])
    return cq, ck


def _scaled_normal(spec, kind, layer, t, n_heads, chans, seq=0):
    g = _rng(spec, kind, layer, t, seq)
    x = g.standard_normal((spec.window, n_heads, spec.head_dim), dtype=np.float32)
    for h in range(n_heads):
        x[:, h, chans[h]] *= np.float32(spec.outlier_scale)
    return x


def n_candidates(spec: WorkloadSpec, p0: int) -> int:
    """Candidate blocks before position p0: blocks tile the past after the
    initial tokens and stop short of the local segment."""
    return max(0, (p0 - spec.n_local_prev - spec.n_init) // spec.block)


def planted_layout(spec: WorkloadSpec, layer: int):
    """(count, noise_std) of planted blocks at this layer."""
    if not spec.vary_planted_by_layer:
        return spec.n_planted, spec.planted_noise
    g = _rng(spec, _KIND_PLANT_CFG, layer)
    cnt = int(g.integers(max(1, spec.n_planted // 4), 2 * spec.n_planted + 1))
    noise = float(spec.planted_noise * g.uniform(0.5, 2.0))
    return cnt, noise


def target_window(spec: WorkloadSpec) -> int:
    return spec.n_windows - 1


@lru_cache(maxsize=256)
def planted_blocks(spec: WorkloadSpec, layer: int) -> np.ndarray:
    """[Hkv, n_planted] block indices planted for the target (last) window."""
    n = n_candidates(spec, target_window(spec) * spec.window)
    cnt, _ = planted_layout(spec, layer)
    cnt = min(cnt, n)
    g = _rng(spec, _KIND_PLANT_POS, layer)
    return np.stack([np.sort(g.choice(n, cnt, replace=False)) for _ in range(spec.n_kv_heads)])


@lru_cache(maxsize=64)
def _target_mean_query(spec: WorkloadSpec, layer: int) -> np.ndarray:
    """Mean of the target window's queries over its tokens and over the query
    heads of each KV group: [Hkv, D] float32."""
    q = gen_q(spec, layer, target_window(spec))
    m = q.astype(np.float64).mean(axis=0)                      # [Hq, D]
    return m.reshape(spec.n_kv_heads, spec.group, spec.head_dim).mean(axis=1).astype(np.float32)


def gen_q(spec: WorkloadSpec, layer: int, t: int) -> np.ndarray:
    """Queries of window t: [W, Hq, D]."""
    cq, _ = outlier_channels(spec, layer)
    return _store(spec, _scaled_normal(spec, _KIND_Q, layer, t, spec.n_q_heads, cq))


def gen_kv(spec: WorkloadSpec, layer: int, t: int):
    """Keys and values of window t: ([W, Hkv, D], [W, Hkv, D]); keys of planted
    blocks are the target window's mean query plus Gaussian noise."""
    _, ck = outlier_channels(spec, layer)
    k = _scaled_normal(spec, _KIND_K, layer, t, spec.n_kv_heads, ck)
    v = _scaled_normal(spec, _KIND_V, layer, t, spec.n_kv_heads, ck)
    if spec.n_planted > 0 and t < target_window(spec):
        pb = planted_blocks(spec, layer)
        _, noise = planted_layout(spec, layer)
        lo, hi = t * spec.window, (t + 1) * spec.window
        mq = None
        for h in range(spec.n_kv_heads):
            for b in pb[h]:
                b0 = spec.n_init + int(b) * spec.block
                s, e = max(b0, lo), min(b0 + spec.block, hi)
                if s >= e:
                    continue
                if mq is None:
                    mq = _target_mean_query(spec, layer)
                g = _rng(spec, _KIND_PLANT_NOISE, layer, int(b) * spec.n_kv_heads + h, t)
                nz = g.standard_normal((e - s, spec.head_dim), dtype=np.float32)
                k[s - lo:e - lo, h, :] = mq[h][None, :] + np.float32(noise) * nz
    return _store(spec, k), _store(spec, v)


def gen_context(spec: WorkloadSpec, layer: int, upto_window: int):
    """K and V of windows [0, upto_window) concatenated: token-major [N, Hkv, D]."""
    ks, vs = [], []
    for t in range(upto_window):
        k, v = gen_kv(spec, layer, t)
        ks.append(k)
        vs.append(v)
    if not ks:
        z = np.zeros((0, spec.n_kv_heads, spec.head_dim), np.float32)
        return z, z.copy()
    return np.concatenate(ks), np.concatenate(vs)


def shuffled_page_table(spec: WorkloadSpec, n_tokens: int, n_phys_pages: int | None = None,
                        seq: int = 0, layer: int = 0) -> np.ndarray:
    """Logical page -> physical page, a seeded permutation (physical order differs
    from logical order).  int32 [ceil(n_tokens / page_tokens)]."""
    n_log = -(-n_tokens // spec.page_tokens)
    n_phys = n_log if n_phys_pages is None else n_phys_pages
    g = _rng(spec, _KIND_PAGES, layer, 0, seq)
    return g.permutation(n_phys)[:n_log].astype(np.int32)


def decode_contexts(spec: WorkloadSpec) -> np.ndarray:
    """Per-sequence prefill lengths for the decode workload, int64 [n_seq]."""
    g = _rng(spec, _KIND_CTX)
    return g.integers(spec.ctx_lo, spec.ctx_hi + 1, size=spec.n_seq).astype(np.int64)


def to_pages(spec: WorkloadSpec, x_tokens: np.ndarray, page_table: np.ndarray,
             n_phys_pages: int) -> np.ndarray:
    """Scatter a token-major [N, Hkv, D] tensor into the paged layout
    [n_phys_pages, Hkv, page_tokens, D] through `page_table` (pure data movement)."""
    n, hkv, d = x_tokens.shape
    pt = spec.page_tokens
    n_log = -(-n // pt)
    pad = n_log * pt - n
    if pad:
        x_tokens = np.concatenate([x_tokens, np.zeros((pad, hkv, d), x_tokens.dtype)])
    pages = np.zeros((n_phys_pages, hkv, pt, d), x_tokens.dtype)
    pages[page_table[:n_log]] = x_tokens.reshape(n_log, pt, hkv, d).transpose(0, 2, 1, 3)
    return pages


# ----------------------------------------------------------------------------
# host <-> device plumbing (no arithmetic: exact conversions only)
# ----------------------------------------------------------------------------
def to_device(x, spec: WorkloadSpec, device="cuda"):
    """A generated float32 array as a device tensor of the workload's dtype (exact: bf16
    workloads are generated on the bf16 grid)."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(device)
    return t.to(torch.bfloat16) if spec.dtype == "bf16" else t


def to_numpy(t) -> np.ndarray:
    """A device tensor as a host array (float32, or float64 for float64 tensors)."""
    import torch
    return t.detach().to(torch.float32).cpu().numpy() if t.dtype != torch.float64 else t.detach().cpu().numpy()
