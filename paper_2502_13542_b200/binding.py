"""Thin Python binding over the C ABI declared in include/actqkv.h.

Argument marshalling only: torch tensors supply device memory and the current
CUDA stream; every step of the path runs in the library's kernels.  There is no
CPU fallback -- if the shared library has not been built, importing this module
raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libactqkv.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2502_13542_b200.build` "
        "(there is no CPU fallback)")
_lib = C.CDLL(LIB_PATH)

F32, BF16 = 0, 1
STATS_CUMULATIVE, STATS_WINDOW_ONLY = 0, 1
REPR_CHUNK_MEAN, REPR_STRIDED_TOKEN = 0, 1
AGG_MEAN, AGG_MAX = 0, 1
THETABAR_STREAMING, THETABAR_ALG1 = 0, 1
PROBE_ACTIVATION, PROBE_MEAN_POOL = 0, 1
ATTN_AUTO, ATTN_GENERAL, ATTN_SINGLE_CTA, ATTN_CLUSTER4 = 0, 1, 2, 3

DEV_BAD_PAGE, DEV_NCAND_CLAMPED, DEV_BAD_PROBE, DEV_BAD_SELECTION, DEV_TIMEOUT, DEV_TABLE_FULL = \
    1, 2, 4, 8, 16, 32


class Config(C.Structure):
    """Mirror of `actqkv_config` (host POD)."""
    _fields_ = [(n, C.c_int32) for n in (
        "n_layers", "n_q_heads", "n_kv_heads", "head_dim", "window", "block", "n_repr", "page_tokens",
        "n_init", "n_local_prev", "k_blocks", "cap_blocks", "dtype", "stats_mode", "repr_mode",
        "agg_mode", "thetabar_mode", "n_cap", "max_pages", "n_phys_pages")] + [
        ("beta", C.c_float), ("sm_scale", C.c_float), ("var_eps", C.c_float), ("out_dtype", C.c_int32),
        ("probe_mode", C.c_int32), ("attention_kernel", C.c_int32), ("test_wait_limit", C.c_int32),
        ("test_drop_k_tile", C.c_int32)]

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == BF16 else torch.float32

    @property
    def torch_out_dtype(self):
        return torch.bfloat16 if self.out_dtype == BF16 else torch.float32

    @property
    def group(self):
        return self.n_q_heads // self.n_kv_heads


class Batch(C.Structure):
    """Mirror of `actqkv_batch`."""
    _fields_ = [("n_seq", C.c_int32), ("n_layers", C.c_int32), ("layer0", C.c_int32)]


class ActQKVError(RuntimeError):
    pass


_P = C.c_void_p
_SIGS = {
    "actqkv_version": ([], C.c_int),
    "actqkv_strerror": ([C.c_int], C.c_char_p),
    "actqkv_budget_state_bytes": ([_P], C.c_int64),
    "actqkv_n_candidates": ([_P, C.c_int64], C.c_int32),
    "actqkv_activation_bias": ([_P, _P, _P, C.c_int32, _P, _P, _P, _P, _P, _P, _P], C.c_int),
    "actqkv_probe_query": ([_P, _P, _P, C.c_int32, _P, _P, _P, _P, _P], C.c_int),
    "actqkv_bias_probe": ([_P, _P, _P, C.c_int32, _P, _P, _P, _P, _P, _P, _P, _P, _P], C.c_int),
    "actqkv_score_blocks": ([_P] * 10, C.c_int),
    "actqkv_select_cutoff": ([_P] * 11, C.c_int),
    "actqkv_score_select": ([_P] * 14, C.c_int),
    "actqkv_retrieval_attention": ([_P, _P, _P, _P, _P, C.c_int32] + [_P] * 10, C.c_int),
    "actqkv_append_window": ([_P, _P, _P, _P, C.c_int32] + [_P] * 8, C.c_int),
    "actqkv_decode_splits": ([_P, _P], C.c_int32),
    "actqkv_decode_workspace_bytes": ([_P, _P, C.c_int32, C.c_int32], C.c_int64),
    "actqkv_decode_attention_static": ([_P, _P, _P, _P, _P, C.c_int32] + [_P] * 8 + [C.c_int32, _P, _P], C.c_int),
    "actqkv_decode_attention": ([_P, _P, _P, _P, _P, C.c_int32] + [_P] * 8 + [C.c_int32, _P, C.c_int64, _P, _P], C.c_int),
}
for _name, (_args, _res) in _SIGS.items():
    _fn = getattr(_lib, _name)          # AttributeError if the library lacks a declared symbol
    _fn.argtypes, _fn.restype = _args, _res

EXPORTED = tuple(_SIGS)


def _ptr(t):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ActQKVError("expected a contiguous CUDA tensor")
    return t.data_ptr()


_raw_current_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream(stream=None):
    """cudaStream_t of `stream`, or of the current stream of the current device.  (Building a
    torch Stream object just to read its handle costs several microseconds per call, a third of
    what it takes to enqueue one of these kernels.)"""
    if stream is not None:
        return stream.cuda_stream
    if _raw_current_stream is not None:
        return _raw_current_stream(torch.cuda.current_device())
    return torch.cuda.current_stream().cuda_stream


def _check(rc):
    if rc != 0:
        raise ActQKVError(f"actqkv error {rc}: {_lib.actqkv_strerror(rc).decode()}")


def _b(batch):
    return C.byref(batch) if batch is not None else None


def version() -> int:
    return _lib.actqkv_version()


def strerror(code: int) -> str:
    return _lib.actqkv_strerror(code).decode()


def budget_state_bytes(cfg: Config) -> int:
    return _lib.actqkv_budget_state_bytes(C.byref(cfg))


def n_candidates(cfg: Config, p0: int) -> int:
    return _lib.actqkv_n_candidates(C.byref(cfg), p0)


def activation_bias(cfg, batch, q, n_tokens, stats_count, stats_mean, stats_m2, phi_l1,
                    phi_full=None, status=None, stream=None):
    _check(_lib.actqkv_activation_bias(C.byref(cfg), _b(batch), _ptr(q), n_tokens, _ptr(stats_count),
                                       _ptr(stats_mean), _ptr(stats_m2), _ptr(phi_l1), _ptr(phi_full),
                                       _ptr(status), _stream(stream)))


def probe_query(cfg, batch, q, n_tokens, phi_l1, probe_qh, probe_kv, status=None, stream=None):
    _check(_lib.actqkv_probe_query(C.byref(cfg), _b(batch), _ptr(q), n_tokens, _ptr(phi_l1),
                                   _ptr(probe_qh), _ptr(probe_kv), _ptr(status), _stream(stream)))


def bias_probe(cfg, batch, q, n_tokens, stats_count, stats_mean, stats_m2, phi_l1, phi_full,
               probe_qh, probe_kv, status=None, stream=None):
    _check(_lib.actqkv_bias_probe(C.byref(cfg), _b(batch), _ptr(q), n_tokens, _ptr(stats_count),
                                  _ptr(stats_mean), _ptr(stats_m2), _ptr(phi_l1), _ptr(phi_full),
                                  _ptr(probe_qh), _ptr(probe_kv), _ptr(status), _stream(stream)))


def score_blocks(cfg, batch, probe_kv, repr_k, repr_inv_norm, n_cand, scores, theta, status=None, stream=None):
    _check(_lib.actqkv_score_blocks(C.byref(cfg), _b(batch), _ptr(probe_kv), _ptr(repr_k),
                                    _ptr(repr_inv_norm), _ptr(n_cand), _ptr(scores), _ptr(theta),
                                    _ptr(status), _stream(stream)))


def select_cutoff(cfg, batch, scores, theta, n_cand, budget_state, sel_idx, sel_count,
                  budget_real=None, status=None, stream=None):
    _check(_lib.actqkv_select_cutoff(C.byref(cfg), _b(batch), _ptr(scores), _ptr(theta), _ptr(n_cand),
                                     _ptr(budget_state), _ptr(sel_idx), _ptr(sel_count),
                                     _ptr(budget_real), _ptr(status), _stream(stream)))


def score_select(cfg, batch, probe_kv, repr_k, repr_inv_norm, n_cand, budget_state, scores, theta,
                 sel_idx, sel_count, budget_real=None, status=None, stream=None):
    _check(_lib.actqkv_score_select(C.byref(cfg), _b(batch), _ptr(probe_kv), _ptr(repr_k),
                                    _ptr(repr_inv_norm), _ptr(n_cand), _ptr(budget_state), _ptr(scores),
                                    _ptr(theta), _ptr(sel_idx), _ptr(sel_count), _ptr(budget_real),
                                    _ptr(status), _stream(stream)))


def retrieval_attention(cfg, batch, q, k_win, v_win, n_tokens, k_pages, v_pages, page_table, pos0,
                        sel_idx, sel_count, out, lse=None, status=None, stream=None):
    _check(_lib.actqkv_retrieval_attention(C.byref(cfg), _b(batch), _ptr(q), _ptr(k_win), _ptr(v_win),
                                           n_tokens, _ptr(k_pages), _ptr(v_pages), _ptr(page_table),
                                           _ptr(pos0), _ptr(sel_idx), _ptr(sel_count), _ptr(out),
                                           _ptr(lse), _ptr(status), _stream(stream)))


def decode_splits(cfg, batch) -> int:
    return _lib.actqkv_decode_splits(C.byref(cfg), _b(batch))


def decode_workspace_bytes(cfg, batch, n_tokens, n_splits=0) -> int:
    return _lib.actqkv_decode_workspace_bytes(C.byref(cfg), _b(batch), n_tokens, n_splits)


def decode_attention(cfg, batch, q, k_win, v_win, n_tokens, k_pages, v_pages, page_table, pos0,
                     sel_idx, sel_count, out, lse=None, n_splits=0, workspace=None, status=None, stream=None):
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(_lib.actqkv_decode_attention(C.byref(cfg), _b(batch), _ptr(q), _ptr(k_win), _ptr(v_win), n_tokens,
                                        _ptr(k_pages), _ptr(v_pages), _ptr(page_table), _ptr(pos0),
                                        _ptr(sel_idx), _ptr(sel_count), _ptr(out), _ptr(lse), n_splits,
                                        _ptr(workspace), ws_bytes, _ptr(status), _stream(stream)))


STATIC_SCRATCH_BYTES = 8 << 20


def decode_attention_static(cfg, batch, q, k_win, v_win, n_tokens, k_pages, v_pages, page_table, pos0,
                            sel_idx, sel_count, out, lse=None, n_splits=0, status=None, stream=None):
    """The split decode attention with the library's own fixed scratch array: no workspace
    argument and no allocation.  Calls that may overlap on one GPU must not both use it."""
    _check(_lib.actqkv_decode_attention_static(C.byref(cfg), _b(batch), _ptr(q), _ptr(k_win), _ptr(v_win),
                                               n_tokens, _ptr(k_pages), _ptr(v_pages), _ptr(page_table),
                                               _ptr(pos0), _ptr(sel_idx), _ptr(sel_count), _ptr(out), _ptr(lse),
                                               n_splits, _ptr(status), _stream(stream)))


def append_window(cfg, batch, k_win, v_win, n_tokens, pos0, k_pages, v_pages, page_table, repr_k,
                  repr_inv_norm, status=None, stream=None):
    _check(_lib.actqkv_append_window(C.byref(cfg), _b(batch), _ptr(k_win), _ptr(v_win), n_tokens,
                                     _ptr(pos0), _ptr(k_pages), _ptr(v_pages), _ptr(page_table),
                                     _ptr(repr_k), _ptr(repr_inv_norm), _ptr(status), _stream(stream)))


# ----------------------------------------------------------------------------
# device-memory plumbing: the caller-owned state of a batch of (sequence, layer) units
# ----------------------------------------------------------------------------
def make_config(spec, *, n_cap=None, max_pages=None, n_phys_pages=None, beta=1.0,
                stats_mode=STATS_CUMULATIVE, repr_mode=REPR_CHUNK_MEAN, agg_mode=AGG_MEAN,
                thetabar_mode=THETABAR_STREAMING, max_context=None, out_dtype=None,
                probe_mode=PROBE_ACTIVATION, attention_kernel=ATTN_AUTO) -> Config:
    """Config for a `workloads.WorkloadSpec`-like object (any object with the same fields)."""
    ctx = max_context if max_context is not None else spec.context + spec.decode_steps
    pages = -(-ctx // spec.page_tokens)
    cfg = Config()
    cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim = \
        spec.n_layers, spec.n_q_heads, spec.n_kv_heads, spec.head_dim
    cfg.window, cfg.block, cfg.n_repr, cfg.page_tokens = spec.window, spec.block, spec.n_repr, spec.page_tokens
    cfg.n_init, cfg.n_local_prev, cfg.k_blocks, cfg.cap_blocks = \
        spec.n_init, spec.n_local_prev, spec.k_blocks, spec.cap_blocks
    cfg.dtype = BF16 if spec.dtype == "bf16" else F32
    cfg.stats_mode, cfg.repr_mode, cfg.agg_mode, cfg.thetabar_mode = stats_mode, repr_mode, agg_mode, thetabar_mode
    cfg.n_cap = n_cap if n_cap is not None else max(1, (ctx - spec.n_init) // spec.block)
    cfg.max_pages = max_pages if max_pages is not None else pages
    cfg.n_phys_pages = n_phys_pages if n_phys_pages is not None else pages
    cfg.beta, cfg.sm_scale, cfg.var_eps = beta, 0.0, 0.0
    cfg.out_dtype = cfg.dtype if out_dtype is None else out_dtype
    cfg.probe_mode, cfg.attention_kernel = probe_mode, attention_kernel
    return cfg


class RetrievalState:
    """All caller-owned device buffers of n_seq x n_layers units, plus `step()`, which enqueues
    the six stages of one window (or decode step) in the paper's order on the current stream."""

    def __init__(self, cfg: Config, n_seq: int = 1, n_layers: int = 1, layer0: int = 0,
                 device="cuda", page_table=None, keep_phi=False, shared_pages=None):
        self.cfg, self.device = cfg, torch.device(device)
        self.batch = Batch(n_seq, n_layers, layer0)
        U = n_seq * n_layers
        dt, dev = cfg.torch_dtype, self.device
        Hq, Hkv, D, W = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.window
        f32 = dict(dtype=torch.float32, device=dev)
        i32 = dict(dtype=torch.int32, device=dev)
        self.stats_count = torch.zeros(U, Hq, dtype=torch.int64, device=dev)
        self.stats_mean = torch.zeros(U, Hq, D, **f32)
        self.stats_m2 = torch.zeros(U, Hq, D, **f32)
        self.phi_l1 = torch.zeros(U, Hq, W, **f32)
        self.phi_full = torch.zeros(U, W, Hq, D, **f32) if keep_phi else None
        self.probe_qh = torch.zeros(U, Hq, D, **f32)
        self.probe_kv = torch.zeros(U, Hkv, D, **f32)
        self.repr_k = torch.zeros(U, Hkv, cfg.n_cap, cfg.n_repr, D, dtype=dt, device=dev)
        self.repr_inv_norm = torch.zeros(U, Hkv, cfg.n_cap, cfg.n_repr, **f32)
        self.scores = torch.zeros(U, Hkv, cfg.n_cap, **f32)
        self.theta = torch.zeros(U, Hkv, **f32)
        self.sel_idx = torch.full((U, Hkv, max(1, cfg.cap_blocks)), -1, **i32)
        self.sel_count = torch.zeros(U, **i32)
        self.budget_real = torch.zeros(U, **f32)
        self.budget_state = torch.zeros(n_seq, budget_state_bytes(cfg) // 8, dtype=torch.float64, device=dev)
        if shared_pages is not None:
            self.k_pages, self.v_pages = shared_pages
        else:
            self.k_pages = torch.zeros(n_layers, cfg.n_phys_pages, Hkv, cfg.page_tokens, D, dtype=dt, device=dev)
            self.v_pages = torch.zeros_like(self.k_pages)
        if page_table is None:
            page_table = torch.arange(cfg.max_pages, dtype=torch.int32).repeat(n_seq, 1)
        self.page_table = torch.as_tensor(page_table, dtype=torch.int32).reshape(n_seq, cfg.max_pages).to(dev).contiguous()
        self.pos0 = torch.zeros(n_seq, dtype=torch.int64, device=dev)
        self.n_cand = torch.zeros(n_seq, **i32)
        self.status = torch.zeros(1, **i32)
        self.host_pos0 = [0] * n_seq

    def set_positions(self, pos0_list):
        """Host knows where each sequence stands; mirrors it to the device arrays."""
        self.host_pos0 = [int(p) for p in pos0_list]
        self.pos0.copy_(torch.tensor(self.host_pos0, dtype=torch.int64), non_blocking=False)
        nc = [n_candidates(self.cfg, p) for p in self.host_pos0]
        self.n_cand.copy_(torch.tensor(nc, dtype=torch.int32), non_blocking=False)

    def step(self, q, k_win, v_win, out, n_tokens=None, lse=None, fused=True, update_probe=True,
             advance=True, overlap_append=False):
        """bias -> probe -> score -> cut-off/select -> attention -> append for every unit.

        overlap_append: enqueue the append on a second stream, concurrent with the other stages (it
        reads only the step's own K / V and writes pages and table rows that no other stage of the
        same step reads); the streams are joined before the step returns."""
        cfg, b = self.cfg, self.batch
        nt = n_tokens if n_tokens is not None else q.shape[-3]

        def fork_append():
            self._fork.record(main)
            self._side.wait_event(self._fork)
            append_window(cfg, b, k_win, v_win, nt, self.pos0, self.k_pages, self.v_pages, self.page_table,
                          self.repr_k, self.repr_inv_norm, self.status, stream=self._side)
            self._join.record(self._side)

        fork_late = False
        if overlap_append:
            if getattr(self, "_side", None) is None:
                self._side = torch.cuda.Stream(device=self.device)
            if getattr(self, "_fork", None) is None:
                self._fork, self._join = torch.cuda.Event(), torch.cuda.Event()
            main = torch.cuda.current_stream()
            # Where the append forks off.  Inside a graph capture: after the selection, beside the
            # attention (earlier it competes with the short kernels the attention waits for).  With
            # plain launches an event recorded between two kernels of the chain would cost the
            # second one its early start, so the fork sits in front of the whole step.
            fork_late = torch.cuda.is_current_stream_capturing()
            if not fork_late:
                fork_append()
        if update_probe:
            if fused:
                bias_probe(cfg, b, q, nt, self.stats_count, self.stats_mean, self.stats_m2, self.phi_l1,
                           self.phi_full, self.probe_qh, self.probe_kv, self.status)
            else:
                activation_bias(cfg, b, q, nt, self.stats_count, self.stats_mean, self.stats_m2,
                                self.phi_l1, self.phi_full, self.status)
                probe_query(cfg, b, q, nt, self.phi_l1, self.probe_qh, self.probe_kv, self.status)
        if fused:
            score_select(cfg, b, self.probe_kv, self.repr_k, self.repr_inv_norm, self.n_cand,
                         self.budget_state, self.scores, self.theta, self.sel_idx, self.sel_count,
                         self.budget_real, self.status)
        else:
            score_blocks(cfg, b, self.probe_kv, self.repr_k, self.repr_inv_norm, self.n_cand,
                         self.scores, self.theta, self.status)
            select_cutoff(cfg, b, self.scores, self.theta, self.n_cand, self.budget_state, self.sel_idx,
                          self.sel_count, self.budget_real, self.status)
        if fork_late:
            fork_append()
        retrieval_attention(cfg, b, q, k_win, v_win, nt, self.k_pages, self.v_pages, self.page_table,
                            self.pos0, self.sel_idx, self.sel_count, out, lse, self.status)
        if overlap_append:
            main.wait_event(self._join)
        else:
            append_window(cfg, b, k_win, v_win, nt, self.pos0, self.k_pages, self.v_pages, self.page_table,
                          self.repr_k, self.repr_inv_norm, self.status)
        if advance:
            self.set_positions([p + nt for p in self.host_pos0])
