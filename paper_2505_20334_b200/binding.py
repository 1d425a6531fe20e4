"""Thin ctypes binding of the C-ABI library ``liblaq`` (see ``include/laq.h``).

Argument marshalling only: every step of the eviction path (Section 4.3, Eq. 4) runs in the
library's CUDA kernels. PyTorch supplies device memory and the current stream. There is no CPU
fallback: if ``liblaq.so`` has not been built, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblaq.so")

LAQ_OK = 0
LAQ_ERR_INVALID_ARG = 1
LAQ_ERR_UNSUPPORTED = 2
LAQ_ERR_WORKSPACE = 3
LAQ_ERR_CUDA = 4
LAQ_ERR_TIMEOUT = 5
LAQ_ERR_INTERNAL = 6
LAQ_POOL_AVG, LAQ_POOL_MAX = 0, 1
LAQ_SCORE_SOFTMAX, LAQ_SCORE_RAW = 0, 1
LAQ_GROUP_SUM, LAQ_GROUP_MAX, LAQ_GROUP_PER_HEAD = 0, 1, 2

EXPORTS = (
    "laq_params_dense_strides", "laq_workspace_bytes", "laq_score", "laq_select", "laq_compact",
    "laq_evict", "laq_last_device_status", "laq_last_launch_count", "laq_status_string",
    "laq_version", "laq_set_stage_events", "laq_host_staging_bytes", "laq_evict_host",
    "laq_score_static", "laq_recall", "laq_last_kernel_clock", "laq_evict_layers",
    "laq_layers_pool_entries", "laq_streaming_indices",
)


class LaqParams(ctypes.Structure):
    """Mirror of ``laq_params`` (field order and types as in laq.h)."""

    _fields_ = [(n, ctypes.c_int32) for n in (
        "n_layers", "batch", "n_q_heads", "n_kv_heads", "head_dim", "prompt_len", "window_len",
        "keep_tail", "pool_kernel", "pool_mode", "budget")] + [("softmax_scale", ctypes.c_float),
        ("tiles_per_task", ctypes.c_int32), ("sched_lag_tasks", ctypes.c_int32),
        ("local_window", ctypes.c_int32), ("score_mode", ctypes.c_int32),
        ("group_mode", ctypes.c_int32), ("reserved0", ctypes.c_int32)] + [
        (f"{t}_stride_{d}", ctypes.c_int64) for t in ("q", "k", "v", "o")
        for d in ("layer", "batch", "head", "pos")] + [("seq_lens", ctypes.POINTER(ctypes.c_int32))]

    def set_seq_lens(self, lens) -> None:
        """Per-prompt lengths (a sequence of `batch` ints, or None). The host array the C struct
        points to is kept alive by this object."""
        if lens is None:
            self._seq_lens_buf = None
            self.seq_lens = ctypes.POINTER(ctypes.c_int32)()
            return
        lens = [int(x) for x in lens]
        if len(lens) != self.batch:
            raise ValueError("seq_lens: one length per batch item is required")
        self._seq_lens_buf = (ctypes.c_int32 * len(lens))(*lens)
        self.seq_lens = ctypes.cast(self._seq_lens_buf, ctypes.POINTER(ctypes.c_int32))


class LaqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (laq_status {status})")


def load_library(path: str = LIB_PATH) -> ctypes.CDLL:
    """Loads a build of the library and declares the argument types of its entry points."""
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python -m paper_2505_20334_b200.build` "
            "(there is no fallback path)")
    lib = ctypes.CDLL(path)
    vp, sz, pp = ctypes.c_void_p, ctypes.c_size_t, ctypes.POINTER(LaqParams)
    lib.laq_params_dense_strides.argtypes = [pp]
    lib.laq_params_dense_strides.restype = None
    lib.laq_workspace_bytes.argtypes = [pp]
    lib.laq_workspace_bytes.restype = sz
    lib.laq_score.argtypes = [pp, vp, vp, vp, vp, sz, vp]
    lib.laq_score.restype = ctypes.c_int
    lib.laq_score_static.argtypes = [pp, vp, vp, vp, vp]
    lib.laq_score_static.restype = ctypes.c_int
    lib.laq_recall.argtypes = [ctypes.c_int64, vp, ctypes.c_int32, vp, ctypes.c_int32, vp, vp, vp]
    lib.laq_recall.restype = ctypes.c_int
    lib.laq_select.argtypes = [pp, vp, vp, vp]
    lib.laq_select.restype = ctypes.c_int
    lib.laq_compact.argtypes = [pp, vp, vp, vp, vp, vp, vp]
    lib.laq_compact.restype = ctypes.c_int
    lib.laq_evict.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.laq_evict.restype = ctypes.c_int
    lib.laq_last_device_status.argtypes = [pp, vp, sz, vp]
    lib.laq_last_device_status.restype = ctypes.c_int
    lib.laq_last_launch_count.argtypes = []
    lib.laq_last_launch_count.restype = ctypes.c_int
    lib.laq_status_string.argtypes = [ctypes.c_int]
    lib.laq_status_string.restype = ctypes.c_char_p
    lib.laq_host_staging_bytes.argtypes = [pp]
    lib.laq_host_staging_bytes.restype = sz
    lib.laq_evict_host.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, sz, vp, sz, vp]
    lib.laq_evict_host.restype = ctypes.c_int
    lib.laq_set_stage_events.argtypes = [vp, vp]
    lib.laq_set_stage_events.restype = None
    lib.laq_last_kernel_clock.argtypes = [vp, sz, vp, ctypes.POINTER(ctypes.c_int64),
                                          ctypes.POINTER(ctypes.c_int64)]
    lib.laq_last_kernel_clock.restype = ctypes.c_int
    i32p = ctypes.POINTER(ctypes.c_int32)
    lib.laq_evict_layers.argtypes = [pp, i32p, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.laq_evict_layers.restype = ctypes.c_int
    lib.laq_layers_pool_entries.argtypes = [pp, i32p]
    lib.laq_layers_pool_entries.restype = sz
    lib.laq_streaming_indices.argtypes = [pp, ctypes.c_int32, vp, vp]
    lib.laq_streaming_indices.restype = ctypes.c_int
    lib.laq_version.argtypes = []
    lib.laq_version.restype = ctypes.c_int
    return lib


lib = load_library()


def status_string(status: int) -> str:
    return lib.laq_status_string(int(status)).decode()


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def make_params(n_layers, batch, n_q_heads, n_kv_heads, head_dim, prompt_len, window_len,
                keep_tail, pool_kernel, budget, softmax_scale=0.0, q=None, k=None, v=None,
                out=None) -> LaqParams:
    """Fills ``laq_params``; strides are dense unless 5-D tensors are given to take them from."""
    p = LaqParams()
    p.n_layers, p.batch, p.n_q_heads, p.n_kv_heads = n_layers, batch, n_q_heads, n_kv_heads
    p.head_dim, p.prompt_len, p.window_len, p.keep_tail = head_dim, prompt_len, window_len, keep_tail
    p.pool_kernel, p.pool_mode, p.budget, p.softmax_scale = pool_kernel, 0, budget, softmax_scale
    lib.laq_params_dense_strides(ctypes.byref(p))
    for name, t in (("q", q), ("k", k), ("v", v), ("o", out)):
        if t is not None:
            if t.dim() != 5 or t.stride(4) != 1:
                raise ValueError(f"{name}: expected a 5-D tensor with unit innermost stride")
            for i, d in enumerate(("layer", "batch", "head", "pos")):
                setattr(p, f"{name}_stride_{d}", t.stride(i))
    return p


def params_for(q: torch.Tensor, k: torch.Tensor, keep_tail: int, pool_kernel: int, budget: int,
               v: Optional[torch.Tensor] = None, out: Optional[torch.Tensor] = None,
               softmax_scale: float = 0.0) -> LaqParams:
    """``laq_params`` for q [NL,Bt,Hq,W,D] and k [NL,Bt,Hkv,L,D] (strides taken from the tensors)."""
    NL, Bt, Hq, W, D = q.shape
    Hkv, L = k.shape[2], k.shape[3]
    return make_params(NL, Bt, Hq, Hkv, D, L, W, keep_tail, pool_kernel, budget, softmax_scale,
                       q=q, k=k, v=v, out=out)


def laq_workspace_bytes(p: LaqParams) -> int:
    return int(lib.laq_workspace_bytes(ctypes.byref(p)))


def alloc_workspace(p: LaqParams, device) -> torch.Tensor:
    n = laq_workspace_bytes(p)
    if n == 0:
        raise LaqError(LAQ_ERR_INVALID_ARG, "laq_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def _ws_args(ws: Optional[torch.Tensor]):
    return _ptr(ws), (0 if ws is None else ws.numel() * ws.element_size())


def laq_score(p: LaqParams, q, k, scores, ws, stream=None, check=True) -> int:
    wp, wn = _ws_args(ws)
    st = lib.laq_score(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(scores), wp, wn, _stream(stream))
    if check and st != LAQ_OK:
        raise LaqError(st, "laq_score")
    return st


STATIC_SCRATCH_BYTES = 8 * 1024 * 1024


def laq_score_static(p: LaqParams, q, k, scores, stream=None, check=True) -> int:
    """``laq_score`` without a workspace argument, for callers that may not allocate device memory:
    the scratch is a fixed ``STATIC_SCRATCH_BYTES`` array inside the library. Calls share that
    array, so two of them must not overlap on the GPU; problems whose scratch does not fit are
    refused with ``LAQ_ERR_WORKSPACE``."""
    st = lib.laq_score_static(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(scores), _stream(stream))
    if check and st != LAQ_OK:
        raise LaqError(st, "laq_score_static")
    return st


def laq_recall(idx_pred: torch.Tensor, idx_gold: torch.Tensor, stream=None):
    """Recall of `idx_pred` against `idx_gold` (Eq. 1-3) for index tensors [..., B] with ascending
    rows; returns (recall fp32 [...], n_common int32 [...])."""
    n_pred, n_gold = idx_pred.shape[-1], idx_gold.shape[-1]
    lead = idx_pred.shape[:-1]
    if idx_gold.shape[:-1] != lead:
        raise ValueError("laq_recall: the two index tensors must agree in all but the last dim")
    a, g = idx_pred.contiguous(), idx_gold.contiguous()
    n_units = a.numel() // n_pred
    common = torch.empty(lead, dtype=torch.int32, device=a.device)
    rec = torch.empty(lead, dtype=torch.float32, device=a.device)
    st = lib.laq_recall(n_units, _ptr(a), n_pred, _ptr(g), n_gold, _ptr(common), _ptr(rec),
                        _stream(stream))
    if st != LAQ_OK:
        raise LaqError(st, "laq_recall")
    return rec, common


def laq_select(p: LaqParams, scores, idx, stream=None, check=True) -> int:
    st = lib.laq_select(ctypes.byref(p), _ptr(scores), _ptr(idx), _stream(stream))
    if check and st != LAQ_OK:
        raise LaqError(st, "laq_select")
    return st


def laq_compact(p: LaqParams, k, v, idx, k_out, v_out, stream=None, check=True) -> int:
    st = lib.laq_compact(ctypes.byref(p), _ptr(k), _ptr(v), _ptr(idx), _ptr(k_out), _ptr(v_out),
                         _stream(stream))
    if check and st != LAQ_OK:
        raise LaqError(st, "laq_compact")
    return st


def laq_evict(p: LaqParams, q, k, v, k_out, v_out, idx, scores, ws, stream=None, check=True) -> int:
    wp, wn = _ws_args(ws)
    st = lib.laq_evict(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(k_out), _ptr(v_out),
                       _ptr(idx), _ptr(scores), wp, wn, _stream(stream))
    if check and st != LAQ_OK:
        raise LaqError(st, "laq_evict")
    return st


def laq_last_device_status(p: LaqParams, ws, stream=None) -> int:
    wp, wn = _ws_args(ws)
    return int(lib.laq_last_device_status(ctypes.byref(p), wp, wn, _stream(stream)))


def laq_last_kernel_clock(ws, stream=None):
    """(SM cycles, nanoseconds) the first block of the last tensor-core scoring launch on `ws` ran for."""
    wp, wn = _ws_args(ws)
    cyc, ns = ctypes.c_int64(0), ctypes.c_int64(0)
    st = lib.laq_last_kernel_clock(wp, wn, _stream(stream), ctypes.byref(cyc), ctypes.byref(ns))
    if st != LAQ_OK:
        raise LaqError(st, "laq_last_kernel_clock")
    return int(cyc.value), int(ns.value)


def laq_last_launch_count() -> int:
    return int(lib.laq_last_launch_count())


def laq_set_stage_events(begin=None, end=None) -> None:
    """begin/end: recorded torch.cuda.Event objects (enable_timing=True) or None to clear."""
    b = None if begin is None else ctypes.c_void_p(begin.cuda_event)
    e = None if end is None else ctypes.c_void_p(end.cuda_event)
    lib.laq_set_stage_events(b, e)


def laq_version() -> int:
    return int(lib.laq_version())


def evict(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, budget: int, pool_kernel: int = 7,
          keep_tail: Optional[int] = None, want_scores: bool = False, ws=None, stream=None,
          softmax_scale: float = 0.0, local_window: int = 0, pool_mode: int = 0,
          score_mode: int = 0, seq_lens=None, group_mode: int = 0):
    """Convenience call: allocates the outputs with torch and runs ``laq_evict``.

    q [NL,Bt,Hq,W,D], k and v [NL,Bt,Hkv,L,D], bf16 CUDA tensors. Returns a dict with 'k_out',
    'v_out' [NL,Bt,Hkv,B,D], 'idx' [NL,Bt,Hkv,B] int32 and, if asked, 'scores' [NL,Bt,Hkv,L-R]
    (with ``group_mode = LAQ_GROUP_PER_HEAD`` every query head selects for itself and the outputs
    have Hq in place of Hkv).
    """
    if not (q.is_cuda and k.is_cuda and v.is_cuda):
        raise ValueError("evict: q, k and v must be CUDA tensors (there is no CPU path)")
    NL, Bt, Hq, W, D = q.shape
    Hkv, L = k.shape[2], k.shape[3]
    R = W if keep_tail is None else keep_tail
    Ho = Hq if group_mode == LAQ_GROUP_PER_HEAD else Hkv
    k_out = torch.empty((NL, Bt, Ho, budget, D), dtype=k.dtype, device=k.device)
    v_out = torch.empty_like(k_out)
    idx = torch.empty((NL, Bt, Ho, budget), dtype=torch.int32, device=k.device)
    scores = torch.empty((NL, Bt, Ho, L - R), dtype=torch.float32, device=k.device) if want_scores else None
    p = params_for(q, k, R, pool_kernel, budget, v=v, out=k_out)
    p.group_mode = group_mode        # how the query heads of a GQA group combine
    p.softmax_scale = softmax_scale  # 0 selects 1/sqrt(head_dim)
    p.local_window = local_window    # > 0: LAQ++ unified window (Eq. 5)
    p.pool_mode = pool_mode          # LAQ_POOL_AVG / LAQ_POOL_MAX
    p.score_mode = score_mode        # LAQ_SCORE_SOFTMAX / LAQ_SCORE_RAW (Eq. 4 read literally)
    p.set_seq_lens(seq_lens)         # prompts of different lengths in one batch
    if ws is None:
        ws = alloc_workspace(p, k.device)
    laq_evict(p, q, k, v, k_out, v_out, idx, scores, ws, stream)
    out = {"k_out": k_out, "v_out": v_out, "idx": idx, "ws": ws, "params": p}
    if want_scores:
        out["scores"] = scores
    return out



def _budget_array(budgets):
    return (ctypes.c_int32 * len(budgets))(*[int(b) for b in budgets])


def laq_layers_pool_entries(p: LaqParams, budgets) -> int:
    return int(lib.laq_layers_pool_entries(ctypes.byref(p), _budget_array(budgets)))


def laq_evict_layers(p: LaqParams, budgets, q, k, v, k_out, v_out, idx, scores, ws, stream=None,
                     check=True) -> int:
    """``laq_evict`` with one budget per layer; idx / k_out / v_out are one ragged pool (laq.h)."""
    wp, wn = _ws_args(ws)
    st = lib.laq_evict_layers(ctypes.byref(p), _budget_array(budgets), _ptr(q), _ptr(k), _ptr(v),
                              _ptr(k_out), _ptr(v_out), _ptr(idx), _ptr(scores), wp, wn, _stream(stream))
    if check and st != LAQ_OK:
        raise LaqError(st, "laq_evict_layers")
    return st


def laq_streaming_indices(p: LaqParams, n_sink: int, idx, stream=None, check=True) -> int:
    st = lib.laq_streaming_indices(ctypes.byref(p), int(n_sink), _ptr(idx), _stream(stream))
    if check and st != LAQ_OK:
        raise LaqError(st, "laq_streaming_indices")
    return st


def evict_layer_budgets(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, budgets, pool_kernel: int = 7,
                        keep_tail: Optional[int] = None, local_window: int = 0, stream=None,
                        seq_lens=None):
    """Eviction with one budget per layer (the paper fixes the budget, Section 5.2, and names
    layer-wise budgets such as PyramidKV's as a combination): one ``laq_evict_layers`` call that
    writes the compressed caches of all layers into one ragged pool. Returns the pool tensors and a
    list with one dict of views per layer ('k_out', 'v_out' [Bt,Hkv,B_l,D], 'idx' [Bt,Hkv,B_l])."""
    NL, Bt, Hq, W, D = q.shape
    Hkv = k.shape[2]
    if len(budgets) != NL:
        raise ValueError("evict_layer_budgets: one budget per layer is required")
    R = W if keep_tail is None else keep_tail
    p = params_for(q, k, R, pool_kernel, max(int(b) for b in budgets), v=v)
    p.local_window = local_window
    p.set_seq_lens(seq_lens)
    entries = laq_layers_pool_entries(p, budgets)
    if entries == 0:
        raise LaqError(LAQ_ERR_INVALID_ARG, "laq_layers_pool_entries")
    idx = torch.empty(entries, dtype=torch.int32, device=k.device)
    k_out = torch.empty((entries, D), dtype=k.dtype, device=k.device)
    v_out = torch.empty_like(k_out)
    ws = alloc_workspace(p, k.device)
    laq_evict_layers(p, budgets, q, k, v, k_out, v_out, idx, None, ws, stream)
    layers, row = [], 0
    for n in range(NL):
        B = int(budgets[n])
        cnt = Bt * Hkv * B
        layers.append({"k_out": k_out[row:row + cnt].view(Bt, Hkv, B, D),
                       "v_out": v_out[row:row + cnt].view(Bt, Hkv, B, D),
                       "idx": idx[row:row + cnt].view(Bt, Hkv, B)})
        row += cnt
    return {"idx": idx, "k_out": k_out, "v_out": v_out, "layers": layers, "params": p, "ws": ws}


def laq_host_staging_bytes(p: LaqParams) -> int:
    return int(lib.laq_host_staging_bytes(ctypes.byref(p)))


def laq_evict_host(p: LaqParams, q_host, k_host, v_host, k_out_host, v_out_host, idx_host, staging,
                   ws, stream=None, check=True) -> int:
    """Host tensors in, host tensors out (see laq.h); `staging` and `ws` are CUDA byte tensors."""
    sp, sn = _ws_args(staging)
    wp, wn = _ws_args(ws)
    st = lib.laq_evict_host(ctypes.byref(p), _ptr(q_host), _ptr(k_host), _ptr(v_host),
                            _ptr(k_out_host), _ptr(v_out_host), _ptr(idx_host), sp, sn, wp, wn,
                            _stream(stream))
    if check and st != LAQ_OK:
        raise LaqError(st, "laq_evict_host")
    return st


class HostEvictor:
    """Buffers for repeated ``laq_evict_host`` calls on one problem shape: device staging and
    workspace, pinned host outputs. Only moves bytes; every step of the path runs in the kernels."""

    def __init__(self, q_shape, k_shape, budget: int, pool_kernel: int = 7,
                 keep_tail: Optional[int] = None, device="cuda"):
        NL, Bt, Hq, W, D = q_shape
        Hkv, L = k_shape[2], k_shape[3]
        R = W if keep_tail is None else keep_tail
        self.params = make_params(NL, Bt, Hq, Hkv, D, L, W, R, pool_kernel, budget)
        self.ws = alloc_workspace(self.params, device)
        self.staging = torch.empty(laq_host_staging_bytes(self.params), dtype=torch.uint8, device=device)
        self.h_k_out = torch.empty((NL, Bt, Hkv, budget, D), dtype=torch.bfloat16, pin_memory=True)
        self.h_v_out = torch.empty_like(self.h_k_out).pin_memory()
        self.h_idx = torch.empty((NL, Bt, Hkv, budget), dtype=torch.int32, pin_memory=True)
        self.h2d_bytes = 2 * (NL * Bt * Hq * W * D + 2 * NL * Bt * Hkv * L * D)
        self.d2h_bytes = 2 * 2 * self.h_k_out.numel() + 4 * self.h_idx.numel()

    def run(self, q_host, k_host, v_host, stream=None):
        for t in (q_host, k_host, v_host):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError("laq_evict_host takes dense host tensors")
        laq_evict_host(self.params, q_host, k_host, v_host, self.h_k_out, self.h_v_out, self.h_idx,
                       self.staging, self.ws, stream)
        # bytes that cross the bus towards the device: Q and K in full; V in full if it has to be
        # staged, else only the kept rows, which the gather reads from the pinned host tensor
        v_bytes = (self.h_v_out.numel() if v_host.is_pinned() else v_host.numel()) * 2
        self.h2d_bytes = 2 * (q_host.numel() + k_host.numel()) + v_bytes
        return self.h_k_out, self.h_v_out, self.h_idx
