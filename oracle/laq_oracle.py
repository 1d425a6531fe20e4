"""ctypes access to the fp64 CPU oracle (``laq_oracle.c``) -- TEST INFRASTRUCTURE ONLY.

The oracle states what Section 4.3 (Eq. 4) computes in plain loops; this module only compiles it
with gcc, marshals numpy arrays and holds no arithmetic of the method. It shares nothing with the
CUDA library and is imported only by the tests, the smoke check and the benchmark's CPU baseline.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "laq_oracle.c")
_LIB = os.path.join(_HERE, "liblaq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compiles the oracle with gcc (-O2, OpenMP over units) if the library is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
    return _LIB


class _Variant(ctypes.Structure):
    _fields_ = [("W_local", ctypes.c_int32), ("pool_mode", ctypes.c_int32),
                ("score_mode", ctypes.c_int32), ("group_mode", ctypes.c_int32),
                ("seq_lens", ctypes.c_void_p)]


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, i, d, i64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_double, ctypes.c_int64
        lib.laq_oracle_unit_colsum.argtypes = [vp, vp, i, i, i, i, d, vp, vp, vp]
        lib.laq_oracle_unit_colsum.restype = None
        lib.laq_oracle_unit_colsum_local.argtypes = [vp, vp, i, i, i, i, i, d, vp, vp, vp]
        lib.laq_oracle_unit_colsum_local.restype = None
        lib.laq_oracle_pool.argtypes = [vp, i, i, vp]
        lib.laq_oracle_pool.restype = None
        lib.laq_oracle_select.argtypes = [vp, i, i, i, vp]
        lib.laq_oracle_select.restype = None
        lib.laq_oracle_select_sorted.argtypes = [vp, i, i, i, vp]
        lib.laq_oracle_select_sorted.restype = None
        lib.laq_oracle_compact.argtypes = [vp, vp, i, i, vp]
        lib.laq_oracle_compact.restype = None
        lib.laq_oracle_evict.argtypes = [vp, vp, vp, i, i, i, i, i, i, i, i, i, i, d, vp, i64,
                                         vp, vp, vp, vp, vp, i]
        lib.laq_oracle_evict.restype = i
        lib.laq_oracle_recall.argtypes = [vp, i, vp, i, vp]
        lib.laq_oracle_recall.restype = d
        lib.laq_oracle_evict_local.argtypes = [vp, vp, vp, i, i, i, i, i, i, i, i, i, i, i, d, vp, i64,
                                               vp, vp, vp, vp, vp, i]
        lib.laq_oracle_evict_local.restype = i
        lib.laq_oracle_pool_max.argtypes = [vp, i, i, vp]
        lib.laq_oracle_pool_max.restype = None
        lib.laq_oracle_unit_rawsum.argtypes = [vp, vp, i, i, i, i, d, vp]
        lib.laq_oracle_unit_rawsum.restype = None
        lib.laq_oracle_evict_variant.argtypes = [vp, vp, vp, i, i, i, i, i, i, i, i, i, i, d,
                                                 ctypes.POINTER(_Variant), vp, i64,
                                                 vp, vp, vp, vp, vp, i]
        lib.laq_oracle_evict_variant.restype = i
        lib.laq_oracle_unit_colsum_heads.argtypes = [vp, vp, i, i, i, i, i, d, vp, i64]
        lib.laq_oracle_unit_colsum_heads.restype = None
        lib.laq_oracle_group_reduce.argtypes = [vp, i, i, i, vp]
        lib.laq_oracle_group_reduce.restype = None
        _lib = lib
    return _lib


def _bits(a) -> np.ndarray:
    """bf16 bit patterns as a C-contiguous uint16 array (accepts uint16 numpy or a bf16 CPU tensor)."""
    if not isinstance(a, np.ndarray):  # torch tensor, bf16 or int16/uint16 view
        import torch

        a = a.detach().cpu().contiguous()
        if a.dtype == torch.bfloat16:
            a = a.view(torch.int16)
        a = a.numpy()
    return np.ascontiguousarray(a).view(np.uint16)


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def unit_colsum(q, k, scale=None, local_window=0):
    """q [G][W][D], k [L][D] bf16 -> (c [L], row_max [G*W], row_sum [G*W]) in fp64. With
    `local_window` > 0 the first that many queries of each head are the causal queries of the last
    prompt positions (the unified window of LAQ++, Eq. 5)."""
    q, k = _bits(q), _bits(k)
    G, W, D = q.shape
    L = k.shape[0]
    assert k.shape[1] == D
    scale = 1.0 / np.sqrt(D) if scale is None else float(scale)
    c = np.empty(L, np.float64)
    m = np.empty(G * W, np.float64)
    l = np.empty(G * W, np.float64)
    _load().laq_oracle_unit_colsum_local(_ptr(q), _ptr(k), G, W, int(local_window), D, L, scale,
                                         _ptr(c), _ptr(m), _ptr(l))
    return c, m, l


def unit_colsum_heads(q, k, scale=None, local_window=0):
    """q [G][W][D], k [L][D] bf16 -> c_heads [G][L]: the column sums of every query head on its own."""
    q, k = _bits(q), _bits(k)
    G, W, D = q.shape
    L = k.shape[0]
    scale = 1.0 / np.sqrt(D) if scale is None else float(scale)
    ch = np.zeros((G, L), np.float64)
    _load().laq_oracle_unit_colsum_heads(_ptr(q), _ptr(k), G, W, int(local_window), D, L, scale,
                                         _ptr(ch), L)
    return ch


def group_reduce(c_heads, mode):
    """[G][L] per-head column sums -> [L]: mode 0 adds the heads, mode 1 takes the largest."""
    ch = np.ascontiguousarray(c_heads, np.float64)
    c = np.empty(ch.shape[1], np.float64)
    _load().laq_oracle_group_reduce(_ptr(ch), ch.shape[0], ch.shape[1], int(mode), _ptr(c))
    return c


def pool(c, Ls, kernel, mode=0):
    """mode 0: average pooling (zero padding, divisor k); mode 1: maximum pooling."""
    c = np.ascontiguousarray(c, np.float64)
    assert c.shape[0] >= Ls
    p = np.empty(Ls, np.float64)
    fn = _load().laq_oracle_pool_max if mode == 1 else _load().laq_oracle_pool
    fn(_ptr(c), Ls, kernel, _ptr(p))
    return p


def unit_rawsum(q, k, scale=None):
    """q [G][W][D], k [L][D] (bf16) -> c [L]: sums of the raw scaled logits over the window rows."""
    q, k = _bits(q), _bits(k)
    G, W, D = q.shape
    L = k.shape[0]
    scale = 1.0 / np.sqrt(D) if scale is None else float(scale)
    c = np.empty(L, np.float64)
    _load().laq_oracle_unit_rawsum(_ptr(q), _ptr(k), G, W, D, L, scale, _ptr(c))
    return c


def select(p, L, R, B, sorted_variant=False):
    """p [L-R] scores (any float dtype, promoted exactly to fp64) -> idx [B] int32."""
    p = np.ascontiguousarray(p, np.float64)
    assert p.shape[0] == L - R and 0 <= R < B <= L
    idx = np.empty(B, np.int32)
    fn = _load().laq_oracle_select_sorted if sorted_variant else _load().laq_oracle_select
    fn(_ptr(p), L, R, B, _ptr(idx))
    return idx


def recall(pred, gold):
    """(|pred n gold| / |gold|, |pred n gold|) for two sets of distinct positions (Eq. 1-3)."""
    pred = np.ascontiguousarray(pred, np.int32)
    gold = np.ascontiguousarray(gold, np.int32)
    n = np.zeros(1, np.int32)
    r = _load().laq_oracle_recall(_ptr(pred), pred.shape[0], _ptr(gold), gold.shape[0], _ptr(n))
    return float(r), int(n[0])


def compact(src, idx):
    src = _bits(src)
    idx = np.ascontiguousarray(idx, np.int32)
    dst = np.empty((idx.shape[0], src.shape[1]), np.uint16)
    _load().laq_oracle_compact(_ptr(src), _ptr(idx), idx.shape[0], src.shape[1], _ptr(dst))
    return dst


def evict(q, k, v, R, kernel, B, scale=None, units=None, want_colsum=False, fast_select=True,
          want_idx=True, local_window=0, pool_mode=0, score_mode=0, seq_lens=None, group_mode=0):
    """Whole step on dense tensors. q [NL][Bt][Hq][W][D], k/v [NL][Bt][Hkv][L][D] (bf16).

    Returns a dict with 'scores' [NL,Bt,Hkv,L-R] fp64, 'idx' [NL,Bt,Hkv,B] int32, 'k_out',
    'v_out' [NL,Bt,Hkv,B,D] uint16 bit patterns, 'threads', and 'colsum' if asked. With `units`
    (unit numbers (layer*Bt+b)*Hkv+h) only those units are computed; the rest stays zero.
    `pool_mode` 1 pools by maximum, `score_mode` 1 sums raw logits instead of attention weights,
    `seq_lens` [Bt] gives every prompt its own length (<= L). `group_mode` 1 combines the query
    heads of a group by maximum instead of sum; 2 lets every query head select for itself, and the
    outputs then have Hq in place of Hkv.
    """
    q, k = _bits(q), _bits(k)
    v = None if v is None else _bits(v)
    NL, Bt, Hq, W, D = q.shape
    Hkv, L = k.shape[2], k.shape[3]
    assert k.shape == (NL, Bt, Hkv, L, D) and Hq % Hkv == 0
    scale = 1.0 / np.sqrt(D) if scale is None else float(scale)
    Ls = L - R
    Ho = Hq if group_mode == 2 else Hkv   # heads of the outputs
    scores = np.zeros((NL, Bt, Ho, Ls), np.float64)
    colsum = np.zeros((NL, Bt, Ho, L), np.float64) if want_colsum else None
    idx = np.zeros((NL, Bt, Ho, B), np.int32) if want_idx else None
    k_out = np.zeros((NL, Bt, Ho, B, D), np.uint16) if want_idx else None
    v_out = np.zeros((NL, Bt, Ho, B, D), np.uint16) if (want_idx and v is not None) else None
    ul = None if units is None else np.ascontiguousarray(units, np.int64)
    sl = None if seq_lens is None else np.ascontiguousarray(seq_lens, np.int32)
    assert sl is None or (sl.shape == (Bt,) and (sl <= L).all() and (sl > B).all())
    assert group_mode == 0 or score_mode == 0
    var = _Variant(int(local_window), int(pool_mode), int(score_mode), int(group_mode), _ptr(sl))
    threads = _load().laq_oracle_evict_variant(
        _ptr(q), _ptr(k), _ptr(v), NL, Bt, Hq, Hkv, D, L, W, R, kernel, B, scale, ctypes.byref(var),
        _ptr(ul), 0 if ul is None else ul.shape[0], _ptr(scores), _ptr(colsum), _ptr(idx), _ptr(k_out),
        _ptr(v_out), 1 if fast_select else 0)
    out = {"scores": scores, "idx": idx, "k_out": k_out, "v_out": v_out, "threads": threads}
    if want_colsum:
        out["colsum"] = colsum
    return out


def evict_layers(q, k, v, R, kernel, budgets, **kw):
    """One budget per layer (layer-wise budgets, Sections 5.1-5.2): layer n is evicted on its own
    with budgets[n], and the results are laid end to end in one ragged pool, layer after layer,
    each layer as [Bt][Hkv][budgets[n]] entries. Returns {'idx' [entries] int32, 'k_out', 'v_out'
    [entries][D] uint16, 'scores' [NL,Bt,Hkv,L-R]}. Keyword arguments as for evict()."""
    q, k = _bits(q), _bits(k)
    v = None if v is None else _bits(v)
    NL = q.shape[0]
    assert len(budgets) == NL
    idx, k_out, v_out, scores = [], [], [], []
    for n in range(NL):
        r = evict(q[n:n + 1], k[n:n + 1], None if v is None else v[n:n + 1], R, kernel, int(budgets[n]), **kw)
        idx.append(r["idx"].reshape(-1))
        k_out.append(r["k_out"].reshape(-1, k.shape[-1]))
        if v is not None:
            v_out.append(r["v_out"].reshape(-1, k.shape[-1]))
        scores.append(r["scores"])
    return {"idx": np.concatenate(idx), "k_out": np.concatenate(k_out),
            "v_out": np.concatenate(v_out) if v is not None else None,
            "scores": np.concatenate(scores)}


def streaming_indices(L, B, n_sink, seq_len=None):
    """The keep-set of a StreamingLLM-style cache for one prompt, as the literal list: the first
    n_sink positions and the last B - n_sink positions of the prompt's Lb = seq_len or L."""
    Lb = L if seq_len is None else int(seq_len)
    assert 0 <= n_sink <= B < Lb <= L
    return np.array(list(range(n_sink)) + list(range(Lb - (B - n_sink), Lb)), np.int32)
