"""ctypes front end of the CPU oracle (``spec_oracle.c``).

Test infrastructure only: the tests, the smoke check and the bench's CPU legs load it; the
product package never does.  Inputs are CPU torch tensors (bf16 for Q/K/V, int32 for lengths
and indices); results come back as fp64 (attention, statistic) or int32 (indices) tensors.

A KV cache is described by any object with the attributes ``k, v`` (bf16 CPU tensors that own
the storage), ``layer_stride, page_stride, head_stride, slot_stride`` (in elements),
``n_layers, page_size, page_table`` (int32 CPU tensor ``[batch, max_pages]`` or ``None``),
``max_pages, batch, n_q_heads, n_kv_heads, head_dim, sm_scale``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spec_oracle.c")
_SRC_CTRL = os.path.join(_HERE, "controller_oracle.c")
_SRC_ACC = os.path.join(_HERE, "accept_oracle.c")
_LIB = os.path.join(_HERE, "libspec_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over the independent (layer, batch, KV head) problems)."""
    newest = max(os.path.getmtime(p) for p in (_SRC, _SRC_CTRL, _SRC_ACC))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest:
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, _SRC_CTRL, _SRC_ACC,
             "-lm"]
        )
    return _LIB


class _KV(ctypes.Structure):
    _fields_ = [
        ("k", ctypes.c_void_p), ("v", ctypes.c_void_p),
        ("layer_stride", ctypes.c_int64), ("page_stride", ctypes.c_int64),
        ("head_stride", ctypes.c_int64), ("slot_stride", ctypes.c_int64),
        ("n_layers", ctypes.c_int32), ("page_size", ctypes.c_int32),
        ("page_table", ctypes.c_void_p),
        ("max_pages", ctypes.c_int32), ("batch", ctypes.c_int32),
        ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32),
        ("sm_scale", ctypes.c_double),
        ("kv_fp8", ctypes.c_int32), ("k_scale", ctypes.c_void_p), ("v_scale", ctypes.c_void_p),
    ]


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_threads.restype = ctypes.c_int
    return _lib


def threads() -> int:
    """Number of OpenMP threads the oracle will use."""
    return int(_load().oracle_threads())


def _cpu(t: torch.Tensor, dtype) -> torch.Tensor:
    assert t.device.type == "cpu" and t.dtype == dtype, (t.device, t.dtype, dtype)
    assert t.is_contiguous()
    return t


def _kv_struct(kv):
    fp8 = bool(getattr(kv, "fp8", False))
    k = _cpu(kv.k, torch.uint8 if fp8 else torch.bfloat16)
    v = _cpu(kv.v, torch.uint8 if fp8 else torch.bfloat16)
    pt = None
    if kv.page_table is not None:
        pt = _cpu(kv.page_table, torch.int32)
    ks = vs = None
    if fp8 and getattr(kv, "k_scale", None) is not None:
        ks, vs = _cpu(kv.k_scale, torch.float32), _cpu(kv.v_scale, torch.float32)
        assert ks.shape == (kv.n_layers, kv.n_kv_heads) and vs.shape == ks.shape
    s = _KV(
        k.data_ptr(), v.data_ptr(), kv.layer_stride, kv.page_stride, kv.head_stride,
        kv.slot_stride, kv.n_layers, kv.page_size, pt.data_ptr() if pt is not None else None,
        kv.max_pages, kv.batch, kv.n_q_heads, kv.n_kv_heads, kv.head_dim,
        float(kv.sm_scale or 0.0), 1 if fp8 else 0,
        ks.data_ptr() if ks is not None else None, vs.data_ptr() if vs is not None else None,
    )
    return s, (k, v, pt, ks, vs)


def e4m3_to_double(byte: int) -> float:
    """The oracle's decoder of one e4m3 byte (exposed for the pins)."""
    lib = _load()
    lib.oracle_e4m3_to_double.restype = ctypes.c_double
    return float(lib.oracle_e4m3_to_double(ctypes.c_int(byte)))


def verify_attn(kv, q, ctx_len, stat_window=16, stat_stride=None, per_head=False, group_max=False):
    """Full-context verification attention and the Eq. 3 statistic.

    Returns ``(out fp64 [L,B,n_q,Hq,D], lse fp64 [L,B,n_q,Hq], stats fp64 [L,B,Hkv,stat_stride])``;
    with ``per_head`` the statistic is kept per attention head: ``[L,B,Hq,stat_stride]``; with
    ``group_max`` it is the largest per-head score of the group at every key (``[L,B,Hkv,stat_stride]``).
    """
    lib = _load()
    s, keep = _kv_struct(kv)
    q = _cpu(q, torch.bfloat16)
    ctx_len = _cpu(ctx_len, torch.int32)
    L, B, n_q, Hq, D = q.shape
    assert (L, B, Hq, D) == (kv.n_layers, kv.batch, kv.n_q_heads, kv.head_dim)
    if stat_stride is None:
        stat_stride = int(ctx_len.max())
    out = torch.zeros(L, B, n_q, Hq, D, dtype=torch.float64)
    lse = torch.zeros(L, B, n_q, Hq, dtype=torch.float64)
    stats = torch.zeros(L, B, Hq if per_head else kv.n_kv_heads, stat_stride, dtype=torch.float64)
    rc = lib.oracle_verify_attn_ex(
        ctypes.byref(s), ctypes.c_void_p(q.data_ptr()), ctypes.c_int(n_q),
        ctypes.c_void_p(ctx_len.data_ptr()), ctypes.c_int(stat_window),
        ctypes.c_void_p(out.data_ptr()), ctypes.c_void_p(lse.data_ptr()),
        ctypes.c_void_p(stats.data_ptr()), ctypes.c_int64(stat_stride),
        ctypes.c_int(2 if group_max else (1 if per_head else 0)),
    )
    if rc != 0:
        raise ValueError("oracle_verify_attn: invalid arguments")
    del keep
    return out, lse, stats


def select_recall(stats, sel_len, k_sink, k_recent, k_total):
    """Eq. 4 index set from fp32 scores ``[L,B,Hkv,stat_stride]``.

    Returns ``(indices int32 [L,B,Hkv,k_total] ascending padded with -1, n_idx int32 [L,B,Hkv])``.
    """
    lib = _load()
    stats = _cpu(stats, torch.float32)
    sel_len = _cpu(sel_len, torch.int32)
    L, B, Hkv, stride = stats.shape
    indices = torch.full((L, B, Hkv, k_total), -7, dtype=torch.int32)
    n_idx = torch.zeros(L, B, Hkv, dtype=torch.int32)
    rc = lib.oracle_select_recall(
        ctypes.c_void_p(stats.data_ptr()), ctypes.c_int64(stride), ctypes.c_int(L),
        ctypes.c_int(B), ctypes.c_int(Hkv), ctypes.c_void_p(sel_len.data_ptr()),
        ctypes.c_int(k_sink), ctypes.c_int(k_recent), ctypes.c_int(k_total),
        ctypes.c_void_p(indices.data_ptr()), ctypes.c_void_p(n_idx.data_ptr()),
    )
    if rc != 0:
        raise ValueError("oracle_select_recall: invalid arguments")
    return indices, n_idx


def sparse_draft_attn(kv, q, indices, n_idx, tail_start, cur_len, per_head=False):
    """Eq. 5 sparse attention of one drafting query per sequence; ``indices`` is ``[L,B,Hkv,k_total]``,
    or ``[L,B,Hq,k_total]`` with ``per_head`` (every attention head gathers its own set).

    Returns ``(out fp64 [L,B,Hq,D], lse fp64 [L,B,Hq])``.
    """
    lib = _load()
    s, keep = _kv_struct(kv)
    q = _cpu(q, torch.bfloat16)
    indices = _cpu(indices, torch.int32)
    n_idx = _cpu(n_idx, torch.int32)
    tail_start = _cpu(tail_start, torch.int32)
    cur_len = _cpu(cur_len, torch.int32)
    L, B, Hq, D = q.shape
    assert (L, B, Hq, D) == (kv.n_layers, kv.batch, kv.n_q_heads, kv.head_dim)
    k_total = indices.shape[-1]
    out = torch.zeros(L, B, Hq, D, dtype=torch.float64)
    lse = torch.zeros(L, B, Hq, dtype=torch.float64)
    assert indices.shape[2] == (Hq if per_head else kv.n_kv_heads)
    rc = lib.oracle_sparse_draft_attn_ex(
        ctypes.byref(s), ctypes.c_void_p(q.data_ptr()), ctypes.c_void_p(indices.data_ptr()),
        ctypes.c_void_p(n_idx.data_ptr()), ctypes.c_int(k_total),
        ctypes.c_void_p(tail_start.data_ptr()), ctypes.c_void_p(cur_len.data_ptr()),
        ctypes.c_void_p(out.data_ptr()), ctypes.c_void_p(lse.data_ptr()), ctypes.c_int(1 if per_head else 0),
    )
    if rc != 0:
        raise ValueError("oracle_sparse_draft_attn: invalid arguments")
    del keep
    return out, lse


# ---- entropy-guided length controller (controller_oracle.c) ------------------------------------


def token_entropy(logits):
    """Shannon entropy (nats) of softmax(logits[r, :]) per row; fp32 or bf16 CPU tensor ``[rows, V]``
    (rows may be strided).  Returns fp64 ``[rows]``."""
    lib = _load()
    assert logits.dim() == 2 and logits.stride(1) == 1 and not logits.is_cuda
    dtype = {torch.float32: 0, torch.bfloat16: 1}[logits.dtype]
    n_rows, vocab = logits.shape
    out = torch.zeros(n_rows, dtype=torch.float64)
    rc = lib.oracle_token_entropy(
        ctypes.c_void_p(logits.data_ptr()), ctypes.c_int(dtype), ctypes.c_int(n_rows), ctypes.c_int(vocab),
        ctypes.c_int64(logits.stride(0)), ctypes.c_void_p(out.data_ptr()))
    if rc != 0:
        raise ValueError("oracle_token_entropy: invalid arguments")
    return out


def controller_update(state, entropy, n_accepted, beta):
    """Eq. "ema": returns the new (mean accepted entropy, mean rejected entropy) as fp64 ``[2]``."""
    lib = _load()
    state = torch.as_tensor(state, dtype=torch.float64).clone().contiguous()
    entropy = torch.as_tensor(entropy, dtype=torch.float64).contiguous()
    rc = lib.oracle_controller_update(
        ctypes.c_void_p(state.data_ptr()), ctypes.c_void_p(entropy.data_ptr()), ctypes.c_int(entropy.numel()),
        ctypes.c_int(int(n_accepted)), ctypes.c_double(float(beta)))
    if rc != 0:
        raise ValueError("oracle_controller_update: invalid arguments")
    return state


def controller_select(state, entropy, cand, c_d, c_v):
    """Eq. "prob" + Eq. "optimal_k": returns ``(k_star, p fp64 [n], score fp64 [n_cand])``."""
    lib = _load()
    state = torch.as_tensor(state, dtype=torch.float64).contiguous()
    entropy = torch.as_tensor(entropy, dtype=torch.float64).contiguous()
    cand = torch.as_tensor(cand, dtype=torch.int32).contiguous()
    k_star = torch.zeros(1, dtype=torch.int32)
    p = torch.zeros(entropy.numel(), dtype=torch.float64)
    score = torch.zeros(cand.numel(), dtype=torch.float64)
    rc = lib.oracle_controller_select(
        ctypes.c_void_p(state.data_ptr()), ctypes.c_void_p(entropy.data_ptr()), ctypes.c_int(entropy.numel()),
        ctypes.c_void_p(cand.data_ptr()), ctypes.c_int(cand.numel()), ctypes.c_double(float(c_d)),
        ctypes.c_double(float(c_v)), ctypes.c_void_p(k_star.data_ptr()), ctypes.c_void_p(p.data_ptr()),
        ctypes.c_void_p(score.data_ptr()))
    if rc != 0:
        raise ValueError("oracle_controller_select: invalid arguments")
    return int(k_star[0]), p, score


def accept_greedy(logits, draft, n_draft=None):
    """Greedy prefix acceptance (Sec. "The Draft-Verification Paradigm").  ``logits``: fp32 or bf16 CPU
    tensor ``[batch, k + 1, V]`` (contiguous); ``draft``: int32 ``[batch, k]``; ``n_draft``: int32
    ``[batch]`` or None.  Returns ``(target [batch, k + 1], n_accepted [batch], next_token [batch])``."""
    lib = _load()
    assert logits.dim() == 3 and logits.is_contiguous() and not logits.is_cuda
    dtype = {torch.float32: 0, torch.bfloat16: 1}[logits.dtype]
    batch, k1, vocab = logits.shape
    draft = torch.as_tensor(draft, dtype=torch.int32).contiguous().view(batch, k1 - 1)
    nd = None if n_draft is None else torch.as_tensor(n_draft, dtype=torch.int32).contiguous()
    target = torch.zeros(batch, k1, dtype=torch.int32)
    n_acc = torch.zeros(batch, dtype=torch.int32)
    nxt = torch.zeros(batch, dtype=torch.int32)
    rc = lib.oracle_accept_greedy(
        ctypes.c_void_p(logits.data_ptr()), ctypes.c_int(dtype), ctypes.c_int(batch), ctypes.c_int(k1),
        ctypes.c_int(vocab), ctypes.c_int64(vocab), ctypes.c_void_p(draft.data_ptr() if draft.numel() else None),
        ctypes.c_void_p(None if nd is None else nd.data_ptr()), ctypes.c_void_p(target.data_ptr()),
        ctypes.c_void_p(n_acc.data_ptr()), ctypes.c_void_p(nxt.data_ptr()))
    if rc != 0:
        raise ValueError("oracle_accept_greedy: invalid arguments")
    return target, n_acc, nxt
