"""ctypes binding of ``libspec_attn.so``: argument marshalling only.

Every function takes CUDA torch tensors (torch is used for device memory and streams), checks
dtypes/devices, passes raw pointers through the C ABI of ``include/spec_attn.h`` and raises
``SpecError`` on a non-zero return code.  There is no CPU fallback: if the library is missing
or the tensors are not on a CUDA device the call fails.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspec_attn.so")

WS_VERIFY, WS_SELECT, WS_DRAFT = 0, 1, 2
VERIFY_AUTO, VERIFY_GENERIC, VERIFY_TCGEN05, VERIFY_TCGEN05_TWOSWEEP, VERIFY_TCGEN05_CACHED = 0, 1, 2, 3, 4
VERIFY_TCGEN05_CACHED_2PASS = 5
# ^ reported by last_verify_impl() only: the score-cache kernel on two halves of the rows
VERIFY_TCGEN05_CACHED_EXPANDED = 6
# ^ reported only: an 8-bit cache expanded to bf16 in the workspace first (head_dim 64)
VERIFY_ACCUMULATE_STATS = 1  # flag of spec_verify_attn_ex: add to the statistic instead of replacing it
VERIFY_STATS_PER_QUERY_HEAD = 2  # flag of spec_verify_attn_ex: one score per attention head
DRAFT_INDICES_PER_QUERY_HEAD = 1  # flag of spec_sparse_draft_attn_ex: one index set per attention head
VERIFY_OUT_BF16 = 4  # flag of spec_verify_attn_ex: bf16 attention output
VERIFY_STATS_GROUP_MAX = 8  # flag of spec_verify_attn_ex: fold the group's per-head scores by max, not sum
DRAFT_OUT_BF16 = 2  # flag of spec_sparse_draft_attn_ex: bf16 attention output
DRAFT_EARLY_GATHER = 4  # flag of spec_sparse_draft_attn_ex: index sets, lengths and recalled rows are older than the
#                         preceding kernel of the stream, so the gather may start before that kernel has finished

EXPORTS = [
    "spec_verify_attn", "spec_select_recall", "spec_sparse_draft_attn", "spec_workspace_bytes",
    "spec_read_status", "spec_set_verify_impl", "spec_last_verify_impl", "spec_launch_count",
    "spec_strerror", "spec_version", "spec_verify_attn_noalloc", "spec_noalloc_scratch_bytes",
    "spec_noalloc_read_status", "spec_token_entropy", "spec_controller_update", "spec_controller_select",
    "spec_token_argmax", "spec_accept_greedy", "spec_verify_attn_ex",
    "spec_sparse_draft_attn_ex", "spec_advance_lengths", "spec_set_wait_limit_cycles",
    "spec_verify_attn_hist", "spec_select_recall_hist", "spec_describe_plan",
]


class SpecError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


class _KV(ctypes.Structure):
    _fields_ = [
        ("k", ctypes.c_void_p), ("v", ctypes.c_void_p),
        ("layer_stride", ctypes.c_int64), ("page_stride", ctypes.c_int64),
        ("head_stride", ctypes.c_int64), ("slot_stride", ctypes.c_int64),
        ("n_layers", ctypes.c_int32), ("page_size", ctypes.c_int32),
        ("page_table", ctypes.c_void_p),
        ("max_pages", ctypes.c_int32), ("batch", ctypes.c_int32),
        ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("n_pages", ctypes.c_int32), ("sm_scale", ctypes.c_float),
        ("kv_dtype", ctypes.c_int32), ("k_scale", ctypes.c_void_p), ("v_scale", ctypes.c_void_p),
    ]


_lib = None


def load() -> ctypes.CDLL:
    """Loads the compiled library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: run `python -m paper_2607_27735_b200.build` "
                "(there is no fallback implementation)")
        lib = ctypes.CDLL(LIB_PATH)
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        lib.spec_verify_attn.argtypes = [ctypes.POINTER(_KV), vp, i32, vp, i32, i32, vp, vp, vp,
                                         i64, vp, ctypes.c_size_t, vp]
        lib.spec_verify_attn_ex.argtypes = [ctypes.POINTER(_KV), vp, i32, vp, i32, i32, vp, vp, vp,
                                            i64, vp, ctypes.c_size_t, ctypes.c_uint32, vp]
        lib.spec_verify_attn_hist.argtypes = [ctypes.POINTER(_KV), vp, i32, vp, i32, i32, vp, vp, vp,
                                              i64, vp, ctypes.c_size_t, ctypes.c_uint32, vp, vp]
        lib.spec_select_recall_hist.argtypes = [vp, i64, i32, i32, i32, vp, i32, i32, i32, vp, vp, vp, vp, vp,
                                                ctypes.c_size_t, vp]
        lib.spec_sparse_draft_attn_ex.argtypes = [ctypes.POINTER(_KV), vp, vp, vp, i32, vp, vp, i32,
                                                  vp, vp, vp, ctypes.c_size_t, ctypes.c_uint32, vp]
        lib.spec_select_recall.argtypes = [vp, i64, i32, i32, i32, vp, i32, i32, i32, vp, vp, vp,
                                           ctypes.c_size_t, vp]
        lib.spec_sparse_draft_attn.argtypes = [ctypes.POINTER(_KV), vp, vp, vp, i32, vp, vp, i32,
                                               vp, vp, vp, ctypes.c_size_t, vp]
        lib.spec_verify_attn_noalloc.argtypes = [ctypes.POINTER(_KV), vp, i32, vp, i32, i32, vp, vp,
                                                 vp, i64, vp]
        lib.spec_noalloc_scratch_bytes.restype = ctypes.c_size_t
        lib.spec_noalloc_read_status.argtypes = [vp]
        f32 = ctypes.c_float
        lib.spec_token_entropy.argtypes = [vp, i32, i32, i32, i64, vp, vp]
        lib.spec_token_argmax.argtypes = [vp, i32, i32, i32, i64, vp, vp, vp]
        lib.spec_accept_greedy.argtypes = [vp, i32, i32, i32, i32, i64, vp, vp, vp, vp, vp, vp]
        lib.spec_advance_lengths.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp, vp]
        lib.spec_controller_update.argtypes = [vp, vp, i32, vp, f32, vp]
        lib.spec_controller_select.argtypes = [vp, vp, i32, vp, i32, f32, f32, vp, vp, vp, vp]
        lib.spec_workspace_bytes.argtypes = [ctypes.c_int, ctypes.POINTER(_KV), i32, i32, i32]
        lib.spec_workspace_bytes.restype = ctypes.c_size_t
        lib.spec_read_status.argtypes = [vp, vp]
        lib.spec_describe_plan.argtypes = [ctypes.c_int, ctypes.POINTER(_KV), i32, i32, i32, ctypes.POINTER(i32 * 8)]
        lib.spec_set_verify_impl.argtypes = [ctypes.c_int]
        lib.spec_set_wait_limit_cycles.argtypes = [ctypes.c_int64]
        lib.spec_set_wait_limit_cycles.restype = ctypes.c_int64
        lib.spec_launch_count.restype = ctypes.c_int64
        lib.spec_strerror.argtypes = [ctypes.c_int]
        lib.spec_strerror.restype = ctypes.c_char_p
        _lib = lib
    return _lib


def strerror(code: int) -> str:
    return load().spec_strerror(code).decode()


def _dev(t: torch.Tensor, dtype, name: str) -> int:
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (no CPU path exists)")
    if t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{name}: expected contiguous {dtype}, got {t.dtype}")
    return t.data_ptr()


KV_BF16, KV_FP8_E4M3 = 0, 1


def _kv_struct(kv) -> _KV:
    fp8 = bool(getattr(kv, "fp8", False))
    _dev(kv.k, torch.uint8 if fp8 else torch.bfloat16, "kv.k")
    _dev(kv.v, torch.uint8 if fp8 else torch.bfloat16, "kv.v")
    pt = None if kv.page_table is None else _dev(kv.page_table, torch.int32, "kv.page_table")
    ks = vs = None
    if fp8 and getattr(kv, "k_scale", None) is not None:
        ks = _dev(kv.k_scale, torch.float32, "kv.k_scale")
        vs = _dev(kv.v_scale, torch.float32, "kv.v_scale")
    return _KV(kv.k.data_ptr(), kv.v.data_ptr(), kv.layer_stride, kv.page_stride, kv.head_stride,
               kv.slot_stride, kv.n_layers, kv.page_size, pt, kv.max_pages, kv.batch,
               kv.n_q_heads, kv.n_kv_heads, kv.head_dim, int(getattr(kv, "n_pages", 0) or 0),
               float(kv.sm_scale or 0.0), KV_FP8_E4M3 if fp8 else KV_BF16, ks, vs)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def workspace_bytes(which: int, kv, n_q: int = 1, max_ctx_len: int = 1, k_total: int = 1) -> int:
    return int(load().spec_workspace_bytes(which, ctypes.byref(_kv_struct(kv)), n_q, max_ctx_len,
                                           k_total))


def alloc_workspace(nbytes: int, device) -> torch.Tensor:
    """A zeroed, 256-byte aligned byte tensor (torch's caching allocator aligns to 512 bytes)."""
    ws = torch.zeros(max(int(nbytes), 256), dtype=torch.uint8, device=device)
    assert ws.data_ptr() % 256 == 0
    return ws


def spec_verify_attn(kv, q, ctx_len, max_ctx_len, stat_window=16, out=None, lse=None, stats=None,
                     stat_stride=None, workspace=None, want_lse=True, accumulate=False, per_head=False,
                     out_bf16=False, score_hist=None, group_max=False):
    """Verification attention + Eq. 3 statistic; returns ``(out, lse, stats, workspace)``.
    ``score_hist`` (uint32-as-int32 ``[L, B, heads, 2048]``, zero before the first use) receives the
    selection's first radix pass (spec_verify_attn_hist).
    ``accumulate`` adds this call's statistic to the given ``stats``; ``per_head`` keeps one score per
    attention head (``stats`` is ``[L, B, n_q_heads, stride]``); both go through spec_verify_attn_ex."""
    lib = load()
    L, B, n_q, Hq, D = q.shape
    dev = q.device
    s = _kv_struct(kv)
    if stat_stride is None:
        stat_stride = (max_ctx_len + 63) // 64 * 64 if stats is None else stats.shape[-1]
    out_dtype = torch.bfloat16 if out_bf16 else torch.float32
    if out is None:
        out = torch.empty(L, B, n_q, Hq, D, dtype=out_dtype, device=dev)
    if lse is None and want_lse:
        lse = torch.empty(L, B, n_q, Hq, dtype=torch.float32, device=dev)
    if stats is None:
        stats = torch.zeros(L, B, kv.n_q_heads if per_head else kv.n_kv_heads, stat_stride,
                            dtype=torch.float32, device=dev)
    if workspace is None:
        workspace = alloc_workspace(workspace_bytes(WS_VERIFY, kv, n_q, max_ctx_len), dev)
    if accumulate and stats is None:
        raise ValueError("accumulate needs the stats tensor that holds the running sums")
    args = (ctypes.byref(s), _dev(q, torch.bfloat16, "q"), n_q, _dev(ctx_len, torch.int32, "ctx_len"),
            max_ctx_len, stat_window, _dev(out, out_dtype, "out"),
            None if lse is None else _dev(lse, torch.float32, "lse"),
            _dev(stats, torch.float32, "stats"), stat_stride, workspace.data_ptr(), workspace.numel())
    if stats.shape[2] != (kv.n_q_heads if per_head else kv.n_kv_heads):
        raise ValueError("stats: wrong head count for this mode")
    flags = ((VERIFY_ACCUMULATE_STATS if accumulate else 0) | (VERIFY_STATS_PER_QUERY_HEAD if per_head else 0) |
             (VERIFY_OUT_BF16 if out_bf16 else 0) | (VERIFY_STATS_GROUP_MAX if group_max else 0))
    if score_hist is not None:
        if score_hist.shape != stats.shape[:3] + (2048,):
            raise ValueError("score_hist: expected [L, B, heads, 2048]")
        rc = lib.spec_verify_attn_hist(*args, flags, _dev(score_hist, torch.int32, "score_hist"), _stream())
    elif flags:
        rc = lib.spec_verify_attn_ex(*args, flags, _stream())
    else:
        rc = lib.spec_verify_attn(*args, _stream())
    if rc != 0:
        raise SpecError(rc, "spec_verify_attn")
    return out, lse, stats, workspace


def spec_verify_attn_noalloc(kv, q, ctx_len, max_ctx_len, stat_window=16, out=None, lse=None,
                             stats=None, want_lse=True):
    """spec_verify_attn on the library's built-in scratch, for callers that cannot allocate a
    workspace (a plugin inside a runtime that owns all device memory).  The output tensors are
    still the caller's; this wrapper creates them only when they are not passed in.
    Returns ``(out, lse, stats)``."""
    lib = load()
    L, B, n_q, Hq, D = q.shape
    dev = q.device
    s = _kv_struct(kv)
    if out is None:
        out = torch.empty(L, B, n_q, Hq, D, dtype=torch.float32, device=dev)
    if lse is None and want_lse:
        lse = torch.empty(L, B, n_q, Hq, dtype=torch.float32, device=dev)
    if stats is None:
        stats = torch.zeros(L, B, kv.n_kv_heads, (max_ctx_len + 63) // 64 * 64,
                            dtype=torch.float32, device=dev)
    rc = lib.spec_verify_attn_noalloc(
        ctypes.byref(s), _dev(q, torch.bfloat16, "q"), n_q, _dev(ctx_len, torch.int32, "ctx_len"),
        max_ctx_len, stat_window, _dev(out, torch.float32, "out"),
        None if lse is None else _dev(lse, torch.float32, "lse"),
        _dev(stats, torch.float32, "stats"), stats.shape[-1], _stream())
    if rc != 0:
        raise SpecError(rc, "spec_verify_attn_noalloc")
    return out, lse, stats


def noalloc_scratch_bytes() -> int:
    return int(load().spec_noalloc_scratch_bytes())


def noalloc_read_status() -> int:
    return int(load().spec_noalloc_read_status(_stream()))


def spec_select_recall(stats, sel_len, k_sink, k_recent, k_total, indices=None, n_indices=None,
                       score_hist=None, hist_len=None):
    """Eq. 4 recall selection; returns ``(indices, n_indices)``.  ``score_hist`` / ``hist_len``: the
    counts a verification call left (spec_select_recall_hist); they are cleared."""
    lib = load()
    L, B, Hkv, stride = stats.shape
    dev = stats.device
    if indices is None:
        indices = torch.empty(L, B, Hkv, k_total, dtype=torch.int32, device=dev)
    if n_indices is None:
        n_indices = torch.empty(L, B, Hkv, dtype=torch.int32, device=dev)
    if score_hist is not None:
        rc = lib.spec_select_recall_hist(
            _dev(stats, torch.float32, "stats"), stride, L, B, Hkv,
            _dev(sel_len, torch.int32, "sel_len"), k_sink, k_recent, k_total,
            _dev(indices, torch.int32, "indices"), _dev(n_indices, torch.int32, "n_indices"),
            _dev(score_hist, torch.int32, "score_hist"), _dev(hist_len, torch.int32, "hist_len"), None, 0, _stream())
    else:
        rc = lib.spec_select_recall(
            _dev(stats, torch.float32, "stats"), stride, L, B, Hkv,
            _dev(sel_len, torch.int32, "sel_len"), k_sink, k_recent, k_total,
            _dev(indices, torch.int32, "indices"), _dev(n_indices, torch.int32, "n_indices"), None, 0,
            _stream())
    if rc != 0:
        raise SpecError(rc, "spec_select_recall")
    return indices, n_indices


def spec_sparse_draft_attn(kv, q, indices, n_indices, tail_start, cur_len, max_tail, out=None,
                           lse=None, workspace=None, want_lse=True, per_head=False, out_bf16=False,
                           early_gather=False):
    """Eq. 5 sparse draft attention; returns ``(out, lse, workspace)``.  ``per_head``: ``indices`` is
    ``[L, B, n_q_heads, k_total]``, one set per attention head (spec_sparse_draft_attn_ex).
    ``early_gather``: the caller's promise behind SPEC_DRAFT_EARLY_GATHER (see the header)."""
    lib = load()
    L, B, Hq, D = q.shape
    dev = q.device
    s = _kv_struct(kv)
    k_total = indices.shape[-1]
    out_dtype = torch.bfloat16 if out_bf16 else torch.float32
    if out is None:
        out = torch.empty(L, B, Hq, D, dtype=out_dtype, device=dev)
    if lse is None and want_lse:
        lse = torch.empty(L, B, Hq, dtype=torch.float32, device=dev)
    if workspace is None:
        workspace = alloc_workspace(workspace_bytes(WS_DRAFT, kv, k_total=k_total + max_tail), dev)
    if indices.shape[2] != (kv.n_q_heads if per_head else kv.n_kv_heads):
        raise ValueError("indices: wrong head count for this mode")
    args = (ctypes.byref(s), _dev(q, torch.bfloat16, "q"), _dev(indices, torch.int32, "indices"),
            _dev(n_indices, torch.int32, "n_indices"), k_total,
            _dev(tail_start, torch.int32, "tail_start"), _dev(cur_len, torch.int32, "cur_len"),
            max_tail, _dev(out, out_dtype, "out"),
            None if lse is None else _dev(lse, torch.float32, "lse"), workspace.data_ptr(),
            workspace.numel())
    if per_head or out_bf16 or early_gather:
        flags = ((DRAFT_INDICES_PER_QUERY_HEAD if per_head else 0) | (DRAFT_OUT_BF16 if out_bf16 else 0) |
                 (DRAFT_EARLY_GATHER if early_gather else 0))
        rc = lib.spec_sparse_draft_attn_ex(*args, flags, _stream())
    else:
        rc = lib.spec_sparse_draft_attn(*args, _stream())
    if rc != 0:
        raise SpecError(rc, "spec_sparse_draft_attn")
    return out, lse, workspace


def spec_token_entropy(logits, entropy=None):
    """Entropy (nats) of softmax(logits[r]) per row; ``logits`` is [rows, vocab] fp32 or bf16 with a
    unit inner stride (rows may be strided).  Returns ``entropy`` ([rows] fp32)."""
    if not logits.is_cuda or logits.dim() != 2 or logits.stride(1) != 1:
        raise ValueError("logits: expected a CUDA [rows, vocab] tensor with unit inner stride")
    if logits.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError(f"logits: expected fp32 or bf16, got {logits.dtype}")
    rows, vocab = logits.shape
    if entropy is None:
        entropy = torch.empty(rows, dtype=torch.float32, device=logits.device)
    rc = load().spec_token_entropy(logits.data_ptr(), 1 if logits.dtype == torch.bfloat16 else 0, rows, vocab,
                                   logits.stride(0) if rows > 1 else max(logits.stride(0), vocab),
                                   _dev(entropy, torch.float32, "entropy"), _stream())
    if rc != 0:
        raise SpecError(rc, "spec_token_entropy")
    return entropy


def _logits_2d(logits):
    if not logits.is_cuda or logits.dim() != 2 or logits.stride(1) != 1:
        raise ValueError("logits: expected a CUDA [rows, vocab] tensor with unit inner stride")
    if logits.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError(f"logits: expected fp32 or bf16, got {logits.dtype}")
    rows, vocab = logits.shape
    return rows, vocab, 1 if logits.dtype == torch.bfloat16 else 0, max(logits.stride(0), vocab)


def spec_token_argmax(logits, token=None, entropy=None, want_entropy=False):
    """Greedy token per row (smallest index of the largest logit), optionally with the row's entropy
    from the same pass.  Returns ``(token, entropy or None)``."""
    rows, vocab, dt, stride = _logits_2d(logits)
    if token is None:
        token = torch.empty(rows, dtype=torch.int32, device=logits.device)
    if entropy is None and want_entropy:
        entropy = torch.empty(rows, dtype=torch.float32, device=logits.device)
    rc = load().spec_token_argmax(logits.data_ptr(), dt, rows, vocab, stride, _dev(token, torch.int32, "token"),
                                  None if entropy is None else _dev(entropy, torch.float32, "entropy"), _stream())
    if rc != 0:
        raise SpecError(rc, "spec_token_argmax")
    return token, entropy


def spec_accept_greedy(logits, draft, n_draft=None, target=None, n_accepted=None, next_token=None):
    """Greedy prefix acceptance; ``logits`` is a contiguous CUDA ``[batch, k + 1, vocab]`` tensor, ``draft``
    int32 ``[batch, k]``.  Returns device tensors ``(target, n_accepted, next_token)``."""
    if not logits.is_cuda or logits.dim() != 3 or not logits.is_contiguous():
        raise ValueError("logits: expected a contiguous CUDA [batch, k + 1, vocab] tensor")
    if logits.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError(f"logits: expected fp32 or bf16, got {logits.dtype}")
    batch, k1, vocab = logits.shape
    dev = logits.device
    if target is None:
        target = torch.empty(batch, k1, dtype=torch.int32, device=dev)
    if n_accepted is None:
        n_accepted = torch.empty(batch, dtype=torch.int32, device=dev)
    if next_token is None:
        next_token = torch.empty(batch, dtype=torch.int32, device=dev)
    rc = load().spec_accept_greedy(
        logits.data_ptr(), 1 if logits.dtype == torch.bfloat16 else 0, batch, k1, vocab, vocab,
        _dev(draft, torch.int32, "draft") if k1 > 1 else None,
        None if n_draft is None else _dev(n_draft, torch.int32, "n_draft"), _dev(target, torch.int32, "target"),
        _dev(n_accepted, torch.int32, "n_accepted"), _dev(next_token, torch.int32, "next_token"), _stream())
    if rc != 0:
        raise SpecError(rc, "spec_accept_greedy")
    return target, n_accepted, next_token


def spec_advance_lengths(committed, n_accepted, k, ctx_verify=None, cur_len=None, max_len=0, workspace=None):
    """committed += n_accepted + 1 on the device (``n_accepted=None``: unchanged), then the lengths of the
    next round: ``ctx_verify`` [batch] and ``cur_len`` [k, batch] (both optional, int32).  ``max_len`` > 0
    holds a sequence whose next round would not fit the cache and records that in ``workspace``."""
    rc = load().spec_advance_lengths(
        _dev(committed, torch.int32, "committed"),
        None if n_accepted is None else _dev(n_accepted, torch.int32, "n_accepted"), committed.numel(), k,
        int(max_len), None if workspace is None else workspace.data_ptr(),
        None if ctx_verify is None else _dev(ctx_verify, torch.int32, "ctx_verify"),
        None if cur_len is None else _dev(cur_len, torch.int32, "cur_len"), _stream())
    if rc != 0:
        raise SpecError(rc, "spec_advance_lengths")
    return committed


def spec_controller_update(state, entropy, n_accepted, beta):
    """Eq. "ema" in place on ``state`` ([2] fp32: accepted mean, rejected mean); ``n_accepted`` is a
    device int32 scalar tensor."""
    rc = load().spec_controller_update(_dev(state, torch.float32, "state"), _dev(entropy, torch.float32, "entropy"),
                                       entropy.numel(), _dev(n_accepted, torch.int32, "n_accepted"), float(beta),
                                       _stream())
    if rc != 0:
        raise SpecError(rc, "spec_controller_update")
    return state


def spec_controller_select(state, entropy, cand, c_d, c_v, k_star=None, p=None, score=None):
    """Eq. "prob" + Eq. "optimal_k"; returns device tensors ``(k_star, p, score)``."""
    dev = entropy.device
    if k_star is None:
        k_star = torch.empty(1, dtype=torch.int32, device=dev)
    if p is None:
        p = torch.empty(entropy.numel(), dtype=torch.float32, device=dev)
    if score is None:
        score = torch.empty(cand.numel(), dtype=torch.float32, device=dev)
    rc = load().spec_controller_select(
        _dev(state, torch.float32, "state"), _dev(entropy, torch.float32, "entropy"), entropy.numel(),
        _dev(cand, torch.int32, "cand"), cand.numel(), float(c_d), float(c_v), _dev(k_star, torch.int32, "k_star"),
        _dev(p, torch.float32, "p"), _dev(score, torch.float32, "score"), _stream())
    if rc != 0:
        raise SpecError(rc, "spec_controller_select")
    return k_star, p, score


def read_status(workspace) -> int:
    return int(load().spec_read_status(workspace.data_ptr(), _stream()))


def describe_plan(which: int, kv_struct, n_q: int = 1, max_ctx_len: int = 1, k_total: int = 1):
    """Host-side split of a call (spec_describe_plan); ``kv_struct`` is a ``binding._KV`` (no tensors needed,
    so this works without a GPU).  Returns the eight integers as a list."""
    out = (ctypes.c_int32 * 8)()
    rc = load().spec_describe_plan(which, ctypes.byref(kv_struct), n_q, max_ctx_len, k_total, ctypes.byref(out))
    if rc != 0:
        raise SpecError(rc, "spec_describe_plan")
    return list(out)


def set_wait_limit_cycles(cycles: int) -> int:
    """Sets the bound of the device-side waits in SM clocks; returns the previous one."""
    return int(load().spec_set_wait_limit_cycles(int(cycles)))


def set_verify_impl(impl: int) -> int:
    return int(load().spec_set_verify_impl(impl))


def last_verify_impl() -> int:
    return int(load().spec_last_verify_impl())


def launch_count() -> int:
    return int(load().spec_launch_count())
