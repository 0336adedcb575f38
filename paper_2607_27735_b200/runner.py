"""One speculative step of the attention hot path on a resident KV cache.

``SpecStepRunner`` owns the output buffers and workspaces of a workload and issues the three
phases through the C ABI on the current stream:

  verify phase : per layer, ``spec_verify_attn`` (dense attention of the k+1 rows + Eq. 3 score)
  select phase : ``spec_select_recall`` for every layer in one launch (the index sets are only
                 needed by the next drafting round, so the layers are independent problems here)
  draft phase  : per drafting step and layer, ``spec_sparse_draft_attn`` (Eq. 5)

``fold_layers=True`` issues verify and draft with ``n_layers = L`` in one launch instead
(independent problems; a kernel-roofline view, not the layer-by-layer dependency chain of a
real decoder).  The phases can be captured into CUDA graphs to take the Python/ctypes launch
cost out of the timed region.
"""
from __future__ import annotations

import torch

from . import binding


class SpecStepRunner:
    def __init__(self, case, fold_layers: bool = False, want_lse: bool = False, per_head: bool = False,
                 fused_hist: bool = False):
        cfg, kv = case.cfg, case.kv
        self.case, self.cfg, self.kv = case, cfg, kv
        self.fold = fold_layers
        self.per_head = per_head  # one score and one index set per attention head (Eq. 3 / Eq. 5 as printed)
        self.fused_hist = fused_hist  # the verification kernel counts the selection's first radix pass
        n_sets = kv.n_q_heads if per_head else kv.n_kv_heads
        dev = kv.k.device
        L, B = kv.n_layers, kv.batch
        self.L = L
        self.max_ctx = int(case.ctx_len.max())
        self.stat_stride = (self.max_ctx + 127) // 128 * 128
        self.out_v = torch.empty(L, B, cfg.n_q, kv.n_q_heads, kv.head_dim, device=dev)
        self.lse_v = torch.empty(L, B, cfg.n_q, kv.n_q_heads, device=dev) if want_lse else None
        self.stats = torch.zeros(L, B, n_sets, self.stat_stride, device=dev)
        self.indices = torch.empty(L, B, n_sets, cfg.k_total, dtype=torch.int32, device=dev)
        self.n_idx = torch.empty(L, B, n_sets, dtype=torch.int32, device=dev)
        self.hist = torch.zeros(L, B, n_sets, 2048, dtype=torch.int32, device=dev) if fused_hist else None
        self.out_d = torch.empty(max(cfg.draft_steps, 1), L, B, kv.n_q_heads, kv.head_dim, device=dev)
        self.q_verify = case.q_verify
        self.q_draft = case.q_draft
        self.ctx_len = case.ctx_len
        self.tail_start = case.ctx_len.clone()
        self.cur_lens = [(case.ctx_len + j + 1).contiguous() for j in range(cfg.draft_steps)]
        kvs = kv if fold_layers else kv.layer_slice(0, 1)
        self.ws_v = binding.alloc_workspace(
            binding.workspace_bytes(binding.WS_VERIFY, kvs, cfg.n_q, self.max_ctx), dev)
        self.ws_d = binding.alloc_workspace(
            binding.workspace_bytes(binding.WS_DRAFT, kvs, k_total=cfg.k_total + cfg.draft_steps), dev)
        self._layers = [kv.layer_slice(l, l + 1) for l in range(L)]
        self.graphs = None

    # -- phases ----------------------------------------------------------------------------
    def verify_phase(self):
        if self.fold:
            binding.spec_verify_attn(self.kv, self.q_verify, self.ctx_len, self.max_ctx,
                                     self.cfg.stat_window, out=self.out_v, lse=self.lse_v,
                                     stats=self.stats, workspace=self.ws_v, want_lse=False,
                                     per_head=self.per_head, score_hist=self.hist)
            return
        for l in range(self.L):
            binding.spec_verify_attn(
                self._layers[l], self.q_verify[l:l + 1], self.ctx_len, self.max_ctx,
                self.cfg.stat_window, out=self.out_v[l:l + 1],
                lse=None if self.lse_v is None else self.lse_v[l:l + 1],
                stats=self.stats[l:l + 1], workspace=self.ws_v, want_lse=False, per_head=self.per_head,
                score_hist=None if self.hist is None else self.hist[l:l + 1])

    def select_phase(self):
        c = self.cfg
        binding.spec_select_recall(self.stats, self.ctx_len, c.k_sink, c.k_recent, c.k_total,
                                   indices=self.indices, n_indices=self.n_idx, score_hist=self.hist,
                                   hist_len=None if self.hist is None else self.ctx_len)

    def draft_phase(self):
        c = self.cfg
        # The index sets and every step's lengths are complete before the phase begins, so every call
        # but the first (whose predecessor in the stream may be their producer) may gather early.
        first = True
        for j in range(c.draft_steps):
            if self.fold:
                binding.spec_sparse_draft_attn(
                    self.kv, self.q_draft[j], self.indices, self.n_idx, self.tail_start,
                    self.cur_lens[j], c.draft_steps, out=self.out_d[j], workspace=self.ws_d,
                    want_lse=False, per_head=self.per_head, early_gather=not first)
                first = False
                continue
            for l in range(self.L):
                binding.spec_sparse_draft_attn(
                    self._layers[l], self.q_draft[j, l:l + 1], self.indices[l:l + 1],
                    self.n_idx[l:l + 1], self.tail_start, self.cur_lens[j], c.draft_steps,
                    out=self.out_d[j, l:l + 1], workspace=self.ws_d, want_lse=False, per_head=self.per_head,
                    early_gather=not first)
                first = False

    def step(self):
        self.verify_phase()
        self.select_phase()
        self.draft_phase()

    # -- CUDA graphs -----------------------------------------------------------------------
    def capture(self):
        """Captures the three phases into three CUDA graphs (after one eager warm-up step).
        Returns the number of kernels each phase launches."""
        self.step()
        torch.cuda.synchronize()
        graphs, counts = [], []
        for phase in (self.verify_phase, self.select_phase, self.draft_phase):
            g = torch.cuda.CUDAGraph()
            before = binding.launch_count()
            with torch.cuda.graph(g):
                phase()
            counts.append(binding.launch_count() - before)
            graphs.append(g)
        self.graphs = graphs
        self.launches_per_phase = counts
        return counts

    def replay(self, events=None):
        """Replays the captured step; ``events`` = 4 CUDA events recorded around the phases."""
        for i, g in enumerate(self.graphs):
            if events is not None:
                events[i].record()
            g.replay()
        if events is not None:
            events[3].record()

    def replay_host_io(self, q_verify_host, q_draft_host, out_v_host, out_d_host):
        """One captured step fed from and drained to pinned host buffers.  The copies that a phase
        does not wait for travel on a second stream: the drafting Q arrives under the verification
        phase, the verification outputs leave under selection and drafting.  Every copy of the step
        is finished (in stream order) when the current stream reaches the end of this call."""
        main = torch.cuda.current_stream()
        if not hasattr(self, "_side"):
            self._side = torch.cuda.Stream()
        side = self._side
        self.q_verify.copy_(q_verify_host, non_blocking=True)
        side.wait_stream(main)  # the previous step's drafting phase has read q_draft
        with torch.cuda.stream(side):
            self.q_draft.copy_(q_draft_host, non_blocking=True)
            q_draft_in = side.record_event()
        self.graphs[0].replay()
        verified = main.record_event()
        with torch.cuda.stream(side):
            side.wait_event(verified)
            out_v_host.copy_(self.out_v, non_blocking=True)
            out_v_gone = side.record_event()
        self.graphs[1].replay()
        main.wait_event(q_draft_in)
        self.graphs[2].replay()
        out_d_host.copy_(self.out_d, non_blocking=True)
        main.wait_event(out_v_gone)

    # -- algorithmic bytes (what the method must move) ---------------------------------------
    def verify_kv_bytes_per_layer(self) -> int:
        kv = self.kv
        return int(self.ctx_len.sum()) * kv.n_kv_heads * kv.head_dim * 2 * 2

    def draft_kv_bytes_per_layer_step(self, j: int) -> int:
        kv, c = self.kv, self.cfg
        rows = sum(min(c.k_total, int(t)) + j + 1 for t in self.ctx_len.tolist())
        return rows * (kv.n_q_heads if self.per_head else kv.n_kv_heads) * kv.head_dim * 2 * 2


class SpecLoopRunner:
    """Speculation rounds chained on the device: draft k steps -> verify -> greedy prefix acceptance
    -> speculation-length controller -> commit m + 1 tokens -> rebuild the recall index, with every
    length in device memory, so that one captured graph is replayed round after round.  The model
    around the attention is absent: the caller supplies each round's verification logits and drafted
    tokens (``logits``, ``draft_tokens`` are overwritten between replays); K/V of every position the
    loop can reach already sit in the cache.  All layers go in one launch per call."""

    def __init__(self, case, committed, vocab: int, c_d: float = 0.05, c_v: float = 1.0, beta: float = 0.9):
        cfg, kv = case.cfg, case.kv
        assert cfg.n_q == cfg.draft_steps + 1, "a round verifies the k drafted tokens plus one"
        self.case, self.cfg, self.kv = case, cfg, kv
        dev = kv.k.device
        L, B, k = kv.n_layers, kv.batch, cfg.draft_steps
        self.k, self.beta, self.c_d, self.c_v = k, beta, c_d, c_v
        self.max_ctx = kv.max_pages * kv.page_size if kv.page_table is not None else int(case.ctx_len.max()) + k + 1
        self.committed = committed.to(device=dev, dtype=torch.int32).clone()
        self.ctx_verify = torch.empty(B, dtype=torch.int32, device=dev)
        self.cur_len = torch.empty(k, B, dtype=torch.int32, device=dev)
        self.stat_stride = (self.max_ctx + 127) // 128 * 128
        self.stats = torch.zeros(L, B, kv.n_kv_heads, self.stat_stride, device=dev)
        self.indices = torch.empty(L, B, kv.n_kv_heads, cfg.k_total, dtype=torch.int32, device=dev)
        self.n_idx = torch.empty(L, B, kv.n_kv_heads, dtype=torch.int32, device=dev)
        self.out_v = torch.empty(L, B, cfg.n_q, kv.n_q_heads, kv.head_dim, device=dev)
        self.out_d = torch.empty(k, L, B, kv.n_q_heads, kv.head_dim, device=dev)
        self.logits = torch.empty(B, k + 1, vocab, dtype=torch.bfloat16, device=dev)
        self.draft_tokens = torch.zeros(B, k, dtype=torch.int32, device=dev)
        self.target = torch.empty(B, k + 1, dtype=torch.int32, device=dev)
        self.n_accepted = torch.zeros(B, dtype=torch.int32, device=dev)
        self.next_token = torch.empty(B, dtype=torch.int32, device=dev)
        self.entropy = torch.empty(k, device=dev)           # of sequence 0's drafted tokens
        self.state = torch.tensor([1.0, 4.0], device=dev)   # tracked mean entropy of accepted / rejected tokens
        self.cand = torch.arange(1, k + 1, dtype=torch.int32, device=dev)
        self.k_star = torch.zeros(1, dtype=torch.int32, device=dev)
        self.p = torch.empty(k, device=dev)
        self.score = torch.empty(k, device=dev)
        self.ws_v = binding.alloc_workspace(binding.workspace_bytes(binding.WS_VERIFY, kv, cfg.n_q, self.max_ctx), dev)
        self.ws_d = binding.alloc_workspace(binding.workspace_bytes(binding.WS_DRAFT, kv, k_total=cfg.k_total + k), dev)
        self.graph = None

    def _verify(self, ctx):
        binding.spec_verify_attn(self.kv, self.case.q_verify, ctx, self.max_ctx, self.cfg.stat_window,
                                 out=self.out_v, stats=self.stats, workspace=self.ws_v, want_lse=False)

    def _select(self):
        c = self.cfg
        binding.spec_select_recall(self.stats, self.committed, c.k_sink, c.k_recent, c.k_total,
                                   indices=self.indices, n_indices=self.n_idx)

    def prime(self):
        """The index of the first round, from a verification pass over the last rows before the
        committed length (what a prefill leaves behind), and the first round's lengths."""
        self._verify(self.committed)
        self._select()
        binding.spec_advance_lengths(self.committed, None, self.k, self.ctx_verify, self.cur_len,
                                     max_len=self.max_ctx, workspace=self.ws_v)

    def round(self):
        for j in range(self.k):
            # step 0 follows the kernels that wrote the index sets and the lengths; the later steps do not
            binding.spec_sparse_draft_attn(self.kv, self.case.q_draft[j], self.indices, self.n_idx, self.committed,
                                           self.cur_len[j], self.k, out=self.out_d[j], workspace=self.ws_d,
                                           want_lse=False, early_gather=j > 0)
        self._verify(self.ctx_verify)
        binding.spec_accept_greedy(self.logits, self.draft_tokens, target=self.target,
                                   n_accepted=self.n_accepted, next_token=self.next_token)
        binding.spec_token_entropy(self.logits[0, :self.k], entropy=self.entropy)
        binding.spec_controller_update(self.state, self.entropy, self.n_accepted[:1], self.beta)
        binding.spec_controller_select(self.state, self.entropy, self.cand, self.c_d, self.c_v,
                                       k_star=self.k_star, p=self.p, score=self.score)
        binding.spec_advance_lengths(self.committed, self.n_accepted, self.k, self.ctx_verify, self.cur_len,
                                     max_len=self.max_ctx, workspace=self.ws_v)
        self._select()

    def capture(self):
        self.prime()
        saved = (self.committed.clone(), self.ctx_verify.clone(), self.cur_len.clone(), self.state.clone())
        self.round()  # warm-up outside the capture
        torch.cuda.synchronize()
        self.committed.copy_(saved[0])
        self.ctx_verify.copy_(saved[1])
        self.cur_len.copy_(saved[2])
        self.state.copy_(saved[3])
        self._verify(self.committed)  # the warm-up round replaced the statistic and the index: rebuild them
        self._select()
        torch.cuda.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            self.round()

    def replay(self):
        self.graph.replay()
