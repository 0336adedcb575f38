"""The per-attention-head form (Eq. 3 and Eq. 5 as printed): one score and one index set per query
head.  Verification (score-cache kernel and generic kernels), selection and drafting against the
oracle's per-head functions, which the CPU pins tie to the per-KV-head form."""
import pytest
import torch

import oracle
from paper_2607_27735_b200 import binding, inputs

pytestmark = pytest.mark.gpu
TOL = 2e-3


@pytest.mark.parametrize("shape,expect_impl", [
    (dict(ctx=(3000, 3000), n_q=5, n_q_heads=8, n_kv_heads=2), binding.VERIFY_TCGEN05_CACHED),
    (dict(ctx=(900, 2100), batch=3, n_q=9, n_q_heads=16, n_kv_heads=2, page_size=16, shuffled_pages=True,
          n_layers=2), binding.VERIFY_TCGEN05_CACHED),                       # groups of 8, ragged, paged
    (dict(ctx=(1500, 1500), n_q=17, n_q_heads=4, n_kv_heads=2), binding.VERIFY_TCGEN05_CACHED),  # window drops row 0
    (dict(ctx=(700, 700), n_q=3, n_q_heads=4, n_kv_heads=4), binding.VERIFY_TCGEN05_CACHED),     # groups of 1
    (dict(ctx=(800, 800), n_q=4, n_q_heads=10, n_kv_heads=2), binding.VERIFY_TCGEN05_CACHED),    # groups of 5
    (dict(ctx=(2300, 2300), n_q=7, n_q_heads=6, n_kv_heads=2, n_layers=2), binding.VERIFY_TCGEN05_CACHED),  # groups of 3, window offset
    (dict(ctx=(500, 500), n_q=2, n_q_heads=20, n_kv_heads=2), binding.VERIFY_GENERIC),            # groups of 10
    (dict(ctx=(600, 600), n_q=4, n_q_heads=8, n_kv_heads=2, head_dim=64), binding.VERIFY_TCGEN05_CACHED),
])
def test_per_head_path_matches_oracle(shape, expect_impl):
    cfg = inputs.small_config(k_total=160, k_recent=16, draft_steps=2, **shape)
    case = inputs.make_case(cfg, device="cuda")
    kv, ctx = case.kv, case.ctx_len
    max_ctx = int(ctx.max())
    out, lse, stats, ws = binding.spec_verify_attn(kv, case.q_verify, ctx, max_ctx, per_head=True)
    assert binding.read_status(ws) == 0
    assert binding.last_verify_impl() == expect_impl
    o_out, o_lse, o_stats = oracle.verify_attn(kv.cpu(), case.q_verify.cpu(), ctx.cpu(), 16, max_ctx, per_head=True)
    assert (out.cpu().double() - o_out).abs().max().item() <= TOL
    assert (lse.cpu().double() - o_lse).abs().max().item() <= TOL
    for b in range(cfg.batch):
        T = int(ctx[b])
        assert (stats[:, b, :, :T].cpu().double() - o_stats[:, b, :, :T]).abs().max().item() <= TOL
    # the group's statistic is the sum of its heads' statistics
    _, _, grouped, _ = binding.spec_verify_attn(kv, case.q_verify, ctx, max_ctx)
    G = cfg.n_q_heads // cfg.n_kv_heads
    folded = stats.view(stats.shape[0], cfg.batch, cfg.n_kv_heads, G, -1).sum(dim=3)
    for b in range(cfg.batch):
        T = int(ctx[b])
        assert (folded[:, b, :, :T] - grouped[:, b, :, :T]).abs().max().item() <= 1e-4
    # selection per attention head: the same kernel with n_q_heads problems, bit-exact
    idx, n = binding.spec_select_recall(stats, ctx, cfg.k_sink, cfg.k_recent, cfg.k_total)
    o_idx, o_n = oracle.select_recall(stats.cpu(), ctx.cpu(), cfg.k_sink, cfg.k_recent, cfg.k_total)
    assert torch.equal(idx.cpu(), o_idx) and torch.equal(n.cpu(), o_n)
    # drafting: every head over its own set
    for step in range(cfg.draft_steps):
        cur = ctx + step + 1
        q = case.q_draft[step].contiguous()
        d_out, d_lse, wd = binding.spec_sparse_draft_attn(kv, q, idx, n, ctx, cur, step + 1, per_head=True)
        assert binding.read_status(wd) == 0
        r_out, r_lse = oracle.sparse_draft_attn(kv.cpu(), q.cpu(), idx.cpu(), n.cpu(), ctx.cpu(), cur.cpu(),
                                                per_head=True)
        assert (d_out.cpu().double() - r_out).abs().max().item() <= TOL
        assert (d_lse.cpu().double() - r_lse).abs().max().item() <= TOL


def test_per_head_accumulates_too():
    cfg = inputs.small_config(ctx=(2000, 2000), n_q=5, n_q_heads=8, n_kv_heads=2)
    case = inputs.make_case(cfg, device="cuda")
    T = int(case.ctx_len.max())
    before = torch.rand(1, 1, 8, T, generator=torch.Generator().manual_seed(1))
    stats = before.cuda()
    binding.spec_verify_attn(case.kv, case.q_verify, case.ctx_len, T, stats=stats, accumulate=True, per_head=True)
    _, _, o_stats = oracle.verify_attn(case.kv.cpu(), case.q_verify.cpu(), case.ctx_len.cpu(), 16, T, per_head=True)
    assert (stats.cpu().double() - (before.double() + o_stats)).abs().max().item() <= TOL


def test_per_head_draft_at_the_8b_shape():
    # 32 attention heads over 8 KV heads, budget 2048 + tail: the gather is four times the default's
    import dataclasses
    cfg = dataclasses.replace(inputs.baseline_configs()["cfg2_8b_32k"], n_layers=1, ctx=(8192, 8192))
    case = inputs.make_case(cfg, device="cuda")
    kv, ctx = case.kv, case.ctx_len
    T = int(ctx.max())
    _, _, stats, _ = binding.spec_verify_attn(kv, case.q_verify, ctx, T, per_head=True)
    idx, n = binding.spec_select_recall(stats, ctx, cfg.k_sink, cfg.k_recent, cfg.k_total)
    cur = ctx + 3
    q = case.q_draft[2].contiguous()
    d_out, d_lse, wd = binding.spec_sparse_draft_attn(kv, q, idx, n, ctx, cur, 3, per_head=True)
    assert binding.read_status(wd) == 0
    r_out, r_lse = oracle.sparse_draft_attn(kv.cpu(), q.cpu(), idx.cpu(), n.cpu(), ctx.cpu(), cur.cpu(), per_head=True)
    assert (d_out.cpu().double() - r_out).abs().max().item() <= TOL
    assert (d_lse.cpu().double() - r_lse).abs().max().item() <= TOL


@pytest.mark.parametrize("seed", range(16))
def test_per_head_random_shapes(seed):
    """The randomised shapes of test_gpu_fuzz.py through the per-head calls (score-cache kernel where
    the shape allows it, generic kernels otherwise)."""
    from test_gpu_fuzz import draw_shape
    shape = draw_shape(1000 + seed)
    if shape["planted"] == 0:
        shape.update(q_mode="iid", q_std=0.3)
    cfg = inputs.small_config(name=f"ph{seed}", **shape)
    case = inputs.make_case(cfg, device="cuda")
    kv, ctx = case.kv, case.ctx_len
    out, lse, stats, ws = binding.spec_verify_attn(kv, case.q_verify, ctx, int(ctx.max()), per_head=True)
    assert binding.read_status(ws) == 0, shape
    o_out, _, o_stats = oracle.verify_attn(kv.cpu(), case.q_verify.cpu(), ctx.cpu(), 16, stats.shape[-1], per_head=True)
    assert (out.cpu().double() - o_out).abs().max().item() <= TOL, shape
    for b in range(cfg.batch):
        T = int(ctx[b])
        assert (stats[:, b, :, :T].cpu().double() - o_stats[:, b, :, :T]).abs().max().item() <= TOL, shape
    idx, n = binding.spec_select_recall(stats, ctx, cfg.k_sink, cfg.k_recent, cfg.k_total)
    o_idx, o_n = oracle.select_recall(stats.cpu(), ctx.cpu(), cfg.k_sink, cfg.k_recent, cfg.k_total)
    assert torch.equal(idx.cpu(), o_idx) and torch.equal(n.cpu(), o_n), shape
    cur = ctx + 1
    q = case.q_draft[0].contiguous()
    d_out, d_lse, wd = binding.spec_sparse_draft_attn(kv, q, idx, n, ctx, cur, 1, per_head=True)
    assert binding.read_status(wd) == 0, shape
    r_out, r_lse = oracle.sparse_draft_attn(kv.cpu(), q.cpu(), idx.cpu(), n.cpu(), ctx.cpu(), cur.cpu(), per_head=True)
    assert (d_out.cpu().double() - r_out).abs().max().item() <= TOL, shape
    fin = torch.isfinite(r_lse)
    assert ((d_lse.cpu().double() - r_lse)[fin]).abs().max().item() <= TOL, shape
