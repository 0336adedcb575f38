"""Max instead of sum over the query heads of a group (SPEC_VERIFY_STATS_GROUP_MAX): the score-cache
kernel and the generic kernels against the oracle's group_max form, the fused histogram and the
selection on top of it, and accumulation across passes."""
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
    (dict(ctx=(500, 500), n_q=2, n_q_heads=20, n_kv_heads=2), binding.VERIFY_GENERIC),            # groups of 10
    (dict(ctx=(600, 600), n_q=4, n_q_heads=8, n_kv_heads=2, head_dim=64), binding.VERIFY_TCGEN05_CACHED),
])
def test_group_max_matches_oracle(shape, expect_impl):
    cfg = inputs.small_config(k_total=160, k_recent=16, **shape)
    case = inputs.make_case(cfg, device="cuda")
    kv, ctx = case.kv, case.ctx_len
    T = int(ctx.max())
    hist = torch.zeros(kv.n_layers, kv.batch, kv.n_kv_heads, 2048, dtype=torch.int32, device="cuda")
    out, lse, stats, ws = binding.spec_verify_attn(kv, case.q_verify, ctx, T, group_max=True, score_hist=hist)
    assert binding.read_status(ws) == 0
    assert binding.last_verify_impl() == expect_impl
    o_out, o_lse, o_stats = oracle.verify_attn(kv.cpu(), case.q_verify.cpu(), ctx.cpu(), 16, T, group_max=True)
    assert (out.cpu().double() - o_out).abs().max().item() <= TOL
    assert (lse.cpu().double() - o_lse).abs().max().item() <= TOL
    for b in range(cfg.batch):
        t = int(ctx[b])
        assert (stats[:, b, :, :t].cpu().double() - o_stats[:, b, :, :t]).abs().max().item() <= TOL
    # it is the maximum of the per-head scores the same kernels write
    _, _, per_head, _ = binding.spec_verify_attn(kv, case.q_verify, ctx, T, per_head=True)
    G = cfg.n_q_heads // cfg.n_kv_heads
    folded = per_head.view(per_head.shape[0], cfg.batch, cfg.n_kv_heads, G, -1).max(dim=3).values
    for b in range(cfg.batch):
        t = int(ctx[b])
        assert torch.equal(folded[:, b, :, :t], stats[:, b, :, :t])
    # selection on top of it, fed with the fused counts: bit-exact against the oracle on the same scores
    idx, n = binding.spec_select_recall(stats, ctx, cfg.k_sink, cfg.k_recent, cfg.k_total, score_hist=hist, hist_len=ctx)
    o_idx, o_n = oracle.select_recall(stats.cpu(), ctx.cpu(), cfg.k_sink, cfg.k_recent, cfg.k_total)
    assert torch.equal(idx.cpu(), o_idx) and torch.equal(n.cpu(), o_n)
    assert int(hist.abs().sum()) == 0
    # accumulation: a second pass adds its own max-folded score to the running sums
    _, _, twice, _ = binding.spec_verify_attn(kv, case.q_verify, ctx, T, group_max=True, accumulate=True,
                                              stats=stats.clone())
    for b in range(cfg.batch):
        t = int(ctx[b])
        assert (twice[:, b, :, :t] - 2 * stats[:, b, :, :t]).abs().max().item() <= 1e-5


def test_group_max_and_per_head_exclude_each_other():
    cfg = inputs.small_config(ctx=(300, 300), n_q=3)
    case = inputs.make_case(cfg, device="cuda")
    with pytest.raises(binding.SpecError) as e:
        binding.spec_verify_attn(case.kv, case.q_verify, case.ctx_len, 300, per_head=True, group_max=True,
                                 stats=torch.zeros(1, 1, cfg.n_q_heads, 320, device="cuda"))
    assert e.value.code == -1
