"""bf16 attention outputs (flags SPEC_VERIFY_OUT_BF16 / SPEC_DRAFT_OUT_BF16): the fp32 result rounded
to nearest even at the store, in every kernel that writes an attention output."""
import pytest
import torch

import oracle
from paper_2607_27735_b200 import binding, inputs

pytestmark = pytest.mark.gpu
TOL = 2e-3


@pytest.mark.parametrize("impl,shape", [
    (binding.VERIFY_AUTO, dict(ctx=(3000, 3000), n_q=5, n_q_heads=8, n_kv_heads=2)),
    (binding.VERIFY_AUTO, dict(ctx=(700, 2600), batch=3, n_q=9, n_q_heads=8, n_kv_heads=2, page_size=16,
                               shuffled_pages=True, n_layers=2)),
    (binding.VERIFY_TCGEN05_TWOSWEEP, dict(ctx=(2100, 2100), n_q=7, n_q_heads=8, n_kv_heads=2)),
    (binding.VERIFY_GENERIC, dict(ctx=(900, 900), n_q=4, n_q_heads=8, n_kv_heads=2, head_dim=64)),
    (binding.VERIFY_AUTO, dict(ctx=(40100, 40100), n_q=32, n_q_heads=4, n_kv_heads=1, planted=0.001)),  # rows in two passes
])
def test_bf16_outputs_are_the_rounded_fp32_outputs(impl, shape):
    cfg = inputs.small_config(k_total=160, k_recent=16, **shape)
    case = inputs.make_case(cfg, device="cuda")
    kv, ctx = case.kv, case.ctx_len
    max_ctx = int(ctx.max())
    prev = binding.set_verify_impl(impl)
    try:
        ref, _, stats, _ = binding.spec_verify_attn(kv, case.q_verify, ctx, max_ctx)
        got, _, stats_b, ws = binding.spec_verify_attn(kv, case.q_verify, ctx, max_ctx, out_bf16=True)
        assert binding.read_status(ws) == 0
    finally:
        binding.set_verify_impl(prev)
    assert got.dtype == torch.bfloat16
    assert torch.equal(got, ref.to(torch.bfloat16))          # same arithmetic, rounded once at the store
    assert torch.equal(stats, stats_b)
    o_out, _, _ = oracle.verify_attn(kv.cpu(), case.q_verify.cpu(), ctx.cpu(), 16, max_ctx)
    err = (got.cpu().double() - o_out).abs()
    assert (err <= TOL + 2.0 ** -8 * o_out.abs()).all()      # the bar plus half a bf16 step
    # draft
    idx, n = binding.spec_select_recall(stats, ctx, cfg.k_sink, cfg.k_recent, cfg.k_total)
    cur = ctx + 1
    q = case.q_draft[0].contiguous()
    d_ref, _, _ = binding.spec_sparse_draft_attn(kv, q, idx, n, ctx, cur, 1)
    d_got, _, wd = binding.spec_sparse_draft_attn(kv, q, idx, n, ctx, cur, 1, out_bf16=True)
    assert binding.read_status(wd) == 0
    assert torch.equal(d_got, d_ref.to(torch.bfloat16))
    r_out, _ = oracle.sparse_draft_attn(kv.cpu(), q.cpu(), idx.cpu(), n.cpu(), ctx.cpu(), cur.cpu())
    assert ((d_got.cpu().double() - r_out).abs() <= TOL + 2.0 ** -8 * r_out.abs()).all()
