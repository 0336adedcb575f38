"""spec_verify_attn_ex with SPEC_VERIFY_ACCUMULATE_STATS: the statistic of a pass is added to the
running sums, in every verification kernel (score-cache, rows in two passes, two-sweep, generic)."""
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
def test_accumulated_statistic_matches_oracle(impl, shape):
    cfg = inputs.small_config(**shape)
    case = inputs.make_case(cfg, device="cuda")
    kv, ctx = case.kv, case.ctx_len
    max_ctx = int(ctx.max())
    gen = torch.Generator().manual_seed(3)
    before = torch.rand(kv.n_layers, cfg.batch, cfg.n_kv_heads, max_ctx, generator=gen)  # running sums so far
    stats = before.cuda()
    prev = binding.set_verify_impl(impl)
    try:
        out, lse, stats, ws = binding.spec_verify_attn(kv, case.q_verify, ctx, max_ctx, stats=stats, accumulate=True)
        assert binding.read_status(ws) == 0
    finally:
        binding.set_verify_impl(prev)
    o_out, o_lse, o_stats = oracle.verify_attn(kv.cpu(), case.q_verify.cpu(), ctx.cpu(), 16, max_ctx)
    assert (out.cpu().double() - o_out).abs().max().item() <= TOL
    for b in range(cfg.batch):
        T = int(ctx[b])
        want = before[:, b, :, :T].double() + o_stats[:, b, :, :T]
        assert (stats[:, b, :, :T].cpu().double() - want).abs().max().item() <= TOL
        assert torch.equal(stats[:, b, :, T:].cpu(), before[:, b, :, T:])  # beyond the context: untouched


def test_two_passes_equal_one_pass():
    """Rows a then b in two calls (the second accumulating) against one call with a + b rows."""
    a, b = 4, 5
    cfg = inputs.small_config(ctx=(5000, 5000), n_q=a + b, n_q_heads=8, n_kv_heads=2, planted=5, seed=8)
    case = inputs.make_case(cfg, device="cuda")
    kv, ctx = case.kv, case.ctx_len
    T = int(ctx.max())
    _, _, one, _ = binding.spec_verify_attn(kv, case.q_verify, ctx, T)
    qa = case.q_verify[:, :, :a].contiguous()
    qb = case.q_verify[:, :, a:].contiguous()
    _, _, two, _ = binding.spec_verify_attn(kv, qa, ctx - b, T)
    two[..., T - b:] = 0            # positions appended since the first pass hold 0
    binding.spec_verify_attn(kv, qb, ctx, T, stats=two, accumulate=True)
    assert (one - two)[..., :T].abs().max().item() <= 2e-5


def test_unknown_flag_is_refused():
    cfg = inputs.small_config()
    case = inputs.make_case(cfg, device="cuda")
    lib = binding.load()
    import ctypes
    kvs = binding._kv_struct(case.kv)
    rc = lib.spec_verify_attn_ex(ctypes.byref(kvs), case.q_verify.data_ptr(), cfg.n_q, case.ctx_len.data_ptr(), 600, 16,
                                 None, None, None, 600, None, 0, 2, None)
    assert rc == -1
