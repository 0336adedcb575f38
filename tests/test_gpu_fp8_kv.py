"""8-bit (e4m3) KV cache as a second workload of the path: verification (the score-cache kernel reading the
bytes at head_dim 128, the same kernel on a bf16 expansion of the cache at head_dim 64, the generic
kernels on the bytes), selection and the sparse draft kernel's fp8 instance against the oracle on the
same bytes and scales, within the 2e-3 bar of the bf16 path."""
import pytest
import torch

import oracle
from paper_2607_27735_b200 import binding, inputs

pytestmark = pytest.mark.gpu
TOL = 2e-3

SHAPES = [
    dict(ctx=(600, 600), k_total=128, head_dim=128),
    dict(ctx=(600, 600), k_total=128, head_dim=64),
    dict(ctx=(100, 100), k_total=128),  # budget >= context
    dict(ctx=(3000, 3000), k_total=1024, k_recent=64, n_q_heads=10, n_kv_heads=2, batch=2),
    dict(ctx=(300, 2000), k_total=256, k_recent=64, batch=3, page_size=16, shuffled_pages=True, planted=0,
         q_mode="iid", q_std=0.09, n_layers=2),
    dict(ctx=(4000, 4000), k_total=2048, k_recent=64, n_q_heads=32, n_kv_heads=8, planted=0.01),
    dict(ctx=(1500, 1500), k_total=512, k_recent=32, n_q_heads=16, n_kv_heads=2),
    dict(ctx=(2500, 2500), k_total=700, k_recent=16, n_q_heads=8, n_kv_heads=2, kv_dist="student_t3"),
]


@pytest.mark.parametrize("shape", SHAPES)
def test_fp8_cache_path_matches_the_oracle(shape):
    cfg = inputs.small_config(draft_steps=3, n_q=5, **shape)
    case = inputs.make_case(cfg, device="cuda")
    kv8 = inputs.quantize_kv_fp8(case.kv)
    kv8_cpu = kv8.cpu()
    ctx = case.ctx_len
    T = int(ctx.max())
    o_out = o_lse = o_stats = None
    for impl in (binding.VERIFY_GENERIC, binding.VERIFY_AUTO):
        binding.set_verify_impl(impl)
        try:
            out, lse, stats, ws = binding.spec_verify_attn(kv8, case.q_verify, ctx, T)
        finally:
            binding.set_verify_impl(binding.VERIFY_AUTO)
        assert binding.read_status(ws) == 0
        if impl == binding.VERIFY_GENERIC:
            assert binding.last_verify_impl() == binding.VERIFY_GENERIC
        else:  # every shape of this list fits the score-cache kernel
            assert binding.last_verify_impl() == (binding.VERIFY_TCGEN05_CACHED_EXPANDED if cfg.head_dim == 64
                                                  else binding.VERIFY_TCGEN05_CACHED)
        if o_out is None:
            o_out, o_lse, o_stats = oracle.verify_attn(kv8_cpu, case.q_verify.cpu(), ctx.cpu(), 16, stats.shape[-1])
        assert (out.cpu().double() - o_out).abs().max().item() <= TOL
        assert (lse.cpu().double() - o_lse).abs().max().item() <= TOL
        for b in range(cfg.batch):
            t = int(ctx[b])
            assert (stats[:, b, :, :t].cpu().double() - o_stats[:, b, :, :t]).abs().max().item() <= TOL
    idx, n = binding.spec_select_recall(stats, ctx, cfg.k_sink, cfg.k_recent, cfg.k_total)
    o_idx, o_n = oracle.select_recall(stats.cpu(), ctx.cpu(), cfg.k_sink, cfg.k_recent, cfg.k_total)
    assert torch.equal(idx.cpu(), o_idx) and torch.equal(n.cpu(), o_n)
    for step in range(cfg.draft_steps):
        cur = ctx + step + 1
        q = case.q_draft[step].contiguous()
        d_out, d_lse, wd = binding.spec_sparse_draft_attn(kv8, q, idx, n, ctx, cur, step + 1, early_gather=step > 0)
        assert binding.read_status(wd) == 0
        r_out, r_lse = oracle.sparse_draft_attn(kv8_cpu, q.cpu(), idx.cpu(), n.cpu(), ctx.cpu(), cur.cpu())
        assert (d_out.cpu().double() - r_out).abs().max().item() <= TOL, step
        fin = torch.isfinite(r_lse)
        assert ((d_lse.cpu().double() - r_lse)[fin]).abs().max().item() <= TOL


@pytest.mark.parametrize("head_dim", [128, 64])
def test_fp8_verify_with_scales_that_are_not_powers_of_two_and_a_short_workspace(head_dim):
    """The kernel applies the scales per (layer, KV head): the expanded copies (fp16 tiles in shared memory
    at head_dim 128, a bf16 copy in the workspace at head_dim 64) leave them out, because a scaled value
    need not be a 16-bit value.  At head_dim 64 a workspace without room for the copy falls back to the
    generic kernels; at head_dim 128 the plain workspace is enough."""
    import dataclasses
    cfg = inputs.small_config(ctx=(700, 1900), n_q=9, batch=2, n_layers=2, n_q_heads=8, n_kv_heads=2,
                              page_size=16, shuffled_pages=True, head_dim=head_dim)
    case = inputs.make_case(cfg, device="cuda")
    kv8 = inputs.quantize_kv_fp8(case.kv)
    g = torch.Generator(device="cuda").manual_seed(5)
    kv8 = dataclasses.replace(
        kv8, k_scale=kv8.k_scale * (0.7 + 0.6 * torch.rand(kv8.k_scale.shape, generator=g, device="cuda")),
        v_scale=kv8.v_scale * (0.7 + 0.6 * torch.rand(kv8.v_scale.shape, generator=g, device="cuda")))
    ctx = case.ctx_len
    o_out, o_lse, o_stats = oracle.verify_attn(kv8.cpu(), case.q_verify.cpu(), ctx.cpu(), 16, 1900)
    full = binding.workspace_bytes(binding.WS_VERIFY, kv8, cfg.n_q, 1900)
    base = binding.workspace_bytes(binding.WS_VERIFY, case.kv, cfg.n_q, 1900)
    assert full > base
    wants = ((full, binding.VERIFY_TCGEN05_CACHED), (base, binding.VERIFY_TCGEN05_CACHED)) if head_dim == 128 else \
            ((full, binding.VERIFY_TCGEN05_CACHED_EXPANDED), (base, binding.VERIFY_GENERIC))
    for nbytes, want in wants:
        ws = binding.alloc_workspace(nbytes, "cuda")
        out, lse, stats, _ = binding.spec_verify_attn(kv8, case.q_verify, ctx, 1900, workspace=ws)
        assert binding.read_status(ws) == 0
        assert binding.last_verify_impl() == want
        assert (out.cpu().double() - o_out).abs().max().item() <= TOL
        assert (lse.cpu().double() - o_lse).abs().max().item() <= TOL
        for b in range(cfg.batch):
            t = int(ctx[b])
            assert (stats[:, b, :, :t].cpu().double() - o_stats[:, b, :, :t]).abs().max().item() <= TOL


def test_fp8_draft_per_head_sets_and_bf16_output():
    cfg = inputs.small_config(ctx=(900, 900), k_total=160, k_recent=16, n_q_heads=8, n_kv_heads=2, draft_steps=1)
    case = inputs.make_case(cfg, device="cuda")
    kv8 = inputs.quantize_kv_fp8(case.kv)
    ctx = case.ctx_len
    _, _, stats, _ = binding.spec_verify_attn(kv8, case.q_verify, ctx, 900, per_head=True)
    idx, n = binding.spec_select_recall(stats, ctx, cfg.k_sink, cfg.k_recent, cfg.k_total)
    q = case.q_draft[0].contiguous()
    out, lse, ws = binding.spec_sparse_draft_attn(kv8, q, idx, n, ctx, ctx + 1, 1, per_head=True)
    assert binding.read_status(ws) == 0
    r_out, _ = oracle.sparse_draft_attn(kv8.cpu(), q.cpu(), idx.cpu(), n.cpu(), ctx.cpu(), (ctx + 1).cpu(), per_head=True)
    assert (out.cpu().double() - r_out).abs().max().item() <= TOL
    o16, _, _ = binding.spec_sparse_draft_attn(kv8, q, idx, n, ctx, ctx + 1, 1, per_head=True, out_bf16=True)
    assert torch.equal(o16, out.to(torch.bfloat16))


def test_fp8_cache_needs_16_byte_rows():
    cfg = inputs.small_config(ctx=(100, 100))
    case = inputs.make_case(cfg, device="cuda")
    kv8 = inputs.quantize_kv_fp8(case.kv)
    import dataclasses
    bad = dataclasses.replace(kv8, slot_stride=kv8.slot_stride + 8)
    with pytest.raises(binding.SpecError) as e:
        binding.spec_verify_attn(bad, case.q_verify, case.ctx_len, 100)
    assert e.value.code == -1


def test_fp8_verify_flags_accumulate_and_bf16_output():
    """The call's flags over an 8-bit cache: a second call with ACCUMULATE doubles the statistic, and the bf16
    output is the fp32 output rounded to nearest even."""
    cfg = inputs.small_config(ctx=(1200, 1200), n_q=9, n_q_heads=8, n_kv_heads=2, planted=4)
    case = inputs.make_case(cfg, device="cuda")
    kv8 = inputs.quantize_kv_fp8(case.kv)
    out, lse, stats, ws = binding.spec_verify_attn(kv8, case.q_verify, case.ctx_len, 1200)
    assert binding.last_verify_impl() == binding.VERIFY_TCGEN05_CACHED
    once = stats.clone()
    binding.spec_verify_attn(kv8, case.q_verify, case.ctx_len, 1200, stats=stats, workspace=ws, accumulate=True)
    assert binding.read_status(ws) == 0
    assert torch.equal(stats, once + once)
    o16, _, _, _ = binding.spec_verify_attn(kv8, case.q_verify, case.ctx_len, 1200, out_bf16=True)
    assert torch.equal(o16, out.to(torch.bfloat16))
