"""Selection's first radix pass fused into the verification call (Eq. 4 on top of Eq. 3): the
counts must be the histogram of the top 11 bits of the scores the GPU wrote, the selection fed
with them must give the same indices bit for bit as the plain selection (and as the oracle on the
same score array), and the pair must leave the count array zero."""
import pytest
import torch

import oracle
from paper_2607_27735_b200 import binding, inputs

pytestmark = pytest.mark.gpu

SHAPES = [
    (binding.VERIFY_AUTO, dict(ctx=(5000, 5000), n_q=9, n_q_heads=32, n_kv_heads=8, planted=50)),
    (binding.VERIFY_AUTO, dict(ctx=(300, 2100), n_q=7, batch=3, page_size=16, shuffled_pages=True, planted=0,
                               q_mode="iid", q_std=0.09, n_q_heads=8, n_kv_heads=2, n_layers=2)),
    (binding.VERIFY_TCGEN05_TWOSWEEP, dict(ctx=(1500, 1500), n_q=5, n_q_heads=8, n_kv_heads=2, planted=8)),
    (binding.VERIFY_GENERIC, dict(ctx=(700, 700), n_q=5, head_dim=64, planted=4)),
]


def bins_of(stats, ctx_len):
    L, B, H, S = stats.shape
    ref = torch.zeros(L, B, H, 2048, dtype=torch.int64)
    bits = (stats.cpu().contiguous().view(torch.int32).to(torch.int64) & 0xFFFFFFFF) >> 21
    for b in range(B):
        t = int(ctx_len[b])
        for l in range(L):
            for h in range(H):
                ref[l, b, h] = torch.bincount(bits[l, b, h, :t], minlength=2048)
    return ref


@pytest.mark.parametrize("impl,shape", SHAPES)
@pytest.mark.parametrize("per_head", [False, True])
def test_fused_histogram_and_selection(impl, shape, per_head):
    if per_head and impl == binding.VERIFY_TCGEN05_TWOSWEEP:
        pytest.skip("the two-sweep kernel keeps no per-head statistic")
    cfg = inputs.small_config(k_total=256, k_recent=64, **shape)
    case = inputs.make_case(cfg, device="cuda")
    kv = case.kv
    T = int(case.ctx_len.max())
    heads = kv.n_q_heads if per_head else kv.n_kv_heads
    hist = torch.zeros(kv.n_layers, kv.batch, heads, 2048, dtype=torch.int32, device="cuda")
    prev = binding.set_verify_impl(impl)
    try:
        for rnd in range(2):  # the second round finds the array cleared by the first round's selection
            _, _, stats, ws = binding.spec_verify_attn(kv, case.q_verify, case.ctx_len, T, per_head=per_head,
                                                       score_hist=hist)
            assert binding.read_status(ws) == 0
            assert torch.equal(hist.cpu().to(torch.int64), bins_of(stats, case.ctx_len))
            # the committed length may be shorter than the verified one (rejected drafts)
            sel = (case.ctx_len - (3 if rnd else 0)).clamp(min=1).int()
            plain = binding.spec_select_recall(stats, sel, cfg.k_sink, cfg.k_recent, cfg.k_total)
            fused = binding.spec_select_recall(stats, sel, cfg.k_sink, cfg.k_recent, cfg.k_total, score_hist=hist,
                                               hist_len=case.ctx_len)
            assert torch.equal(plain[0], fused[0]) and torch.equal(plain[1], fused[1])
            o_idx, o_n = oracle.select_recall(stats.cpu(), sel.cpu(), cfg.k_sink, cfg.k_recent, cfg.k_total)
            assert torch.equal(fused[0].cpu(), o_idx) and torch.equal(fused[1].cpu(), o_n)
            assert int(hist.abs().sum()) == 0
    finally:
        binding.set_verify_impl(prev)


def test_counts_that_do_not_cover_the_span_fall_back_to_the_sweep():
    g = torch.Generator(device="cuda").manual_seed(5)
    stats = torch.rand(1, 2, 2, 3000, generator=g, device="cuda") ** 6
    sel = torch.tensor([3000, 2500], dtype=torch.int32, device="cuda")
    short = torch.tensor([2000, 2500], dtype=torch.int32, device="cuda")  # sequence 0: counts end before the span does
    hist = torch.randint(0, 5, (1, 2, 2, 2048), dtype=torch.int32, device="cuda")  # garbage for sequence 0
    bits = (stats[0, 1].cpu().contiguous().view(torch.int32).to(torch.int64) & 0xFFFFFFFF) >> 21
    for h in range(2):
        hist[0, 1, h] = torch.bincount(bits[h, :2500], minlength=2048).int().cuda()
    fused = binding.spec_select_recall(stats, sel, 4, 64, 512, score_hist=hist, hist_len=short)
    o_idx, o_n = oracle.select_recall(stats.cpu(), sel.cpu(), 4, 64, 512)
    assert torch.equal(fused[0].cpu(), o_idx) and torch.equal(fused[1].cpu(), o_n)
    assert int(hist.abs().sum()) == 0


@pytest.mark.parametrize("head_dim", [128, 64])
def test_fused_histogram_over_an_8bit_cache(head_dim):
    """The same pair over an e4m3 cache: the score-cache kernel's 8-bit instances count in their statistic
    pass (head_dim 128: tiles expanded in shared memory; head_dim 64: the bf16 expansion in the workspace)."""
    cfg = inputs.small_config(ctx=(900, 2600), n_q=9, batch=2, n_layers=2, n_q_heads=8, n_kv_heads=2, page_size=16,
                              shuffled_pages=True, planted=6, k_total=256, k_recent=64, head_dim=head_dim)
    case = inputs.make_case(cfg, device="cuda")
    kv8 = inputs.quantize_kv_fp8(case.kv)
    T = int(case.ctx_len.max())
    hist = torch.zeros(kv8.n_layers, kv8.batch, kv8.n_kv_heads, 2048, dtype=torch.int32, device="cuda")
    for rnd in range(2):
        _, _, stats, ws = binding.spec_verify_attn(kv8, case.q_verify, case.ctx_len, T, score_hist=hist)
        assert binding.read_status(ws) == 0
        assert binding.last_verify_impl() == (binding.VERIFY_TCGEN05_CACHED if head_dim == 128
                                              else binding.VERIFY_TCGEN05_CACHED_EXPANDED)
        assert torch.equal(hist.cpu().to(torch.int64), bins_of(stats, case.ctx_len))
        plain = binding.spec_select_recall(stats, case.ctx_len, cfg.k_sink, cfg.k_recent, cfg.k_total)
        fused = binding.spec_select_recall(stats, case.ctx_len, cfg.k_sink, cfg.k_recent, cfg.k_total,
                                           score_hist=hist, hist_len=case.ctx_len)
        assert torch.equal(plain[0], fused[0]) and torch.equal(plain[1], fused[1])
        assert int(hist.abs().sum()) == 0
