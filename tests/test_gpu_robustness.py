"""Device-side guards: lengths and page-table entries outside their bounds are clamped or skipped
and reported in the status word (nothing leaves the buffers, outputs stay finite), a bounded wait
that cannot complete gives up with SPEC_ERR_TIMEOUT and leaves the context usable, and the
early-gather launch mode of the draft call gives the same bits as the plain one."""
import dataclasses
import time

import pytest
import torch

import oracle
from paper_2607_27735_b200 import binding, inputs

pytestmark = pytest.mark.gpu
TOL = 2e-3
BAD_INDEX, TIMEOUT = -6, -5


@pytest.mark.parametrize("impl,head_dim", [(binding.VERIFY_AUTO, 128), (binding.VERIFY_TCGEN05_TWOSWEEP, 128),
                                           (binding.VERIFY_GENERIC, 128), (binding.VERIFY_AUTO, 64)])
def test_verify_clamps_a_context_length_beyond_the_host_bound(impl, head_dim):
    cfg = inputs.small_config(ctx=(900, 900), n_q=5, batch=2, head_dim=head_dim, planted=4)
    case = inputs.make_case(cfg, device="cuda")
    T = 900
    pad = 256
    stride = 1024
    guard = torch.full((2 * 2 * stride + 2 * pad,), -3.0, device="cuda")
    stats = guard[pad:-pad].view(1, 2, 2, stride)
    too_long = case.ctx_len.clone()
    too_long[1] = T + 1
    too_short = case.ctx_len.clone()
    too_short[0] = 2  # fewer tokens than rows
    prev = binding.set_verify_impl(impl)
    try:
        ref = binding.spec_verify_attn(case.kv, case.q_verify, case.ctx_len, T, stat_stride=stride)
        assert binding.read_status(ref[3]) == 0
        for lens in (too_long, too_short):
            out, lse, st, ws = binding.spec_verify_attn(case.kv, case.q_verify, lens, T, stats=stats)
            assert binding.read_status(ws) == BAD_INDEX
            assert binding.read_status(ws) == 0  # reading acknowledges it
            assert torch.isfinite(out).all()
            assert (guard[:pad] == -3.0).all() and (guard[-pad:] == -3.0).all()
        # the clamped sequence was verified at the bound: same result as the in-range call
        out, _, _, ws = binding.spec_verify_attn(case.kv, case.q_verify, too_long, T, stat_stride=stride)
        assert torch.equal(out[0, 1], ref[0][0, 1])
    finally:
        binding.set_verify_impl(prev)


def test_draft_clamps_lengths_and_skips_bad_page_entries():
    cfg = inputs.small_config(ctx=(400, 400), k_total=64, batch=2, page_size=16, shuffled_pages=True,
                              draft_steps=2, planted=0, q_mode="iid")
    case = inputs.make_case(cfg, device="cuda")
    kv = case.kv
    cap = kv.max_pages * kv.page_size
    idx = torch.arange(64, dtype=torch.int32, device="cuda").repeat(1, 2, 2, 1).contiguous()
    n = torch.full((1, 2, 2), 64, dtype=torch.int32, device="cuda")
    q = case.q_draft[0].contiguous()
    tail = case.ctx_len.clone()
    ref, _, ws = binding.spec_sparse_draft_attn(kv, q, idx, n, tail, tail + 1, 1)
    assert binding.read_status(ws) == 0
    # a current length beyond the cache: clamped (the tail then holds the rows up to the capacity)
    beyond = torch.tensor([cap + 50, 401], dtype=torch.int32, device="cuda")
    start = torch.tensor([cap - 2, 400], dtype=torch.int32, device="cuda")
    out, _, ws = binding.spec_sparse_draft_attn(kv, q, idx, n, start, beyond, 4)
    assert binding.read_status(ws) == BAD_INDEX and torch.isfinite(out).all()
    assert torch.equal(out[0, 1], ref[0, 1])  # the other sequence is untouched by it
    # a tail longer than the launch was sized for: truncated and reported
    out, _, ws = binding.spec_sparse_draft_attn(kv, q, idx, n, tail - 8, tail + 1, 2)
    assert binding.read_status(ws) == BAD_INDEX and torch.isfinite(out).all()
    # a page-table entry outside the pool: the rows behind it are skipped
    bad = dataclasses.replace(kv, page_table=kv.page_table.clone())
    bad.page_table[0, 1] = kv.n_pages if kv.n_pages else kv.batch * kv.max_pages
    out, _, ws = binding.spec_sparse_draft_attn(bad, q, idx, n, tail, tail + 1, 1)
    assert binding.read_status(ws) == BAD_INDEX and torch.isfinite(out).all()
    assert torch.equal(out[0, 1], ref[0, 1])
    o_idx = idx.clone().cpu()
    keep = torch.tensor([p for p in range(64) if p // 16 != 1], dtype=torch.int32)
    o_idx[0, 0, :, :48] = keep
    o_idx[0, 0, :, 48:] = -1
    o_n = n.clone().cpu()
    o_n[0, 0] = 48
    o_out, _ = oracle.sparse_draft_attn(kv.cpu(), q.cpu(), o_idx, o_n, tail.cpu(), (tail + 1).cpu())
    assert (out.cpu().double() - o_out).abs().max().item() <= TOL


def test_generic_verify_reports_a_bad_page_entry():
    cfg = inputs.small_config(ctx=(300, 300), n_q=3, page_size=16, shuffled_pages=True, head_dim=64, planted=0)
    case = inputs.make_case(cfg, device="cuda")
    bad = dataclasses.replace(case.kv, page_table=case.kv.page_table.clone())
    bad.page_table[0, 2] = -7
    prev = binding.set_verify_impl(binding.VERIFY_GENERIC)
    try:
        out, _, _, ws = binding.spec_verify_attn(bad, case.q_verify, case.ctx_len, 300)
        assert binding.read_status(ws) == BAD_INDEX and torch.isfinite(out).all()
    finally:
        binding.set_verify_impl(prev)


@pytest.mark.parametrize("head_dim", [128, 64])
def test_verify_over_an_8bit_cache_reports_bad_lengths_and_page_entries(head_dim):
    """Both ways of reading an 8-bit cache (tiles expanded in shared memory at head_dim 128, pages expanded
    into the workspace at head_dim 64) follow the same rules: a page-table entry outside the pool is
    replaced and reported, a length beyond the host bound is clamped, and nothing is written outside the
    workspace."""
    cfg = inputs.small_config(ctx=(500, 700), n_q=5, batch=2, page_size=16, shuffled_pages=True, planted=0,
                              head_dim=head_dim)
    case = inputs.make_case(cfg, device="cuda")
    kv8 = inputs.quantize_kv_fp8(case.kv)
    T = int(case.ctx_len.max())
    longest = int(case.ctx_len.argmax())
    need = binding.workspace_bytes(binding.WS_VERIFY, kv8, cfg.n_q, T)
    pad = 4096
    guard = torch.zeros(need + 2 * pad, dtype=torch.uint8, device="cuda")
    guard[:pad] = 0x5a
    guard[-pad:] = 0x5a
    ws = guard[pad:-pad]
    assert ws.data_ptr() % 256 == 0
    ref = binding.spec_verify_attn(kv8, case.q_verify, case.ctx_len, T, workspace=ws)
    assert binding.read_status(ws) == 0
    assert binding.last_verify_impl() == (binding.VERIFY_TCGEN05_CACHED if head_dim == 128
                                          else binding.VERIFY_TCGEN05_CACHED_EXPANDED)
    bad = dataclasses.replace(kv8, page_table=kv8.page_table.clone())
    bad.page_table[longest, 3] = kv8.page_table.numel() + 5
    out, _, _, _ = binding.spec_verify_attn(bad, case.q_verify, case.ctx_len, T, workspace=ws)
    assert binding.read_status(ws) == BAD_INDEX and torch.isfinite(out).all()
    assert torch.equal(out[0, 1 - longest], ref[0][0, 1 - longest])  # the other sequence is unaffected
    too_long = case.ctx_len.clone()
    too_long[longest] = T + 1
    out, _, _, _ = binding.spec_verify_attn(kv8, case.q_verify, too_long, T, workspace=ws)
    assert binding.read_status(ws) == BAD_INDEX and torch.isfinite(out).all()
    assert (guard[:pad] == 0x5a).all() and (guard[-pad:] == 0x5a).all()


def test_advance_lengths_holds_a_sequence_at_the_capacity():
    committed = torch.tensor([100, 990, 500], dtype=torch.int32, device="cuda")
    m = torch.tensor([3, 4, 0], dtype=torch.int32, device="cuda")
    k = 4
    ctx = torch.empty(3, dtype=torch.int32, device="cuda")
    cur = torch.empty(k, 3, dtype=torch.int32, device="cuda")
    ws = binding.alloc_workspace(256, "cuda")
    binding.spec_advance_lengths(committed, m, k, ctx, cur, max_len=1000, workspace=ws)
    assert committed.tolist() == [104, 995, 501]  # 990 + 5 = 995: 995 + 5 = 1000 still fits
    assert binding.read_status(ws) == 0
    binding.spec_advance_lengths(committed, m, k, ctx, cur, max_len=1000, workspace=ws)
    assert committed.tolist() == [108, 995, 502]  # 1000 + 5 would not fit: held at 1000 - 5
    assert ctx.tolist() == [113, 1000, 507]
    assert cur[:, 1].tolist() == [996, 997, 998, 999]
    assert binding.read_status(ws) == BAD_INDEX


def test_a_wait_that_cannot_complete_times_out_and_the_context_stays_usable():
    """The cross-CTA counters of the verification workspace are pre-set so that "every CTA of the head
    has published" can never become true; with a short limit the kernel gives up, records
    SPEC_ERR_TIMEOUT and returns.  A following call on a re-zeroed workspace matches the oracle."""
    cfg = inputs.small_config(ctx=(3000, 3000), n_q=5, n_q_heads=8, n_kv_heads=2, planted=8)
    case = inputs.make_case(cfg, device="cuda")
    T = 3000
    ws = binding.alloc_workspace(binding.workspace_bytes(binding.WS_VERIFY, case.kv, cfg.n_q, T), "cuda")
    ws.view(torch.int32)[64:64 + 16] = -(1 << 20)  # the counters follow the 256-byte status block
    old = binding.set_wait_limit_cycles(4_000_000)  # about 2 ms of SM clocks
    prev = binding.set_verify_impl(binding.VERIFY_TCGEN05_CACHED)
    try:
        t0 = time.perf_counter()
        binding.spec_verify_attn(case.kv, case.q_verify, case.ctx_len, T, workspace=ws)
        status = binding.read_status(ws)
        elapsed = time.perf_counter() - t0
        assert status == TIMEOUT
        assert elapsed < 2.0
    finally:
        binding.set_wait_limit_cycles(old)
        binding.set_verify_impl(prev)
    ws.zero_()
    out, lse, stats, _ = binding.spec_verify_attn(case.kv, case.q_verify, case.ctx_len, T, workspace=ws)
    assert binding.read_status(ws) == 0
    o_out, _, o_stats = oracle.verify_attn(case.kv.cpu(), case.q_verify.cpu(), case.ctx_len.cpu(), 16, stats.shape[-1])
    assert (out.cpu().double() - o_out).abs().max().item() <= TOL
    assert (stats.cpu().double() - o_stats).abs().max().item() <= TOL


def test_early_gather_gives_the_same_bits():
    cfg = inputs.small_config(ctx=(2500, 2500), k_total=1024, k_recent=64, n_q_heads=32, n_kv_heads=8,
                              draft_steps=3, planted=20)
    case = inputs.make_case(cfg, device="cuda")
    _, _, stats, _ = binding.spec_verify_attn(case.kv, case.q_verify, case.ctx_len, 2500)
    idx, n = binding.spec_select_recall(stats, case.ctx_len, cfg.k_sink, cfg.k_recent, cfg.k_total)
    torch.cuda.synchronize()
    outs = {}
    for early in (False, True):
        res = []
        for j in range(cfg.draft_steps):
            out, lse, ws = binding.spec_sparse_draft_attn(case.kv, case.q_draft[j].contiguous(), idx, n, case.ctx_len,
                                                          case.ctx_len + j + 1, cfg.draft_steps,
                                                          early_gather=early and j > 0)
            res.append((out, lse))
            assert binding.read_status(ws) == 0
        outs[early] = res
    for (a, la), (b, lb) in zip(outs[False], outs[True]):
        assert torch.equal(a, b) and torch.equal(la, lb)
