"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded bf16 inputs.  Bars: attention outputs, statistic and LSE within 2e-3 max-abs per tensor
(bf16 inputs, fp32 accumulation); recall indices bit-exact on identical score arrays."""
import dataclasses

import pytest
import torch

import oracle
from paper_2607_27735_b200 import binding, inputs

pytestmark = pytest.mark.gpu
TOL = 2e-3


def run_verify(case, stat_window=16, impl=binding.VERIFY_AUTO):
    kv = case.kv
    prev = binding.set_verify_impl(impl)
    try:
        out, lse, stats, ws = binding.spec_verify_attn(
            kv, case.q_verify, case.ctx_len, int(case.ctx_len.max()), stat_window)
        status = binding.read_status(ws)
        assert status == 0, (status, ws[:16].view(torch.int32).tolist())
    finally:
        binding.set_verify_impl(prev)
    return out, lse, stats


def oracle_verify(case, stat_window=16, stat_stride=None):
    return oracle.verify_attn(case.kv.cpu(), case.q_verify.cpu(), case.ctx_len.cpu(), stat_window,
                              stat_stride)


def check_verify(case, stat_window=16, impl=binding.VERIFY_AUTO):
    out, lse, stats = run_verify(case, stat_window, impl)
    o_out, o_lse, o_stats = oracle_verify(case, stat_window, stats.shape[-1])
    assert torch.isfinite(out).all() and torch.isfinite(stats).all()
    e_out = (out.cpu().double() - o_out).abs().max().item()
    e_lse = (lse.cpu().double() - o_lse).abs().max().item()
    ctx = case.ctx_len.cpu()
    e_st = 0.0
    for b in range(case.kv.batch):
        T = int(ctx[b])
        e_st = max(e_st, (stats[:, b, :, :T].cpu().double() - o_stats[:, b, :, :T]).abs().max().item())
    assert e_out <= TOL, f"out max-abs {e_out}"
    assert e_st <= TOL, f"stats max-abs {e_st}"
    assert e_lse <= TOL, f"lse max-abs {e_lse}"
    return out, lse, stats


VERIFY_SHAPES = [
    dict(ctx=(1, 1), n_q=1, planted=0),
    dict(ctx=(5, 5), n_q=5, planted=0),
    dict(ctx=(17, 17), n_q=2, planted=1, head_dim=64),
    dict(ctx=(63, 63), n_q=9, planted=2),
    dict(ctx=(64, 64), n_q=16, planted=2, head_dim=64),
    dict(ctx=(65, 65), n_q=17, planted=2),
    dict(ctx=(257, 257), n_q=5, n_q_heads=5, n_kv_heads=1),
    dict(ctx=(2048, 2048), n_q=5, head_dim=64, planted=8, planted_mult=4.0, planted_noise=False),
    dict(ctx=(1500, 1500), n_q=9, n_q_heads=10, n_kv_heads=2, batch=2, n_layers=2),
    dict(ctx=(200, 1100), n_q=7, batch=3, page_size=16, shuffled_pages=True, planted=0,
         q_mode="iid", q_std=0.09, n_q_heads=8, n_kv_heads=2),
    dict(ctx=(900, 900), n_q=3, n_q_heads=8, n_kv_heads=8, page_size=128, shuffled_pages=True),
    dict(ctx=(777, 777), n_q=32, n_q_heads=8, n_kv_heads=2, kv_dist="student_t3"),
]


@pytest.mark.parametrize("impl", [binding.VERIFY_GENERIC, binding.VERIFY_AUTO])
@pytest.mark.parametrize("shape", VERIFY_SHAPES)
def test_verify_parity(shape, impl):
    cfg = inputs.small_config(**shape)
    case = inputs.make_case(cfg, device="cuda")
    check_verify(case, impl=impl)
    if impl == binding.VERIFY_AUTO and cfg.head_dim == 128 and cfg.n_q * cfg.group <= 96:
        # the fast path really ran
        assert binding.last_verify_impl() in (binding.VERIFY_TCGEN05_TWOSWEEP, binding.VERIFY_TCGEN05_CACHED)


TCGEN05_SHAPES = [
    dict(ctx=(128, 128), n_q=1, planted=0),
    dict(ctx=(129, 129), n_q=2, planted=0),
    dict(ctx=(5000, 5000), n_q=9, n_q_heads=32, n_kv_heads=8, planted=50),          # 8B shape
    dict(ctx=(20000, 20000), n_q=9, n_q_heads=32, n_kv_heads=8, planted=200),       # several tiles per CTA
    dict(ctx=(9000, 9000), n_q=7, n_q_heads=40, n_kv_heads=8, batch=2, kv_dist="student_t3"),
    dict(ctx=(3000, 9000), n_q=7, n_q_heads=32, n_kv_heads=8, batch=4, page_size=16,
         shuffled_pages=True, planted=0, q_mode="iid", q_std=0.09, n_layers=2),
    dict(ctx=(4100, 4100), n_q=17, n_q_heads=32, n_kv_heads=8, planted=40),         # R=68 > W rows
    dict(ctx=(2500, 2500), n_q=24, n_q_heads=16, n_kv_heads=4, planted=10),         # R=96
    dict(ctx=(6000, 6000), n_q=5, n_q_heads=8, n_kv_heads=1, page_size=256, shuffled_pages=True),
    # every width of the score tile (16 ... 128 columns): the lane reduction of the row partials takes a
    # different sequence of halving and in-place steps for 8, 16, 24, 32, 40 and 56 columns per thread
    dict(ctx=(1900, 1900), n_q=2, n_q_heads=8, n_kv_heads=2),                        # R=8   -> 16 columns
    dict(ctx=(1900, 1900), n_q=7, n_q_heads=8, n_kv_heads=2),                        # R=28  -> 32
    dict(ctx=(1900, 1900), n_q=15, n_q_heads=8, n_kv_heads=2),                       # R=60  -> 64
    dict(ctx=(1900, 1900), n_q=19, n_q_heads=8, n_kv_heads=2),                       # R=76  -> 80
    dict(ctx=(1900, 1900), n_q=26, n_q_heads=8, n_kv_heads=2, batch=2),              # R=104 -> 112
    dict(ctx=(1900, 1900), n_q=31, n_q_heads=8, n_kv_heads=2),                       # R=124 -> 128
]


@pytest.mark.parametrize("impl", [binding.VERIFY_TCGEN05_TWOSWEEP, binding.VERIFY_TCGEN05_CACHED])
@pytest.mark.parametrize("shape", TCGEN05_SHAPES)
def test_verify_tcgen05_parity(shape, impl):
    cfg = inputs.small_config(**shape)
    if impl == binding.VERIFY_TCGEN05_TWOSWEEP and cfg.n_q * cfg.group > 96:
        pytest.skip("the two-sweep kernel takes up to 96 rows per KV head")
    case = inputs.make_case(cfg, device="cuda")
    check_verify(case, impl=impl)
    assert binding.last_verify_impl() == impl


def test_verify_tcgen05_ignores_garbage_beyond_the_context():
    """Cache slots past ctx_len may hold anything (NaN included): they must not leak."""
    cfg = inputs.small_config(ctx=(1000, 1000), n_q=5, planted=5)
    case = inputs.make_case(cfg, device="cuda")
    kv = case.kv
    kv.k[:, :, :, 1000:] = float("nan")
    kv.v[:, :, :, 1000:] = float("nan")
    check_verify(case, impl=binding.VERIFY_TCGEN05_TWOSWEEP)
    check_verify(case, impl=binding.VERIFY_TCGEN05_CACHED)


@pytest.mark.parametrize("window", [1, 4, 16])
def test_verify_stat_window(window):
    cfg = inputs.small_config(ctx=(400, 400), n_q=9)
    case = inputs.make_case(cfg, device="cuda")
    _, _, stats = check_verify(case, stat_window=window)
    mass = stats[0, 0, :, :400].sum(-1)
    assert (mass - cfg.group * min(window, 9)).abs().max() < 1e-2


@pytest.mark.parametrize("shape,window", [
    (dict(ctx=(40000, 40000), n_q=32, n_q_heads=4, n_kv_heads=1, planted=0.001), 16),  # 128 rows x 313 tiles: over the cache
    (dict(ctx=(77000, 77000), n_q=17, n_q_heads=4, n_kv_heads=1, planted=0.001), 16),  # 9 + 8 rows, window drops row 0
    (dict(ctx=(77000, 77000), n_q=17, n_q_heads=4, n_kv_heads=1, planted=0.001), 4),   # window inside the second pass only
    (dict(ctx=(40100, 40100), n_q=31, n_q_heads=4, n_kv_heads=1, page_size=64, shuffled_pages=True, planted=0.001), 20),
])
def test_verify_rows_in_two_passes(shape, window):
    """One (layer, sequence) whose rows do not fit the score cache: AUTO verifies the two halves of
    the rows separately with the score-cache kernel and adds their statistics."""
    cfg = inputs.small_config(**shape)
    case = inputs.make_case(cfg, device="cuda")
    _, _, stats = check_verify(case, stat_window=window)
    assert binding.last_verify_impl() == binding.VERIFY_TCGEN05_CACHED_2PASS
    T = int(case.ctx_len[0])
    mass = stats[0, 0, :, :T].sum(-1)
    assert (mass - cfg.group * min(window, cfg.n_q)).abs().max() < 1e-2


def test_verify_is_deterministic_and_leaves_padding_untouched():
    cfg = inputs.small_config(ctx=(300, 1000), batch=2, n_q=5, planted=0, q_mode="iid")
    case = inputs.make_case(cfg, device="cuda")
    kv = case.kv
    T = int(case.ctx_len.max())
    stride = T + 64
    outs = []
    for _ in range(2):
        stats = torch.full((1, 2, 2, stride), -3.0, device="cuda")
        o, l, s, _ = binding.spec_verify_attn(kv, case.q_verify, case.ctx_len, T, stats=stats)
        outs.append((o.clone(), l.clone(), s.clone()))
    for a, b in zip(outs[0], outs[1]):
        assert torch.equal(a, b)
    s = outs[0][2]
    for b in range(2):
        assert (s[0, b, :, int(case.ctx_len[b]):] == -3.0).all()  # beyond ctx_len: not written


# ---------------------------------------------------------------------------------------------


def check_select(stats, sel_len, k_sink, k_recent, k_total):
    idx, n = binding.spec_select_recall(stats, sel_len, k_sink, k_recent, k_total)
    o_idx, o_n = oracle.select_recall(stats.cpu(), sel_len.cpu(), k_sink, k_recent, k_total)
    assert torch.equal(n.cpu(), o_n)
    assert torch.equal(idx.cpu(), o_idx)
    return idx, n


@pytest.mark.parametrize("T,k_sink,k_recent,k_total", [
    (64, 4, 8, 24), (20, 4, 8, 24), (24, 4, 8, 24), (25, 4, 8, 24), (300, 4, 64, 68),
    (2048, 4, 64, 256), (10000, 0, 0, 1), (9000, 8, 256, 2048), (40000, 4, 64, 2048),
    (33, 0, 0, 32), (5000, 4, 64, 4000),
])
def test_select_bit_exact_random_and_tied_scores(T, k_sink, k_recent, k_total):
    g = torch.Generator(device="cuda").manual_seed(T + k_total)
    L, B, H = 2, 2, 3
    sel_len = torch.tensor([T, max(1, T - 5)], dtype=torch.int32, device="cuda")
    smooth = torch.rand(L, B, H, T + 3, generator=g, device="cuda") ** 8  # probabilities-like
    check_select(smooth, sel_len, k_sink, k_recent, k_total)
    tied = torch.randint(0, 4, (L, B, H, T + 3), generator=g, device="cuda").float() * 0.125
    check_select(tied, sel_len, k_sink, k_recent, k_total)
    check_select(torch.zeros_like(tied), sel_len, k_sink, k_recent, k_total)
    tiny = smooth * 1e-38  # denormals order like their bit patterns too
    check_select(tiny, sel_len, k_sink, k_recent, k_total)


@pytest.mark.parametrize("T,n_tied", [
    (20000, 40), (20000, 1500), (20000, 3000), (20000, 9000), (131072 + 64, 40), (140000, 40), (140000, 3000),
])
def test_select_ties_at_the_threshold_and_long_contexts(T, n_tied):
    """The threshold's score repeated n_tied times (a handful: ranked by position in shared memory;
    thousands: the ordered compaction), and contexts on both sides of the position bitmap's reach."""
    g = torch.Generator(device="cuda").manual_seed(T + n_tied)
    L, B, H = 1, 2, 2
    k_sink, k_recent, k_total = 4, 64, 2048
    sel_len = torch.tensor([T, T - 7], dtype=torch.int32, device="cuda")
    stats = torch.rand(L, B, H, T, generator=g, device="cuda") ** 6
    kth = stats[..., k_sink:T - k_recent - 7].topk(k_total - k_sink - k_recent, dim=-1).values[..., -1:]
    where = torch.rand(L, B, H, T, generator=g, device="cuda").argsort(dim=-1)[..., :n_tied]
    stats.scatter_(-1, where, kth.expand(L, B, H, n_tied).contiguous())
    check_select(stats, sel_len, k_sink, k_recent, k_total)


def test_select_on_gpu_statistic_and_end_to_end_overlap():
    cfg = inputs.baseline_configs()["cfg1_tiny"]
    case = inputs.make_case(cfg, device="cuda")
    _, _, stats = check_verify(case)
    idx, n = check_select(stats, case.ctx_len, cfg.k_sink, cfg.k_recent, cfg.k_total)
    # end to end: oracle statistic -> oracle select, compared as sets (near-ties may differ)
    _, _, o_stats = oracle_verify(case)
    o_idx, _ = oracle.select_recall(o_stats.float(), case.ctx_len.cpu(), cfg.k_sink, cfg.k_recent,
                                    cfg.k_total)
    for h in range(cfg.n_kv_heads):
        a, b = set(idx[0, 0, h].tolist()), set(o_idx[0, 0, h].tolist())
        assert len(a & b) / cfg.k_total > 0.97
        assert all(int(p) in a for p in case.planted_pos[0, 0, h])


# ---------------------------------------------------------------------------------------------


def check_draft(case, idx, n_idx, tail_start, cur_len, step=0):
    kv = case.kv
    q = case.q_draft[step].contiguous()
    max_tail = int((cur_len - tail_start).clamp(min=0).max())
    out, lse, ws = binding.spec_sparse_draft_attn(kv, q, idx, n_idx, tail_start, cur_len, max_tail)
    assert binding.read_status(ws) == 0
    o_out, o_lse = oracle.sparse_draft_attn(kv.cpu(), q.cpu(), idx.cpu(), n_idx.cpu(),
                                            tail_start.cpu(), cur_len.cpu())
    e = (out.cpu().double() - o_out).abs().max().item()
    assert e <= TOL, f"draft out max-abs {e}"
    fin = torch.isfinite(o_lse)
    assert ((lse.cpu().double() - o_lse)[fin]).abs().max().item() <= TOL
    return out


DRAFT_SHAPES = [
    dict(ctx=(600, 600), k_total=128, head_dim=128),
    dict(ctx=(600, 600), k_total=128, head_dim=64),
    dict(ctx=(100, 100), k_total=128),  # budget >= context
    dict(ctx=(3000, 3000), k_total=1024, k_recent=64, n_q_heads=10, n_kv_heads=2, batch=2),
    dict(ctx=(300, 2000), k_total=256, k_recent=64, batch=3, page_size=16, shuffled_pages=True,
         planted=0, q_mode="iid", q_std=0.09, n_layers=2),
    dict(ctx=(700, 700), k_total=100, k_sink=0, k_recent=0, n_q_heads=8, n_kv_heads=8),
    # 8 problems x 2048 keys: the planner takes clusters of six (two calls resident together)
    dict(ctx=(4000, 4000), k_total=2048, k_recent=64, n_q_heads=32, n_kv_heads=8, planted=0.01),
    # 4104-key lists on 2 problems: shares of 528 keys run in rounds through two buffers
    dict(ctx=(6000, 6000), k_total=4096, k_recent=64, n_q_heads=8, n_kv_heads=2, planted=0.01),
    # group of 8 query heads: one MMA each for the hi and the lo part of P
    dict(ctx=(1500, 1500), k_total=512, k_recent=32, n_q_heads=16, n_kv_heads=2),
]


@pytest.mark.parametrize("shape", DRAFT_SHAPES)
def test_draft_parity_after_verify_and_select(shape):
    cfg = inputs.small_config(draft_steps=3, **shape)
    case = inputs.make_case(cfg, device="cuda")
    _, _, stats = run_verify(case)
    idx, n = binding.spec_select_recall(stats, case.ctx_len, cfg.k_sink, cfg.k_recent, cfg.k_total)
    for step in range(cfg.draft_steps):
        cur = case.ctx_len + step + 1
        check_draft(case, idx, n, case.ctx_len, cur, step)


def test_draft_with_full_budget_equals_dense_verification():
    cfg = inputs.small_config(ctx=(500, 500), n_q=1, k_total=512, draft_steps=1)
    case = inputs.make_case(cfg, device="cuda")
    out_v, lse_v, stats = run_verify(case)
    t1 = case.ctx_len - 1
    idx, n = binding.spec_select_recall(stats, t1.int(), cfg.k_sink, cfg.k_recent, cfg.k_total)
    q1 = case.q_verify[:, :, 0].contiguous()
    out_d, lse_d, _ = binding.spec_sparse_draft_attn(case.kv, q1, idx, n, t1.int(), case.ctx_len, 1)
    assert (out_d - out_v[:, :, 0]).abs().max().item() <= TOL
    assert (lse_d - lse_v[:, :, 0]).abs().max().item() <= TOL


def test_draft_empty_and_tail_only_key_sets():
    cfg = inputs.small_config(ctx=(200, 200), k_total=32, draft_steps=2, batch=2)
    case = inputs.make_case(cfg, device="cuda")
    idx = torch.full((1, 2, 2, 32), -1, dtype=torch.int32, device="cuda")
    n = torch.zeros(1, 2, 2, dtype=torch.int32, device="cuda")
    tail_start = torch.tensor([200, 200], dtype=torch.int32, device="cuda")
    cur = torch.tensor([202, 200], dtype=torch.int32, device="cuda")  # second: nothing to attend
    out = check_draft(case, idx, n, tail_start, cur)
    assert (out[0, 1] == 0).all()


def test_draft_flags_out_of_range_index_and_skips_it():
    cfg = inputs.small_config(ctx=(200, 200), k_total=16, draft_steps=1)
    case = inputs.make_case(cfg, device="cuda")
    good = torch.arange(16, dtype=torch.int32, device="cuda").repeat(1, 1, 2, 1)
    bad = good.clone()
    bad[0, 0, 1, 5] = 100000
    n = torch.full((1, 1, 2), 16, dtype=torch.int32, device="cuda")
    q = case.q_draft[0].contiguous()
    out, _, ws = binding.spec_sparse_draft_attn(case.kv, q, bad, n, case.ctx_len, case.ctx_len + 1, 1)
    assert binding.read_status(ws) == -6
    ref, _, ws2 = binding.spec_sparse_draft_attn(case.kv, q, good, n, case.ctx_len, case.ctx_len + 1, 1)
    assert binding.read_status(ws2) == 0
    assert torch.equal(out[0, 0, :4], ref[0, 0, :4])  # the other KV head is unaffected
    assert torch.isfinite(out).all()


# ---------------------------------------------------------------------------------------------


def test_host_side_argument_errors_launch_nothing():
    cfg = inputs.small_config(ctx=(100, 100))
    case = inputs.make_case(cfg, device="cuda")
    before = binding.launch_count()
    with pytest.raises(binding.SpecError) as e:
        binding.spec_verify_attn(case.kv, case.q_verify, case.ctx_len, 100,
                                 workspace=binding.alloc_workspace(256, "cuda"))
    assert e.value.code == -3
    bad = dataclasses.replace(case.kv, head_dim=96)
    with pytest.raises(binding.SpecError) as e:
        binding.spec_verify_attn(bad, case.q_verify, case.ctx_len, 100,
                                 workspace=binding.alloc_workspace(1 << 20, "cuda"))
    assert e.value.code == -2
    with pytest.raises(binding.SpecError) as e:
        binding.spec_select_recall(torch.zeros(1, 1, 2, 100, device="cuda"), case.ctx_len, 8, 8, 12)
    assert e.value.code == -1
    with pytest.raises(ValueError):
        binding.spec_select_recall(torch.zeros(1, 1, 2, 100), case.ctx_len, 4, 4, 12)
    assert binding.launch_count() == before


def test_outputs_do_not_overrun_their_buffers():
    cfg = inputs.small_config(ctx=(333, 333), n_q=5, k_total=64, draft_steps=1)
    case = inputs.make_case(cfg, device="cuda")
    L, B, n_q, Hq, D = case.q_verify.shape
    pad = 512
    big = torch.full((L * B * n_q * Hq * D + 2 * pad,), 7.5, device="cuda")
    out = big[pad:-pad].view(L, B, n_q, Hq, D)
    binding.spec_verify_attn(case.kv, case.q_verify, case.ctx_len, 333, out=out)
    torch.cuda.synchronize()
    assert (big[:pad] == 7.5).all() and (big[-pad:] == 7.5).all()
    ibig = torch.full((2 * 64 + 2 * pad,), -9, dtype=torch.int32, device="cuda")
    idx = ibig[pad:-pad].view(1, 1, 2, 64)
    stats = torch.rand(1, 1, 2, 400, device="cuda")
    binding.spec_select_recall(stats, case.ctx_len, 4, 16, 64, indices=idx)
    torch.cuda.synchronize()
    assert (ibig[:pad] == -9).all() and (ibig[-pad:] == -9).all()
