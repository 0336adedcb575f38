"""Parity at the full sizes of the five baseline workloads, through the same runner and launch
configuration bench.py times (one launch per layer for verify/draft, one select launch).

The oracle cannot redo a whole 32K..128K-context step in test time, so each workload is
checked on SAMPLED (layer, sequence, KV head) problems: the sampled head's K/V rows are copied
out into a one-head cache and the oracle recomputes that problem completely (every query row,
the whole score vector, the index set, the draft outputs).  The context lengths, batch, page
layout, budget and speculation length are the workload's own; only the layer count of the larger
workloads is cut (layers are independent and identically shaped), as stated per case."""
import dataclasses

import pytest
import torch

import oracle
from paper_2607_27735_b200 import binding, inputs, runner

pytestmark = pytest.mark.gpu
TOL = 2e-3


def one_head_cache(kv, layer, b, h, T):
    """CPU copy of one (layer, sequence, KV head) as a contiguous one-head cache."""
    pos = torch.arange(T, device=kv.k.device)
    page = pos // kv.page_size
    slot = pos % kv.page_size
    phys = (b * kv.max_pages + page) if kv.page_table is None else kv.page_table[b][page].long()
    k = kv.k[layer, phys, h, slot].cpu().contiguous().view(1, 1, 1, T, kv.head_dim)
    v = kv.v[layer, phys, h, slot].cpu().contiguous().view(1, 1, 1, T, kv.head_dim)
    D = kv.head_dim
    G = kv.n_q_heads // kv.n_kv_heads
    ks = vs = None
    if kv.fp8:  # e4m3 bytes: the head's scales go with them
        ks = kv.k_scale[layer:layer + 1, h:h + 1].cpu().contiguous()
        vs = kv.v_scale[layer:layer + 1, h:h + 1].cpu().contiguous()
    return inputs.KVCache(k=k, v=v, layer_stride=T * D, page_stride=T * D, head_stride=T * D,
                          slot_stride=D, n_layers=1, page_size=T, page_table=None, max_pages=1,
                          batch=1, n_q_heads=G, n_kv_heads=1, head_dim=D, sm_scale=0.0, n_pages=1,
                          fp8=kv.fp8, k_scale=ks, v_scale=vs)


def check_samples(case, run, samples):
    cfg, kv = case.cfg, case.kv
    G = cfg.group
    torch.cuda.synchronize()
    worst = dict(out=0.0, stats=0.0, draft=0.0, overlap=1.0)
    for (layer, b, h) in samples:
        T = int(case.ctx_len[b])
        cap = T + cfg.draft_steps
        sub = one_head_cache(kv, layer, b, h, cap)
        q = case.q_verify[layer, b, :, h * G:(h + 1) * G].cpu().contiguous().view(1, 1, cfg.n_q, G, -1)
        tlen = torch.tensor([T], dtype=torch.int32)
        o_out, o_lse, o_stats = oracle.verify_attn(sub, q, tlen, cfg.stat_window, T)
        g_out = run.out_v[layer, b, :, h * G:(h + 1) * G].cpu().double()
        g_stats = run.stats[layer, b, h, :T].cpu()
        worst["out"] = max(worst["out"], (g_out - o_out[0, 0]).abs().max().item())
        worst["stats"] = max(worst["stats"], (g_stats.double() - o_stats[0, 0, 0]).abs().max().item())
        # recall indices: bit-exact on the identical (GPU) score array
        o_idx, o_n = oracle.select_recall(g_stats.view(1, 1, 1, T).contiguous(), tlen, cfg.k_sink,
                                          cfg.k_recent, cfg.k_total)
        assert torch.equal(run.indices[layer, b, h].cpu(), o_idx[0, 0, 0])
        assert int(run.n_idx[layer, b, h]) == int(o_n[0, 0, 0])
        # end to end (oracle scores -> oracle select), reported as overlap
        e_idx, _ = oracle.select_recall(o_stats.float(), tlen, cfg.k_sink, cfg.k_recent, cfg.k_total)
        a, bb = set(o_idx[0, 0, 0].tolist()), set(e_idx[0, 0, 0].tolist())
        worst["overlap"] = min(worst["overlap"], len(a & bb) / max(1, len(a)))
        for j in range(cfg.draft_steps):
            qd = case.q_draft[j, layer, b, h * G:(h + 1) * G].cpu().contiguous().view(1, 1, G, -1)
            d_out, _ = oracle.sparse_draft_attn(sub, qd, o_idx, o_n, tlen,
                                                torch.tensor([T + j + 1], dtype=torch.int32))
            g_d = run.out_d[j, layer, b, h * G:(h + 1) * G].cpu().double()
            worst["draft"] = max(worst["draft"], (g_d - d_out[0, 0]).abs().max().item())
    assert worst["out"] <= TOL, worst
    assert worst["stats"] <= TOL, worst
    assert worst["draft"] <= TOL, worst
    return worst


def run_config(cfg, samples, fold=False):
    case = inputs.make_case(cfg, device="cuda")
    run = runner.SpecStepRunner(case, fold_layers=fold)
    run.step()
    assert binding.read_status(run.ws_v) == 0 and binding.read_status(run.ws_d) == 0
    return case, run, check_samples(case, run, samples)


def test_cfg1_tiny_every_head():
    cfg = inputs.baseline_configs()["cfg1_tiny"]
    _, _, worst = run_config(cfg, [(0, 0, 0), (0, 0, 1)])
    assert binding.last_verify_impl() == binding.VERIFY_TCGEN05_CACHED  # head_dim 64 on the tcgen05 path
    assert worst["overlap"] > 0.97


def test_cfg2_8bit_cache_full_context_sampled_heads():
    """The headline shape over an e4m3 copy of the cache (4 of its 32 layers; scales that are not powers of
    two): the score-cache kernel reads the bytes itself, two units of four heads per layer as over bf16."""
    cfg = dataclasses.replace(inputs.baseline_configs()["cfg2_8b_32k"], n_layers=4)
    case = inputs.make_case(cfg, device="cuda")
    kv8 = inputs.quantize_kv_fp8(case.kv)
    g = torch.Generator(device="cuda").manual_seed(11)
    kv8 = dataclasses.replace(
        kv8, k_scale=kv8.k_scale * (0.8 + 0.4 * torch.rand(kv8.k_scale.shape, generator=g, device="cuda")),
        v_scale=kv8.v_scale * (0.8 + 0.4 * torch.rand(kv8.v_scale.shape, generator=g, device="cuda")))
    case8 = dataclasses.replace(case, kv=kv8)
    run = runner.SpecStepRunner(case8)
    run.step()
    assert binding.read_status(run.ws_v) == 0 and binding.read_status(run.ws_d) == 0
    assert binding.last_verify_impl() == binding.VERIFY_TCGEN05_CACHED
    worst = check_samples(case8, run, [(0, 0, 0), (2, 0, 3), (3, 0, 7)])
    assert worst["overlap"] > 0.9
    mass = run.stats[:, 0, :, :32768].sum(-1)
    assert (mass - cfg.group * cfg.n_q).abs().max().item() < 0.05


def test_cfg2_8b_32k_full_step_sampled_heads():
    """All 32 layers, the launch configuration of the headline bench line."""
    cfg = inputs.baseline_configs()["cfg2_8b_32k"]
    case, run, worst = run_config(cfg, [(0, 0, 0), (17, 0, 5), (31, 0, 7)])
    assert binding.last_verify_impl() == binding.VERIFY_TCGEN05_CACHED
    assert worst["overlap"] > 0.9
    # the mass of the score: every contributing row adds 1
    mass = run.stats[:, 0, :, :32768].sum(-1)
    assert (mass - cfg.group * cfg.n_q).abs().max().item() < 0.05
    # planted heavy hitters outside sink/recent are recalled
    hits = 0
    for (l, h) in [(0, 0), (17, 5), (31, 7)]:
        chosen = set(run.indices[l, 0, h].tolist())
        pl = case.planted_pos[l, 0, h].tolist()
        hits += sum(p in chosen for p in pl) / len(pl)
    assert hits / 3 > 0.9


@pytest.mark.parametrize("k", [1, 2, 8, 16])
def test_cfg3_128k_speculation_length_sweep(k):
    """131072-token context, 4 of the 32 layers, the workload's sweep of speculation lengths (k = 4
    runs in the drift test below); k = 16 gives 68 rows per KV head and a window longer than W."""
    cfg = dataclasses.replace(inputs.baseline_configs(k)["cfg3_8b_128k"], n_layers=4)
    run_config(cfg, [(0, 0, 1), (3, 0, 6)])


def test_cfg4_ragged_paged_batch():
    """Batch 8, contexts drawn from 8192..65536, 16-token shuffled pages, 4 of the 32 layers."""
    cfg = dataclasses.replace(inputs.baseline_configs()["cfg4_ragged_paged"], n_layers=4)
    case = inputs.make_case(cfg, device="cuda")
    ctx = case.ctx_len.tolist()
    b_short, b_long = ctx.index(min(ctx)), ctx.index(max(ctx))
    run = runner.SpecStepRunner(case)
    run.step()
    assert binding.read_status(run.ws_v) == 0 and binding.read_status(run.ws_d) == 0
    check_samples(case, run, [(0, b_short, 0), (3, b_long, 7), (2, 3, 4)])


def test_cfg5_32b_shape_student_t_values():
    """Group of 5 query heads per KV head, batch 4, 65536 context, heavy-tailed K/V, 8 sink + 256
    recent; 4 of the 64 layers."""
    cfg = dataclasses.replace(inputs.baseline_configs()["cfg5_32b_64k"], n_layers=4)
    run_config(cfg, [(0, 0, 0), (3, 3, 7)])


def test_128k_index_follows_resampled_heavy_hitters():
    """Third workload, full context and budget, 2 of its 32 layers: between speculation rounds
    each planted position moves with probability 0.1.  The index rebuilt from each round's GPU
    statistic must hold (nearly) all CURRENT planted positions, the ones that just moved in
    included, and the draft output over that index must match the oracle on a sampled head."""
    cfg = dataclasses.replace(inputs.baseline_configs(4)["cfg3_8b_128k"], n_layers=2)
    case = inputs.make_case(cfg, device="cuda")
    run = runner.SpecStepRunner(case)
    G = cfg.group
    for step in range(3):
        before = case.planted_pos.clone()
        moved = inputs.resample_planted(case, 0.1, step)
        assert moved > 0
        run.step()
        torch.cuda.synchronize()
        assert binding.read_status(run.ws_v) == 0 and binding.read_status(run.ws_d) == 0
        hit_all, n_all, hit_new, n_new = 0, 0, 0, 0
        for layer in range(cfg.n_layers):
            for h in range(cfg.n_kv_heads):
                chosen = set(run.indices[layer, 0, h, :int(run.n_idx[layer, 0, h])].tolist())
                cur = set(case.planted_pos[layer, 0, h].tolist())
                new = cur - set(before[layer, 0, h].tolist())
                hit_all += len(cur & chosen)
                n_all += len(cur)
                hit_new += len(new & chosen)
                n_new += len(new)
        assert n_new > 0
        # 3 x the direction plus unit noise: a planted key sits about 5 sigma above the background
        assert hit_all / n_all > 0.97, (step, hit_all, n_all)
        assert hit_new / n_new > 0.95, (step, hit_new, n_new)
    # the last round's draft outputs on one sampled head, against the oracle over the GPU's index
    layer, b, h = 1, 0, 5
    T = int(case.ctx_len[b])
    sub = one_head_cache(case.kv, layer, b, h, T + cfg.draft_steps)
    idx = run.indices[layer, b, h].cpu().view(1, 1, 1, -1).contiguous()
    n = run.n_idx[layer, b, h].cpu().view(1, 1, 1).contiguous()
    for j in range(cfg.draft_steps):
        q = case.q_draft[j, layer, b, h * G:(h + 1) * G].cpu().contiguous().view(1, 1, G, -1)
        o_out, _ = oracle.sparse_draft_attn(sub, q, idx, n, torch.tensor([T], dtype=torch.int32),
                                            torch.tensor([T + j + 1], dtype=torch.int32))
        g_out = run.out_d[j, layer, b, h * G:(h + 1) * G].cpu().double()
        assert (g_out - o_out[0, 0]).abs().max().item() < TOL
