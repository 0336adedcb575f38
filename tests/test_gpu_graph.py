"""The three calls inside one captured CUDA graph, replayed with lengths that change in device
memory between replays (nothing about a launch may depend on the lengths seen at capture time:
only on the host-side bounds max_ctx_len, k_total and max_tail)."""
import pytest
import torch

import oracle
from paper_2607_27735_b200 import binding, inputs

pytestmark = pytest.mark.gpu
TOL = 2e-3


@pytest.mark.parametrize("shape", [
    dict(ctx=(1500, 1500), batch=2, n_q=5, n_q_heads=8, n_kv_heads=2, k_total=256, k_recent=32),
    dict(ctx=(2000, 2000), batch=3, n_q=7, n_q_heads=8, n_kv_heads=2, k_total=192, k_recent=16,
         page_size=16, shuffled_pages=True, n_layers=2),
])
def test_graph_replay_with_changing_lengths(shape):
    cfg = inputs.small_config(draft_steps=2, **shape)
    case = inputs.make_case(cfg, device="cuda")
    kv = case.kv
    L, B, max_ctx = kv.n_layers, cfg.batch, int(case.ctx_len.max())
    dev = kv.k.device
    ctx = case.ctx_len.clone()
    cur = (case.ctx_len + 1).clone()
    out = torch.empty(L, B, cfg.n_q, cfg.n_q_heads, cfg.head_dim, device=dev)
    lse = torch.empty(L, B, cfg.n_q, cfg.n_q_heads, device=dev)
    stats = torch.zeros(L, B, cfg.n_kv_heads, max_ctx, device=dev)
    idx = torch.empty(L, B, cfg.n_kv_heads, cfg.k_total, dtype=torch.int32, device=dev)
    n_idx = torch.empty(L, B, cfg.n_kv_heads, dtype=torch.int32, device=dev)
    d_out = torch.empty(L, B, cfg.n_q_heads, cfg.head_dim, device=dev)
    d_lse = torch.empty(L, B, cfg.n_q_heads, device=dev)
    ws_v = binding.alloc_workspace(binding.workspace_bytes(binding.WS_VERIFY, kv, cfg.n_q, max_ctx), dev)
    ws_d = binding.alloc_workspace(binding.workspace_bytes(binding.WS_DRAFT, kv, k_total=cfg.k_total + 2), dev)
    q_d = case.q_draft[0].contiguous()

    def step():
        binding.spec_verify_attn(kv, case.q_verify, ctx, max_ctx, out=out, lse=lse, stats=stats, workspace=ws_v)
        binding.spec_select_recall(stats, ctx, cfg.k_sink, cfg.k_recent, cfg.k_total, indices=idx, n_indices=n_idx)
        binding.spec_sparse_draft_attn(kv, q_d, idx, n_idx, ctx, cur, 2, out=d_out, lse=d_lse, workspace=ws_d)

    step()  # warm-up outside the capture (first-call set-up of the library)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()

    gen = torch.Generator().manual_seed(5)
    for trial in range(3):
        new_ctx = torch.randint(cfg.n_q + 40, max_ctx + 1, (B,), generator=gen, dtype=torch.int32)
        if trial == 2:
            new_ctx[0] = cfg.k_total - 3  # a sequence shorter than the budget: every position is kept
        ctx.copy_(new_ctx)
        cur.copy_(new_ctx + 1 + (trial % 2))
        graph.replay()
        torch.cuda.synchronize()
        assert binding.read_status(ws_v) == 0 and binding.read_status(ws_d) == 0
        o_out, o_lse, o_stats = oracle.verify_attn(kv.cpu(), case.q_verify.cpu(), ctx.cpu(), 16, max_ctx)
        assert (out.cpu().double() - o_out).abs().max().item() <= TOL
        assert (lse.cpu().double() - o_lse).abs().max().item() <= TOL
        for b in range(B):
            T = int(new_ctx[b])
            assert (stats[:, b, :, :T].cpu().double() - o_stats[:, b, :, :T]).abs().max().item() <= TOL
        r_idx, r_n = oracle.select_recall(stats.cpu(), ctx.cpu(), cfg.k_sink, cfg.k_recent, cfg.k_total)
        assert torch.equal(n_idx.cpu(), r_n)
        for l in range(L):
            for b in range(B):
                for h in range(cfg.n_kv_heads):
                    n = int(r_n[l, b, h])
                    assert torch.equal(idx[l, b, h, :n].cpu(), r_idx[l, b, h, :n])
        r_out, r_lse = oracle.sparse_draft_attn(kv.cpu(), q_d.cpu(), idx.cpu(), n_idx.cpu(), ctx.cpu(), cur.cpu())
        assert (d_out.cpu().double() - r_out).abs().max().item() <= TOL
        assert (d_lse.cpu().double() - r_lse).abs().max().item() <= TOL


def test_runner_step_with_host_buffers_matches_the_resident_step():
    """runner.replay_host_io overlaps the host copies with the phases on a second stream; the
    bytes that come back must be those of the plain replay, step after step."""
    import dataclasses

    from paper_2607_27735_b200 import runner
    cfg = dataclasses.replace(inputs.baseline_configs()["cfg2_8b_32k"], n_layers=2, ctx=(4096, 4096))
    case = inputs.make_case(cfg, device="cuda")
    run = runner.SpecStepRunner(case)
    run.capture()
    run.replay()
    torch.cuda.synchronize()
    ref_v, ref_d = run.out_v.cpu(), run.out_d.cpu()
    qv, qd = case.q_verify.cpu().pin_memory(), case.q_draft.cpu().pin_memory()
    ov = torch.empty(run.out_v.shape).pin_memory()
    od = torch.empty(run.out_d.shape).pin_memory()
    run.q_verify.zero_()
    run.q_draft.zero_()
    for _ in range(3):
        ov.zero_()
        od.zero_()
        run.replay_host_io(qv, qd, ov, od)
        torch.cuda.synchronize()
        assert torch.equal(ov, ref_v) and torch.equal(od, ref_d)
