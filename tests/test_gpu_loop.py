"""Speculation rounds chained on the device (runner.SpecLoopRunner): one captured graph replayed
round after round, the committed length advancing by the accepted prefix + 1 in device memory.
Every round is checked against the oracle at the lengths a host-side simulation predicts."""
import random

import pytest
import torch

import oracle
from paper_2607_27735_b200 import binding, inputs, runner

pytestmark = pytest.mark.gpu
TOL = 2e-3


def test_rounds_follow_the_host_simulation():
    k, rounds, vocab = 4, 5, 2048
    cfg = inputs.small_config(ctx=(1200, 1200), batch=2, n_q=k + 1, n_q_heads=8, n_kv_heads=2, k_total=128,
                              k_recent=16, draft_steps=k, n_layers=2, planted=8, seed=77)
    case = inputs.make_case(cfg, device="cuda")
    kv = case.kv
    committed0 = torch.tensor([500, 640], dtype=torch.int32)
    loop = runner.SpecLoopRunner(case, committed0, vocab)
    loop.capture()
    rng = random.Random(5)
    sim = committed0.clone()
    kv_cpu, qv_cpu, qd_cpu = kv.cpu(), case.q_verify.cpu(), case.q_draft.cpu()
    state = torch.tensor([1.0, 4.0], dtype=torch.float64)
    for r in range(rounds):
        logits = inputs.make_logits(2 * (k + 1), vocab, seed=100 + r).view(2, k + 1, vocab).contiguous()
        greedy, _, _ = oracle.accept_greedy(logits, torch.zeros(2, k, dtype=torch.int32))
        draft = greedy[:, :k].clone()
        for b in range(2):
            cut = rng.randint(0, k)
            if cut < k:
                draft[b, cut] = (draft[b, cut] + 7) % vocab
        loop.logits.copy_(logits)
        loop.draft_tokens.copy_(draft)
        idx_before, n_before = loop.indices.cpu(), loop.n_idx.cpu()
        assert torch.equal(loop.committed.cpu(), sim)
        loop.replay()
        torch.cuda.synchronize()
        assert binding.read_status(loop.ws_v) == 0 and binding.read_status(loop.ws_d) == 0
        # drafting steps of this round: the index built at the committed length, the tail behind it
        for j in range(k):
            r_out, _ = oracle.sparse_draft_attn(kv_cpu, qd_cpu[j], idx_before, n_before, sim, sim + j + 1)
            assert (loop.out_d[j].cpu().double() - r_out).abs().max().item() <= TOL, (r, j)
        # verification of the k + 1 rows behind the committed length
        ctx_v = sim + k + 1
        o_out, _, o_stats = oracle.verify_attn(kv_cpu, qv_cpu, ctx_v, 16, loop.stat_stride)
        assert (loop.out_v.cpu().double() - o_out).abs().max().item() <= TOL, r
        for b in range(2):
            T = int(ctx_v[b])
            assert (loop.stats[:, b, :, :T].cpu().double() - o_stats[:, b, :, :T]).abs().max().item() <= TOL
        # acceptance and the committed length
        _, m, nxt = oracle.accept_greedy(logits, draft)
        assert torch.equal(loop.n_accepted.cpu(), m) and torch.equal(loop.next_token.cpu(), nxt)
        sim = sim + m + 1
        assert torch.equal(loop.committed.cpu(), sim)
        assert torch.equal(loop.ctx_verify.cpu(), sim + k + 1)
        assert torch.equal(loop.cur_len.cpu(), torch.stack([sim + j + 1 for j in range(k)]))
        # controller: sequence 0's drafted tokens
        ent = oracle.token_entropy(logits[0, :k])
        state = oracle.controller_update(state, ent, int(m[0]), 0.9)
        assert (loop.state.cpu().double() - state).abs().max().item() <= 2e-4
        assert 1 <= int(loop.k_star) <= k
        # the index of the next round: built at the new committed length from this round's statistic
        o_idx, o_n = oracle.select_recall(loop.stats.cpu(), sim, cfg.k_sink, cfg.k_recent, cfg.k_total)
        assert torch.equal(loop.indices.cpu(), o_idx) and torch.equal(loop.n_idx.cpu(), o_n)
    assert int(sim.min()) > int(committed0.min()) + rounds  # the loop moved
