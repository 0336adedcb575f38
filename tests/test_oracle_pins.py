"""Pins of the CPU oracle against things other than itself: a library fp64 softmax
attention, closed forms, limits, brute force, and structural invariants."""
import math

import pytest
import torch

import oracle
from paper_2607_27735_b200 import inputs
from conftest import dense_rows


def torch_verify_reference(case, stat_window=16):
    """softmax(Q K^T * scale + causal mask) V with torch fp64 ops, one (l, b, h, g) at a time."""
    kv, cfg = case.kv, case.cfg
    L, B, n_q, Hq, D = case.q_verify.shape
    G = Hq // kv.n_kv_heads
    W = min(stat_window, n_q)
    smax = int(case.ctx_len.max())
    out = torch.zeros(L, B, n_q, Hq, D, dtype=torch.float64)
    lse = torch.zeros(L, B, n_q, Hq, dtype=torch.float64)
    stats = torch.zeros(L, B, kv.n_kv_heads, smax, dtype=torch.float64)
    for l in range(L):
        for b in range(B):
            T = int(case.ctx_len[b])
            for h in range(kv.n_kv_heads):
                K = dense_rows(kv, kv.k, l, b, h, range(T))
                V = dense_rows(kv, kv.v, l, b, h, range(T))
                for g in range(G):
                    q = case.q_verify[l, b, :, h * G + g].to(torch.float64)  # [n_q, D]
                    s = q @ K.T / math.sqrt(D)
                    row_pos = torch.arange(T - n_q, T)[:, None]
                    s = s.masked_fill(torch.arange(T)[None, :] > row_pos, float("-inf"))
                    p = torch.softmax(s, dim=-1)
                    out[l, b, :, h * G + g] = p @ V
                    lse[l, b, :, h * G + g] = torch.logsumexp(s, dim=-1)
                    stats[l, b, h, :T] += p[n_q - W:].sum(0)
    return out, lse, stats


SHAPES = [
    dict(n_q_heads=4, n_kv_heads=4, head_dim=64, ctx=(37, 37), n_q=1),
    dict(n_q_heads=8, n_kv_heads=2, head_dim=64, ctx=(130, 130), n_q=5),
    dict(n_q_heads=10, n_kv_heads=2, head_dim=128, ctx=(65, 65), n_q=17),
    dict(n_q_heads=8, n_kv_heads=2, head_dim=128, ctx=(40, 90), n_q=3, batch=3, page_size=16,
         shuffled_pages=True, n_layers=2),
]


@pytest.mark.parametrize("shape", SHAPES)
def test_verify_matches_library_softmax_attention(shape):
    cfg = inputs.small_config(planted=3, **shape)
    case = inputs.make_case(cfg)
    out, lse, stats = oracle.verify_attn(case.kv, case.q_verify, case.ctx_len)
    ro, rl, rs = torch_verify_reference(case)
    assert (out - ro).abs().max() < 1e-12
    assert (lse - rl).abs().max() < 1e-12
    assert (stats - rs).abs().max() < 1e-12


@pytest.mark.parametrize("n_q,window", [(1, 16), (5, 16), (17, 16), (9, 4)])
def test_statistic_mass_is_group_times_window_rows(n_q, window):
    cfg = inputs.small_config(n_q=n_q, ctx=(300, 300), n_q_heads=8, n_kv_heads=2)
    case = inputs.make_case(cfg)
    _, _, stats = oracle.verify_attn(case.kv, case.q_verify, case.ctx_len, stat_window=window)
    expect = cfg.group * min(window, n_q)
    assert (stats.sum(-1) - expect).abs().max() < 1e-9
    assert stats.min() >= 0.0


def test_identical_keys_closed_form():
    """All keys equal: p = 1/(pos+1), O = running mean of V, statistic = G * sum of 1/(pos_j+1)
    over the window rows that can see the key.  Pins mask alignment, window rule, GQA sum."""
    cfg = inputs.small_config(n_q=17, ctx=(50, 50), n_q_heads=6, n_kv_heads=2, head_dim=64,
                              planted=0)
    case = inputs.make_case(cfg)
    kv = case.kv
    kv.k[:] = kv.k.reshape(-1, 64)[0]  # one key row everywhere
    out, lse, stats = oracle.verify_attn(kv, case.q_verify, case.ctx_len, stat_window=16)
    T, n_q, G = 50, 17, 3
    for h in range(2):
        V = dense_rows(kv, kv.v, 0, 0, h, range(T))
        for j in range(n_q):
            pos = T - n_q + j
            mean_v = V[: pos + 1].mean(0)
            for g in range(G):
                assert (out[0, 0, j, h * G + g] - mean_v).abs().max() < 1e-12
        expect = torch.zeros(T, dtype=torch.float64)
        for j in range(1, n_q):  # W=16 of 17 rows: row 0 is outside the window
            pos = T - n_q + j
            expect[: pos + 1] += G / (pos + 1)
        assert (stats[0, 0, h, :T] - expect).abs().max() < 1e-12


def test_golden_three_token_example():
    """tests/golden/identical_keys_T3.txt: hand-computed case (T=3, n_q=2, G=1, identical keys)."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "identical_keys_T3.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    golden = {r[0]: [float(x) for x in r[1:]] for r in rows}
    cfg = inputs.small_config(n_q=2, ctx=(3, 3), n_q_heads=1, n_kv_heads=1, head_dim=64, planted=0,
                              draft_steps=0)
    case = inputs.make_case(cfg)
    kv = case.kv
    kv.k[:] = 0.5
    kv.v[:] = 0
    for i, val in enumerate(golden["v"]):
        kv.v[0, 0, 0, i, :] = val
    out, _, stats = oracle.verify_attn(kv, case.q_verify, case.ctx_len)
    assert torch.allclose(stats[0, 0, 0, :3], torch.tensor(golden["stats"], dtype=torch.float64),
                          atol=1e-12)
    assert torch.allclose(out[0, 0, :, 0, 0], torch.tensor(golden["out"], dtype=torch.float64),
                          atol=1e-12)


def test_one_hot_limit():
    """A key equal to 50x the (unit) query direction takes all the mass."""
    cfg = inputs.small_config(n_q=4, ctx=(200, 200), n_q_heads=4, n_kv_heads=1, head_dim=64,
                              planted=0)
    case = inputs.make_case(cfg)
    kv = case.kv
    qdir = case.direction[0, 0, 0]
    hot = 77
    kv.k[0, 0, 0, hot] = (50.0 * qdir / qdir.norm() * math.sqrt(64.0)).to(torch.bfloat16)
    out, _, stats = oracle.verify_attn(kv, case.q_verify, case.ctx_len)
    v_hot = kv.v[0, 0, 0, hot].to(torch.float64)
    assert (out[0, 0] - v_hot).abs().max() < 1e-6
    assert abs(float(stats[0, 0, 0, hot]) - 16.0) < 1e-6  # R = n_q * G rows


def test_prefix_permutation_invariance():
    """Permuting (K, V) rows that every window row can see permutes the statistic, keeps O."""
    cfg = inputs.small_config(n_q=3, ctx=(90, 90), head_dim=64)
    case = inputs.make_case(cfg)
    out, _, stats = oracle.verify_attn(case.kv, case.q_verify, case.ctx_len)
    T, n_q = 90, 3
    perm = torch.randperm(T - n_q, generator=torch.Generator().manual_seed(1))
    kv = case.kv
    k2, v2 = kv.k.clone(), kv.v.clone()
    k2[0, 0, :, : T - n_q] = kv.k[0, 0, :, perm]
    v2[0, 0, :, : T - n_q] = kv.v[0, 0, :, perm]
    import dataclasses
    kvp = dataclasses.replace(kv, k=k2, v=v2)
    out2, _, stats2 = oracle.verify_attn(kvp, case.q_verify, case.ctx_len)
    assert (out - out2).abs().max() < 1e-12
    assert (stats[..., perm] - stats2[..., : T - n_q]).abs().max() < 1e-12


# ---------------------------------------------------------------------------------------------
# select


def brute_select(st, T, k_sink, k_recent, k_total):
    if T <= k_total:
        return list(range(T))
    cand = list(range(k_sink, T - k_recent))
    cand.sort(key=lambda i: (-float(st[i]), i))
    chosen = cand[: k_total - k_sink - k_recent]
    return sorted(list(range(k_sink)) + chosen + list(range(T - k_recent, T)))


@pytest.mark.parametrize("T,k_sink,k_recent,k_total", [
    (64, 4, 8, 24), (64, 0, 0, 10), (20, 4, 8, 24), (24, 4, 8, 24), (25, 4, 8, 24),
    (300, 4, 64, 68), (300, 4, 64, 100), (13, 13, 0, 13), (40, 5, 5, 10),
])
def test_select_brute_force_with_ties(T, k_sink, k_recent, k_total):
    g = torch.Generator().manual_seed(T * 31 + k_total)
    # few distinct values: many exact ties, including across the selection threshold
    stats = (torch.randint(0, 5, (2, 2, 3, T + 7), generator=g).float()) * 0.25
    sel_len = torch.tensor([T, max(1, T - 3)], dtype=torch.int32)
    idx, n = oracle.select_recall(stats, sel_len, k_sink, k_recent, k_total)
    for l in range(2):
        for b in range(2):
            for h in range(3):
                want = brute_select(stats[l, b, h], int(sel_len[b]), k_sink, k_recent, k_total)
                got = idx[l, b, h, : int(n[l, b, h])].tolist()
                assert got == want
                assert int(n[l, b, h]) == min(k_total, int(sel_len[b]))
                assert (idx[l, b, h, int(n[l, b, h]):] == -1).all()


def test_select_all_equal_scores_takes_lowest_positions():
    stats = torch.ones(1, 1, 1, 100)
    idx, n = oracle.select_recall(stats, torch.tensor([100], dtype=torch.int32), 2, 3, 15)
    assert idx[0, 0, 0].tolist() == list(range(0, 12)) + [97, 98, 99]


def test_select_set_matches_torch_topk_on_distinct_values():
    g = torch.Generator().manual_seed(5)
    T, k_sink, k_recent, k_total = 5000, 4, 64, 512
    stats = torch.rand(1, 2, 4, T, generator=g)
    idx, n = oracle.select_recall(stats, torch.tensor([T, T], dtype=torch.int32), k_sink,
                                  k_recent, k_total)
    k_mid = k_total - k_sink - k_recent
    for b in range(2):
        for h in range(4):
            mid = stats[0, b, h, k_sink:T - k_recent]
            top = (mid.topk(k_mid).indices + k_sink).sort().values
            got = idx[0, b, h]
            assert got[:k_sink].tolist() == list(range(k_sink))
            assert got[-k_recent:].tolist() == list(range(T - k_recent, T))
            assert torch.equal(got[k_sink:-k_recent].long(), top)
            assert len(set(got.tolist())) == k_total  # no duplicates: sink/recent are excluded


# ---------------------------------------------------------------------------------------------
# draft


def test_draft_matches_library_softmax_on_explicit_subset():
    cfg = inputs.small_config(ctx=(300, 300), n_q=2, draft_steps=3, batch=2, n_layers=2,
                              page_size=16, shuffled_pages=True)
    case = inputs.make_case(cfg)
    kv = case.kv
    g = torch.Generator().manual_seed(9)
    k_total = 40
    idx = torch.full((2, 2, 2, k_total), -1, dtype=torch.int32)
    n_idx = torch.zeros(2, 2, 2, dtype=torch.int32)
    tail_start = torch.tensor([290, 300], dtype=torch.int32)
    cur_len = torch.tensor([293, 300], dtype=torch.int32)  # second sequence: empty tail
    for l in range(2):
        for b in range(2):
            for h in range(2):
                n = int(torch.randint(1, k_total + 1, (1,), generator=g))
                sel = torch.randperm(int(tail_start[b]), generator=g)[:n].sort().values
                idx[l, b, h, :n] = sel.int()
                n_idx[l, b, h] = n
    q = case.q_draft[0]
    out, lse = oracle.sparse_draft_attn(kv, q, idx, n_idx, tail_start, cur_len)
    G = cfg.group
    for l in range(2):
        for b in range(2):
            for h in range(2):
                keys = idx[l, b, h, : int(n_idx[l, b, h])].tolist() + list(
                    range(int(tail_start[b]), int(cur_len[b])))
                K = dense_rows(kv, kv.k, l, b, h, keys)
                V = dense_rows(kv, kv.v, l, b, h, keys)
                for gg in range(G):
                    qq = q[l, b, h * G + gg].to(torch.float64)
                    s = K @ qq / math.sqrt(cfg.head_dim)
                    p = torch.softmax(s, 0)
                    assert (out[l, b, h * G + gg] - p @ V).abs().max() < 1e-12
                    assert abs(float(lse[l, b, h * G + gg] - torch.logsumexp(s, 0))) < 1e-12


def test_budget_at_least_context_reduces_draft_to_dense_attention():
    """select with k_total >= T' keeps 0..T'-1, and the draft then equals verification with
    n_q = 1 on the same cache (the query being the last cached position)."""
    cfg = inputs.small_config(ctx=(150, 150), n_q=1, draft_steps=1, head_dim=64)
    case = inputs.make_case(cfg)
    T = 150
    stats = torch.rand(1, 1, 2, T)
    idx, n = oracle.select_recall(stats, torch.tensor([T - 1], dtype=torch.int32), 4, 16, 256)
    assert idx[0, 0, 0, : T - 1].tolist() == list(range(T - 1)) and int(n[0, 0, 0]) == T - 1
    q1 = case.q_verify[:, :, 0]  # [L, B, Hq, D]
    d_out, d_lse = oracle.sparse_draft_attn(
        case.kv, q1, idx, n, torch.tensor([T - 1], dtype=torch.int32),
        torch.tensor([T], dtype=torch.int32))
    v_out, v_lse, _ = oracle.verify_attn(case.kv, case.q_verify, case.ctx_len)
    assert (d_out - v_out[:, :, 0]).abs().max() < 1e-12
    assert (d_lse - v_lse[:, :, 0]).abs().max() < 1e-12


def test_planted_heavy_hitters_are_recalled():
    """Tiny baseline workload: every planted position outside sink/recent lands in the index
    set and the planted set carries most of the window's attention mass."""
    cfg = inputs.baseline_configs()["cfg1_tiny"]
    case = inputs.make_case(cfg)
    _, _, stats = oracle.verify_attn(case.kv, case.q_verify, case.ctx_len)
    idx, _ = oracle.select_recall(stats.float(), case.ctx_len, cfg.k_sink, cfg.k_recent,
                                  cfg.k_total)
    for h in range(cfg.n_kv_heads):
        chosen = set(idx[0, 0, h].tolist())
        planted = case.planted_pos[0, 0, h].tolist()
        assert all(p in chosen for p in planted)
        assert stats[0, 0, h][planted].sum() / stats[0, 0, h].sum() > 0.5


def test_resampled_heavy_hitters_are_recalled_from_the_fresh_statistic():
    """Third workload's drift, scaled down: every round some planted positions move; the index
    rebuilt from that round's statistic holds the CURRENT set, an index kept from the round
    before misses exactly the positions that moved in."""
    cfg = inputs.small_config(ctx=(3000, 3000), planted=0.02, k_total=256, k_recent=16,
                              planted_mult=4.0, planted_noise=False, seed=5)
    case = inputs.make_case(cfg)
    prev_idx = None
    for step in range(3):
        moved = inputs.resample_planted(case, 0.25, step)
        assert moved > 0
        _, _, stats = oracle.verify_attn(case.kv, case.q_verify, case.ctx_len)
        idx, _ = oracle.select_recall(stats.float(), case.ctx_len, cfg.k_sink, cfg.k_recent,
                                      cfg.k_total)
        for h in range(cfg.n_kv_heads):
            planted = set(case.planted_pos[0, 0, h].tolist())
            assert len(planted) == case.planted_pos.shape[-1]  # positions stay distinct
            assert planted <= set(idx[0, 0, h].tolist())
            if prev_idx is not None:
                stale = set(prev_idx[0, 0, h].tolist())
                assert len(planted - stale) > 0  # the drift is visible to a stale index
        prev_idx = idx


# ---- entropy-guided length controller -----------------------------------------------------------


def test_entropy_closed_forms():
    """Uniform logits -> ln V; two equal peaks far above the rest -> ln 2; one dominant logit -> 0;
    adding a constant to a row changes nothing."""
    V = 1000
    z = torch.zeros(4, V)
    z[1, :2] = 80.0
    z[2, 7] = 200.0
    z[3] = torch.linspace(-3, 3, V)
    h = oracle.token_entropy(z)
    assert abs(h[0].item() - math.log(V)) < 1e-12
    assert abs(h[1].item() - math.log(2)) < 1e-9
    assert h[2].item() < 1e-12
    h_shift = oracle.token_entropy(z + 5.0)
    assert (h - h_shift).abs().max().item() < 1e-5  # fp32 inputs: the shift itself rounds


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_entropy_matches_library_softmax(dtype):
    gen = torch.Generator().manual_seed(3)
    z = (3.0 * torch.randn(5, 4099, generator=gen)).to(dtype)
    p = torch.softmax(z.double(), dim=-1)
    ref = -(p * torch.log(p.clamp_min(1e-300))).sum(-1)
    view = z[:, :4000]  # strided rows
    p2 = torch.softmax(view.double(), dim=-1)
    ref2 = -(p2 * torch.log(p2.clamp_min(1e-300))).sum(-1)
    assert (oracle.token_entropy(z) - ref).abs().max().item() < 1e-10
    assert (oracle.token_entropy(view) - ref2).abs().max().item() < 1e-10


def test_controller_update_and_select_closed_forms():
    # equal centres => p = 1/2 for every token => expected length 1 + sum 2^-m
    k_star, p, score = oracle.controller_select([1.0, 1.0], [0.3, 2.0, 5.0, 0.1], [1, 2, 4], 0.1, 1.0)
    assert (p - 0.5).abs().max().item() < 1e-15
    want = [(1 + 0.5) / 1.1, (1 + 0.75) / 1.2, (1 + 0.9375) / 1.4]
    assert max(abs(a - b) for a, b in zip(score.tolist(), want)) < 1e-14
    assert k_star == 2
    # entropies on the accepted centre, rejected centre far away => p -> 1: longer is better while C_d < C_v
    k_star, p, _ = oracle.controller_select([0.5, 40.0], [0.5] * 8, [2, 4, 8], 0.05, 1.0)
    assert (1 - p).max().item() < 1e-15 and k_star == 8
    # ... and the other way round: nothing is expected to pass, the shortest candidate wins
    k_star, p, _ = oracle.controller_select([40.0, 0.5], [0.5] * 8, [2, 4, 8], 0.05, 1.0)
    assert p.max().item() < 1e-15 and k_star == 2
    # exact tie (C_d = 0, p = 0): the smaller candidate
    k_star, _, score = oracle.controller_select([40.0, 0.5], [0.5] * 8, [4, 2], 0.0, 1.0)
    assert score[0] == score[1] and k_star == 2
    # Eq. "ema": 3 of 5 accepted
    s = oracle.controller_update([1.0, 2.0], [0.2, 0.4, 0.6, 3.0, 5.0], 3, 0.9)
    assert abs(s[0].item() - (0.9 * 1.0 + 0.1 * 0.4)) < 1e-15 and abs(s[1].item() - (0.9 * 2.0 + 0.1 * 4.0)) < 1e-15
    # an empty class leaves its mean alone
    s = oracle.controller_update([1.0, 2.0], [0.2, 0.4], 2, 0.5)
    assert abs(s[0].item() - 0.65) < 1e-15 and s[1].item() == 2.0
    s = oracle.controller_update([1.0, 2.0], [0.2, 0.4], 0, 0.5)
    assert s[0].item() == 1.0 and abs(s[1].item() - 1.15) < 1e-15


def test_controller_select_against_plain_python():
    rng = __import__("random").Random(11)
    for _ in range(50):
        n = rng.randint(1, 20)
        ent = [rng.uniform(0, 6) for _ in range(n)]
        state = [rng.uniform(0, 3), rng.uniform(1, 6)]
        cand = sorted(rng.sample(range(1, n + 1), rng.randint(1, min(5, n))))
        c_d, c_v = rng.uniform(0.01, 0.5), rng.uniform(0.5, 2.0)
        k_star, p, score = oracle.controller_select(state, ent, cand, c_d, c_v)
        ps = [math.exp(-abs(h - state[0])) / (math.exp(-abs(h - state[0])) + math.exp(-abs(h - state[1]))) for h in ent]
        best, best_k = -1.0, None
        for k in cand:
            exp_len, pref = 1.0, 1.0
            for i in range(k):
                pref *= ps[i]
                exp_len += pref
            sc = exp_len / (k * c_d + c_v)
            if sc > best:
                best, best_k = sc, k
        assert k_star == best_k
        assert max(abs(a - b) for a, b in zip(p.tolist(), ps)) < 1e-14


# ---- prefix acceptance (Sec. "The Draft-Verification Paradigm", greedy reading) ----

def test_accept_argmax_matches_library_and_breaks_ties_low():
    gen = torch.Generator().manual_seed(4)
    logits = torch.randn(3, 5, 777, generator=gen)
    draft = torch.zeros(3, 4, dtype=torch.int32)
    target, _, _ = oracle.accept_greedy(logits, draft)
    assert torch.equal(target.long(), logits.argmax(dim=-1))          # tie-free rows: any argmax agrees
    tied = torch.zeros(1, 2, 50)
    tied[0, 0, [7, 30, 31]] = 2.5                                       # equal maxima: the smallest index
    tied[0, 1, :] = -1.0                                                # a constant row: index 0
    target, _, _ = oracle.accept_greedy(tied.to(torch.bfloat16), torch.zeros(1, 1, dtype=torch.int32))
    assert target.tolist() == [[7, 0]]


def test_accept_prefix_rule_on_constructed_cases():
    k, V = 6, 64
    want = torch.tensor([[5, 9, 9, 40, 63, 0, 17]])                     # the target model's greedy tokens

    def logits_for(tokens):
        lg = torch.zeros(tokens.shape[0], tokens.shape[1], V)
        lg.scatter_(2, tokens.long().unsqueeze(-1), 3.0)
        return lg

    lg = logits_for(want)
    # every drafted token right: m = k, the corrected token is the bonus row's
    t, m, nxt = oracle.accept_greedy(lg, want[:, :k].int())
    assert t.tolist() == want.tolist() and m.tolist() == [6] and nxt.tolist() == [17]
    # first one wrong: nothing accepted, the corrected token is row 0's
    d = want[:, :k].clone().int()
    d[0, 0] = 6
    _, m, nxt = oracle.accept_greedy(lg, d)
    assert m.tolist() == [0] and nxt.tolist() == [5]
    # mismatch at j = 3; the matches after it must not count
    d = want[:, :k].clone().int()
    d[0, 3] = 41
    _, m, nxt = oracle.accept_greedy(lg, d)
    assert m.tolist() == [3] and nxt.tolist() == [40]
    # ragged speculation lengths: only n_draft tokens are looked at
    batch = logits_for(want.repeat(3, 1))
    d3 = want[:, :k].repeat(3, 1).int()
    _, m, nxt = oracle.accept_greedy(batch, d3, n_draft=[0, 2, 6])
    assert m.tolist() == [0, 2, 6] and nxt.tolist() == [5, 9, 17]
    # k = 0 (plain decoding step): one row, no draft
    _, m, nxt = oracle.accept_greedy(lg[:, :1].contiguous(), torch.zeros(1, 0, dtype=torch.int32))
    assert m.tolist() == [0] and nxt.tolist() == [5]


# ---- the statistic is additive over consecutive verification passes (Eq. 3 as a sum over rows) ----

def test_statistic_of_two_consecutive_passes_adds_up():
    """Rows a then b, verified in two passes (the first against the context that ends where the
    second one's rows begin), give the attention outputs and the Eq. 3 sums of one pass over a + b
    rows: the window is a sum over query rows, each row's probabilities depend on its own prefix
    only.  Catches a window or causal-offset mistake in the oracle without retyping its formula."""
    from paper_2607_27735_b200 import inputs
    a, b = 3, 4
    cfg = inputs.small_config(ctx=(300, 300), n_q=a + b, n_q_heads=8, n_kv_heads=2, planted=3, seed=21)
    case = inputs.make_case(cfg)
    T = int(case.ctx_len[0])
    out, lse, stats = oracle.verify_attn(case.kv, case.q_verify, case.ctx_len, 16)
    qa = case.q_verify[:, :, :a].contiguous()
    qb = case.q_verify[:, :, a:].contiguous()
    out_a, lse_a, st_a = oracle.verify_attn(case.kv, qa, case.ctx_len - b, 16, stat_stride=T)
    out_b, lse_b, st_b = oracle.verify_attn(case.kv, qb, case.ctx_len, 16, stat_stride=T)
    assert (out[:, :, :a] - out_a).abs().max().item() < 1e-12 and (out[:, :, a:] - out_b).abs().max().item() < 1e-12
    assert (lse[:, :, :a] - lse_a).abs().max().item() < 1e-12 and (lse[:, :, a:] - lse_b).abs().max().item() < 1e-12
    assert (stats - (st_a + st_b)).abs().max().item() < 1e-12
    assert st_a[..., T - b:].abs().max().item() == 0.0   # the first pass cannot see the second one's keys


# ---- per-attention-head form of Eq. 3 / Eq. 5 (the paper's literal "per-head" indices) ----

def test_per_head_statistic_sums_to_the_group_statistic():
    from paper_2607_27735_b200 import inputs
    cfg = inputs.small_config(ctx=(200, 260), batch=2, n_q=5, n_q_heads=8, n_kv_heads=2, planted=2, seed=31)
    case = inputs.make_case(cfg)
    out, lse, st = oracle.verify_attn(case.kv, case.q_verify, case.ctx_len, 16)
    out_h, lse_h, st_h = oracle.verify_attn(case.kv, case.q_verify, case.ctx_len, 16, per_head=True)
    L, B, Hq, S = st_h.shape
    assert torch.equal(out, out_h) and torch.equal(lse, lse_h)
    assert (st_h.view(L, B, 2, 4, S).sum(dim=3) - st).abs().max().item() < 1e-12
    # every head's last-row probabilities sum to 1 over the keys, so each head's statistic sums to n_q
    for b in range(B):
        T = int(case.ctx_len[b])
        assert (st_h[:, b, :, :T].sum(dim=-1) - cfg.n_q).abs().max().item() < 1e-9
    # one query head per KV head: the two forms are the same thing
    cfg1 = inputs.small_config(ctx=(150, 150), n_q=3, n_q_heads=2, n_kv_heads=2, seed=32)
    c1 = inputs.make_case(cfg1)
    assert torch.equal(oracle.verify_attn(c1.kv, c1.q_verify, c1.ctx_len, 16)[2],
                       oracle.verify_attn(c1.kv, c1.q_verify, c1.ctx_len, 16, per_head=True)[2])


def test_per_head_draft_with_shared_sets_is_the_group_draft():
    from paper_2607_27735_b200 import inputs
    cfg = inputs.small_config(ctx=(300, 300), n_q=3, n_q_heads=8, n_kv_heads=2, k_total=64, k_recent=8, seed=33)
    case = inputs.make_case(cfg)
    _, _, st = oracle.verify_attn(case.kv, case.q_verify, case.ctx_len, 16)
    idx, n = oracle.select_recall(st.float(), case.ctx_len, cfg.k_sink, cfg.k_recent, cfg.k_total)
    cur = case.ctx_len + 1
    q = case.q_draft[0].contiguous()
    ref_out, ref_lse = oracle.sparse_draft_attn(case.kv, q, idx, n, case.ctx_len, cur)
    idx_h = idx.repeat_interleave(4, dim=2).contiguous()     # every head of a group gets the group's set
    n_h = n.repeat_interleave(4, dim=2).contiguous()
    out_h, lse_h = oracle.sparse_draft_attn(case.kv, q, idx_h, n_h, case.ctx_len, cur, per_head=True)
    assert torch.equal(ref_out, out_h) and torch.equal(ref_lse, lse_h)
    # a head whose own set is the whole context attends densely: equals the verification row at that position
    full = torch.arange(300, dtype=torch.int32).view(1, 1, 1, 300).expand(1, 1, 8, 300).contiguous()
    n_full = torch.full((1, 1, 8), 300, dtype=torch.int32)
    dense, _ = oracle.sparse_draft_attn(case.kv, q, full, n_full, case.ctx_len, case.ctx_len, per_head=True)
    kv_plus = case.kv
    qv = q.view(1, 1, 1, 8, -1).contiguous()
    ver, _, _ = oracle.verify_attn(kv_plus, qv, case.ctx_len, 16)
    assert (dense - ver[:, :, 0]).abs().max().item() < 1e-12


# ---- max instead of sum over the query heads of a group (the other way to fold a GQA group) ----

def test_group_max_statistic_bounds_closed_form_and_mass():
    """oracle.verify_attn(group_max=True): the largest per-head Eq. 3 score of the group at every key.
    Pins: it is the elementwise maximum of the (separately pinned) per-head scores; it lies between
    sum / G and sum; with one head per group it is the summed form bit for bit; on identical keys
    every head gives the same probabilities 1 / (pos + 1), so the closed form is the per-head one;
    and its mass over the keys lies in [min(W, n_q), G min(W, n_q)] and is NOT G min(W, n_q) in
    general, which is why the hot path sums (the sum keeps "every row adds 1 per head")."""
    from paper_2607_27735_b200 import inputs
    cfg = inputs.small_config(ctx=(220, 300), batch=2, n_q=5, n_q_heads=8, n_kv_heads=2, planted=3, seed=41)
    case = inputs.make_case(cfg)
    G = 4
    out, lse, st_sum = oracle.verify_attn(case.kv, case.q_verify, case.ctx_len, 16)
    out_m, lse_m, st_max = oracle.verify_attn(case.kv, case.q_verify, case.ctx_len, 16, group_max=True)
    _, _, st_h = oracle.verify_attn(case.kv, case.q_verify, case.ctx_len, 16, per_head=True)
    assert torch.equal(out, out_m) and torch.equal(lse, lse_m)
    L, B, Hq, S = st_h.shape
    assert torch.equal(st_h.view(L, B, 2, G, S).max(dim=3).values, st_max)
    assert (st_max <= st_sum + 1e-15).all() and (st_max >= st_sum / G - 1e-15).all()
    for b in range(B):
        T = int(case.ctx_len[b])
        mass = st_max[:, b, :, :T].sum(-1)
        assert (mass >= cfg.n_q - 1e-9).all() and (mass <= G * cfg.n_q + 1e-9).all()
        assert (mass < G * cfg.n_q - 1e-3).all()  # heads disagree on these inputs: strictly below the sum's mass
    # one head per group: nothing to fold
    c1 = inputs.make_case(inputs.small_config(ctx=(150, 150), n_q=3, n_q_heads=2, n_kv_heads=2, seed=42))
    assert torch.equal(oracle.verify_attn(c1.kv, c1.q_verify, c1.ctx_len, 16)[2],
                       oracle.verify_attn(c1.kv, c1.q_verify, c1.ctx_len, 16, group_max=True)[2])
    # identical keys: p = 1 / (pos + 1) for every head, so max over heads = one head's score
    T, n_q, W = 40, 6, 4
    c2 = inputs.make_case(inputs.small_config(ctx=(T, T), n_q=n_q, n_q_heads=6, n_kv_heads=2, planted=0, seed=43))
    c2.kv.k[:] = c2.kv.k[:, :, :, :1, :]  # every slot holds the first slot's key
    _, _, st2 = oracle.verify_attn(c2.kv, c2.q_verify, c2.ctx_len, W, group_max=True)
    want = torch.zeros(T, dtype=torch.float64)
    for j in range(n_q - W, n_q):
        pos = T - n_q + j
        want[:pos + 1] += 1.0 / (pos + 1)
    assert (st2[0, 0] - want).abs().max().item() < 1e-12


# ---- 8-bit (e4m3) KV cache: the same attention on dequantised values ----

def test_e4m3_decoder_matches_the_library_cast():
    """All 256 byte patterns against torch's float8_e4m3fn (an independent decoder), NaN patterns included."""
    raw = torch.arange(256, dtype=torch.int32).to(torch.uint8)
    lib = raw.view(torch.float8_e4m3fn).double()
    for b in range(256):
        mine = oracle.e4m3_to_double(b)
        if math.isnan(float(lib[b])):
            assert math.isnan(mine) and (b & 0x7f) == 0x7f
        else:
            assert mine == float(lib[b]), b
    assert oracle.e4m3_to_double(0x7e) == 448.0 and oracle.e4m3_to_double(0x01) == 2.0 ** -9


def test_fp8_cache_is_the_bf16_oracle_on_the_dequantised_cache():
    """Verification (output, LSE, score) and drafting over an e4m3 cache with per-(layer, head) power-of-two
    scales equal, bit for bit, the pinned bf16 functions on the cache of dequantised values (which bf16
    holds exactly), contiguous and paged."""
    from paper_2607_27735_b200 import inputs
    for kw in (dict(ctx=(180, 260), batch=2, n_q=5, n_q_heads=8, n_kv_heads=2, n_layers=2, planted=3, seed=51),
               dict(ctx=(90, 200), batch=3, n_q=3, page_size=16, shuffled_pages=True, planted=0, q_mode="iid",
                    head_dim=64, seed=52)):
        cfg = inputs.small_config(k_total=64, k_recent=8, draft_steps=1, **kw)
        case = inputs.make_case(cfg)
        kv8 = inputs.quantize_kv_fp8(case.kv)
        deq = inputs.dequantize_kv_fp8(kv8)
        assert (kv8.k_scale > 0).all() and torch.equal(torch.log2(kv8.k_scale), torch.log2(kv8.k_scale).round())
        a = oracle.verify_attn(kv8, case.q_verify, case.ctx_len, 16)
        b = oracle.verify_attn(deq, case.q_verify, case.ctx_len, 16)
        for x, y in zip(a, b):
            assert torch.equal(x, y)
        # and it is a different problem from the unquantised one (the cast rounds to 4 significant bits)
        c = oracle.verify_attn(case.kv, case.q_verify, case.ctx_len, 16)
        assert (a[0] - c[0]).abs().max().item() > 1e-4
        idx, n = oracle.select_recall(a[2].float(), case.ctx_len, cfg.k_sink, cfg.k_recent, cfg.k_total)
        q = case.q_draft[0].contiguous()
        d8 = oracle.sparse_draft_attn(kv8, q, idx, n, case.ctx_len, case.ctx_len + 1)
        dd = oracle.sparse_draft_attn(deq, q, idx, n, case.ctx_len, case.ctx_len + 1)
        assert torch.equal(d8[0], dd[0]) and torch.equal(d8[1], dd[1])
