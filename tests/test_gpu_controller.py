"""Speculation-length controller on the GPU against the fp64 oracle, through the C ABI:
token entropies (one pass over the logits), the tracked means (Eq. "ema"), the acceptance
probabilities (Eq. "prob") and the selected length (Eq. "optimal_k").

Tolerances: the kernels compute in fp32 with hardware exponentials; an entropy is a sum of
about |z| + ln V sized terms, so 2e-4 absolute covers it with margin; means, probabilities and
scores are a few fp32 operations each (1e-5).  The selected length is an argmax: it must be
the argmax (smaller length on ties) of the scores the device itself wrote, bit for bit, and it
must equal the oracle's choice whenever the oracle's two best scores differ by more than the
score tolerance."""
import random

import pytest
import torch

import oracle
from paper_2607_27735_b200 import binding, inputs

pytestmark = pytest.mark.gpu
ENT_TOL = 2e-4
TOL = 1e-5


@pytest.mark.parametrize("rows,vocab,dtype,stride,offset", [
    (1, 128256, torch.bfloat16, None, 0),     # one drafted token: a row over a cluster of eight
    (8, 128256, torch.bfloat16, None, 0),
    (40, 128256, torch.bfloat16, None, 0),    # clusters of two
    (5, 32000, torch.float32, None, 0),
    (300, 1003, torch.bfloat16, 1003, 0),     # ragged vocabulary, rows not 16-byte aligned
    (7, 50257, torch.bfloat16, 50304, 0),     # padded rows
    (3, 4096, torch.bfloat16, 4096, 3),       # base pointer off the vector boundary
    (3, 4099, torch.float32, 4100, 1),
    (2, 1, torch.float32, None, 0),           # a single token: entropy 0
    (4, 7, torch.bfloat16, None, 0),
])
def test_entropy_matches_oracle(rows, vocab, dtype, stride, offset):
    logits = inputs.make_logits(rows, vocab, dtype, seed=rows + vocab, row_stride=stride, offset=offset)
    ref = oracle.token_entropy(logits)
    got = binding.spec_token_entropy(logits.cuda() if stride is None and offset == 0 else
                                     _same_layout(logits, "cuda"))
    assert (got.cpu().double() - ref).abs().max().item() <= ENT_TOL


def _same_layout(view, device):
    """Moves a strided view to the device keeping stride and storage offset."""
    base = torch.empty(view.storage_offset() + (view.shape[0] - 1) * view.stride(0) + view.shape[1] + 8,
                       dtype=view.dtype, device=device)
    out = base.as_strided(view.shape, view.stride(), view.storage_offset())
    out.copy_(view)
    return out


def test_entropy_special_rows():
    V = 128256
    logits = torch.zeros(4, V)
    logits[1, 77] = 200.0                    # one-hot limit
    logits[2] = 55.5                         # uniform, shifted
    logits[3, :2] = 30.0                     # two equal tokens far above the rest
    got = binding.spec_token_entropy(logits.cuda()).cpu().double()
    ref = oracle.token_entropy(logits)
    assert (got - ref).abs().max().item() <= ENT_TOL
    assert abs(got[0].item() - torch.log(torch.tensor(float(V))).item()) <= ENT_TOL
    assert abs(got[1].item()) <= ENT_TOL


def test_update_chain_matches_oracle():
    rng = random.Random(3)
    state = torch.tensor([1.0, 3.0], device="cuda")
    ref = torch.tensor([1.0, 3.0], dtype=torch.float64)
    n_acc = torch.zeros(1, dtype=torch.int32, device="cuda")
    for step in range(40):
        k = rng.choice([1, 2, 4, 8, 16, 33, 100])
        m = rng.choice([0, k, rng.randint(0, k)])
        ent = torch.rand(k, generator=torch.Generator().manual_seed(step)) * 6.0
        beta = rng.choice([0.0, 0.5, 0.9, 0.99, 1.0])
        n_acc.fill_(m)
        binding.spec_controller_update(state, ent.cuda(), n_acc, beta)
        ref = oracle.controller_update(ref, ent.double(), m, beta)
        assert (state.cpu().double() - ref).abs().max().item() <= TOL * 10, (step, k, m, beta)
    # out-of-range acceptance counts are clamped
    before = state.clone()
    ent = torch.tensor([2.0, 4.0], device="cuda")
    n_acc.fill_(9)
    binding.spec_controller_update(state, ent, n_acc, 0.5)
    assert abs(state[0].item() - (0.5 * before[0].item() + 0.5 * 3.0)) <= TOL * 10
    assert state[1].item() == before[1].item()


def _argmax_small_on_ties(score, cand):
    best, best_s = 0, -1.0
    for s, k in zip(score.tolist(), cand.tolist()):
        if s > best_s or (s == best_s and k < best):
            best, best_s = k, s
    return best


@pytest.mark.parametrize("seed", range(24))
def test_select_matches_oracle(seed):
    rng = random.Random(50 + seed)
    n = rng.choice([1, 2, 8, 16, 31, 32, 33, 100, 256])
    gen = torch.Generator().manual_seed(seed)
    ent = torch.rand(n, generator=gen) * rng.choice([0.5, 3.0, 8.0])
    state = torch.tensor([rng.uniform(0.0, 3.0), rng.uniform(0.0, 6.0)])
    if seed % 6 == 5:
        state[1] = state[0]                   # equal centres: every p is exactly one half
    cand = sorted(rng.sample(range(1, n + 1), min(n, rng.choice([1, 3, 8, 20]))))
    if seed % 4 == 1:
        rng.shuffle(cand)                     # order of the candidates must not matter
    cand = torch.tensor(cand, dtype=torch.int32)
    c_d, c_v = rng.choice([(1.0, 1.0), (0.05, 1.0), (1.0, 0.0), (0.3, 2.5), (0.0, 1.0)])
    k_star, p, score = binding.spec_controller_select(state.cuda(), ent.cuda(), cand.cuda(), c_d, c_v)
    r_k, r_p, r_score = oracle.controller_select(state.double(), ent.double(), cand, c_d, c_v)
    assert (p.cpu().double() - r_p).abs().max().item() <= TOL
    rel = ((score.cpu().double() - r_score).abs() / r_score.abs().clamp_min(1e-30)).max().item()
    assert rel <= TOL
    assert int(k_star) == _argmax_small_on_ties(score.cpu(), cand)
    top = torch.sort(r_score, descending=True).values
    if top.numel() == 1 or (top[0] - top[1]) / top[0] > 4 * TOL:
        assert int(k_star) == r_k


def test_select_ignores_invalid_candidates_and_rejects_long_inputs():
    ent = torch.full((8,), 1.0, device="cuda")
    state = torch.tensor([1.0, 5.0], device="cuda")
    cand = torch.tensor([0, 9, -3, 4, 100], dtype=torch.int32, device="cuda")
    k_star, _, score = binding.spec_controller_select(state, ent, cand, 0.1, 1.0)
    assert int(k_star) == 4
    assert score.cpu().tolist()[:3] == [-1.0, -1.0, -1.0] and score[4].item() == -1.0
    k_star, _, _ = binding.spec_controller_select(state, ent, cand[:3].contiguous(), 0.1, 1.0)
    assert int(k_star) == 0
    with pytest.raises(binding.SpecError):
        binding.spec_controller_select(state, torch.ones(257, device="cuda"),
                                       torch.tensor([1], dtype=torch.int32, device="cuda"), 1.0, 1.0)
    with pytest.raises(binding.SpecError):
        binding.spec_controller_update(state, ent, torch.zeros(1, dtype=torch.int32, device="cuda"), 1.5)


def test_controller_inside_one_graph():
    """Entropy -> update -> select captured once; the replays see new logits and new acceptance
    counts through device memory only."""
    k, V = 8, 32000
    logits = torch.empty(k, V, dtype=torch.bfloat16, device="cuda")
    ent = torch.empty(k, device="cuda")
    state = torch.tensor([1.0, 4.0], device="cuda")
    n_acc = torch.zeros(1, dtype=torch.int32, device="cuda")
    cand = torch.arange(1, k + 1, dtype=torch.int32, device="cuda")
    k_star = torch.zeros(1, dtype=torch.int32, device="cuda")
    p = torch.empty(k, device="cuda")
    score = torch.empty(k, device="cuda")

    def step():
        binding.spec_token_entropy(logits, entropy=ent)
        binding.spec_controller_update(state, ent, n_acc, 0.9)
        binding.spec_controller_select(state, ent, cand, 0.08, 1.0, k_star=k_star, p=p, score=score)

    logits.copy_(inputs.make_logits(k, V, seed=99))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    state.copy_(torch.tensor([1.0, 4.0]))
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    ref_state = torch.tensor([1.0, 4.0], dtype=torch.float64)
    for trial in range(4):
        lg = inputs.make_logits(k, V, seed=trial)
        logits.copy_(lg)
        m = [3, 0, 8, 5][trial]
        n_acc.fill_(m)
        graph.replay()
        torch.cuda.synchronize()
        r_ent = oracle.token_entropy(lg)
        ref_state = oracle.controller_update(ref_state, r_ent, m, 0.9)
        r_k, r_p, r_score = oracle.controller_select(ref_state, r_ent, cand.cpu(), 0.08, 1.0)
        assert (ent.cpu().double() - r_ent).abs().max().item() <= ENT_TOL
        assert (state.cpu().double() - ref_state).abs().max().item() <= ENT_TOL
        assert (p.cpu().double() - r_p).abs().max().item() <= 2 * ENT_TOL
        assert int(k_star) == _argmax_small_on_ties(score.cpu(), cand.cpu())
        top = torch.sort(r_score, descending=True).values
        if (top[0] - top[1]) / top[0] > 1e-3:
            assert int(k_star) == r_k
