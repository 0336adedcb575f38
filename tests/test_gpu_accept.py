"""Greedy tokens and prefix acceptance on the GPU against the oracle, through the C ABI.
Integer results: bit-exact, including which of several equal maxima is reported (the smallest
index) when the equal values sit in different threads, warps and CTAs of the cluster."""
import random

import pytest
import torch

import oracle
from paper_2607_27735_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def _oracle_argmax(logits2d):
    rows, vocab = logits2d.shape
    t, _, _ = oracle.accept_greedy(logits2d.contiguous().view(rows, 1, vocab), torch.zeros(rows, 0, dtype=torch.int32))
    return t.view(rows)


def _same_layout(view, device):
    base = torch.empty(view.storage_offset() + (view.shape[0] - 1) * view.stride(0) + view.shape[1] + 8,
                       dtype=view.dtype, device=device)
    out = base.as_strided(view.shape, view.stride(), view.storage_offset())
    out.copy_(view)
    return out


@pytest.mark.parametrize("rows,vocab,dtype,stride,offset", [
    (1, 128256, torch.bfloat16, None, 0),
    (9, 128256, torch.bfloat16, None, 0),
    (40, 128256, torch.bfloat16, None, 0),
    (200, 32000, torch.float32, None, 0),
    (300, 1003, torch.bfloat16, 1003, 0),
    (7, 50257, torch.bfloat16, 50304, 0),
    (3, 4096, torch.bfloat16, 4096, 3),
    (3, 4099, torch.float32, 4100, 1),
    (2, 1, torch.float32, None, 0),
])
def test_argmax_and_fused_entropy_match_oracle(rows, vocab, dtype, stride, offset):
    logits = inputs.make_logits(rows, vocab, dtype, seed=3 * rows + vocab, row_stride=stride, offset=offset)
    gen = torch.Generator().manual_seed(rows)
    # bf16 logits tie by themselves; plant more: copy each row's maximum to a few other places
    for r in range(rows):
        top = logits[r].max()
        where = torch.randint(0, vocab, (3,), generator=gen)
        logits[r, where] = top
    if rows > 1:
        logits[1] = 0.25  # a constant row: index 0
    dev_logits = _same_layout(logits, "cuda")
    token, ent = binding.spec_token_argmax(dev_logits, want_entropy=True)
    assert torch.equal(token.cpu(), _oracle_argmax(logits))
    assert (ent.cpu().double() - oracle.token_entropy(logits)).abs().max().item() <= 2e-4
    token_only, none = binding.spec_token_argmax(dev_logits)
    assert none is None and torch.equal(token_only, token)
    assert torch.equal(binding.spec_token_entropy(dev_logits), ent)  # the same arithmetic with or without the argmax


@pytest.mark.parametrize("seed", range(12))
def test_accept_matches_oracle(seed):
    rng = random.Random(700 + seed)
    batch = rng.choice([1, 2, 5, 16, 64])
    k = rng.choice([0, 1, 2, 4, 8, 16])
    vocab = rng.choice([1000, 32000, 128256]) if batch * (k + 1) <= 200 else 1000
    dtype = rng.choice([torch.bfloat16, torch.bfloat16, torch.float32])
    logits = inputs.make_logits(batch * (k + 1), vocab, dtype, seed=seed).view(batch, k + 1, vocab).contiguous()
    greedy = _oracle_argmax(logits.view(-1, vocab)).view(batch, k + 1)
    # drafts that agree with the target up to a random point, disagree there, and agree again after
    gen = torch.Generator().manual_seed(seed)
    draft = greedy[:, :k].clone()
    for b in range(batch):
        cut = rng.randint(0, k)
        if cut < k:
            draft[b, cut] = (draft[b, cut] + 1 + rng.randrange(vocab - 1)) % vocab if vocab > 1 else draft[b, cut]
    n_draft = None
    if seed % 3 == 2 and k > 0:
        n_draft = torch.randint(0, k + 1, (batch,), generator=gen, dtype=torch.int32)
    t, m, nxt = binding.spec_accept_greedy(logits.cuda(), draft.cuda(), None if n_draft is None else n_draft.cuda())
    r_t, r_m, r_nxt = oracle.accept_greedy(logits, draft, n_draft)
    assert torch.equal(t.cpu(), r_t) and torch.equal(m.cpu(), r_m) and torch.equal(nxt.cpu(), r_nxt)


def test_accept_full_width_batch_and_clamped_lengths():
    # the 8B family's vocabulary, 64 sequences x (8 + 1) rows: the fourth workload's verification output
    batch, k, vocab = 64, 8, 128256
    logits = inputs.make_logits(batch * (k + 1), vocab, seed=77).view(batch, k + 1, vocab).contiguous()
    greedy = _oracle_argmax(logits.view(-1, vocab)).view(batch, k + 1)
    draft = greedy[:, :k].clone()
    draft[::3, 5] += 1
    draft[1::3, 0] += 1
    n_draft = torch.full((batch,), 99, dtype=torch.int32)   # out of range: clamped to k
    n_draft[7] = -4                                         # clamped to 0
    t, m, nxt = binding.spec_accept_greedy(logits.cuda(), draft.cuda(), n_draft.cuda())
    clamped = n_draft.clamp(0, k)
    r_t, r_m, r_nxt = oracle.accept_greedy(logits, draft, clamped)
    assert torch.equal(t.cpu(), r_t) and torch.equal(m.cpu(), r_m) and torch.equal(nxt.cpu(), r_nxt)
    assert set(m.tolist()) >= {0, 5, 8}


def test_accept_argument_errors():
    logits = torch.zeros(2, 3, 64, device="cuda")
    draft = torch.zeros(2, 2, dtype=torch.int32, device="cuda")
    with pytest.raises(ValueError):
        binding.spec_accept_greedy(logits[:, :, :32], draft)           # not contiguous
    with pytest.raises(ValueError):
        binding.spec_accept_greedy(logits.half(), draft)
    lib = binding.load()
    assert lib.spec_accept_greedy(None, 0, 1, 2, 8, 8, None, None, None, None, None, None) == -1
    assert lib.spec_token_argmax(logits.data_ptr(), 0, 6, 64, 32, draft.data_ptr(), None, None) == -1  # stride < vocab
