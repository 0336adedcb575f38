"""The no-workspace entry point (collected last on purpose: if it fails, `-x` has already run
every other test).

spec_verify_attn_noalloc serves callers that cannot allocate device memory: its scratch is a
fixed array inside the library.  The test calls it through the C ABI twice in a row (the second
call finds the first call's leftovers in the array) and checks each result against the CPU oracle
within the parity tolerance of the other GPU tests, and against the regular entry point on the
same inputs bit for bit (the same deterministic kernels run on either scratch).  A second shape
then reuses the same array with a different layout."""
import pytest
import torch

import oracle
from paper_2607_27735_b200 import binding, inputs

pytestmark = pytest.mark.gpu
TOL = 2e-3


def _compare(cfg):
    case = inputs.make_case(cfg, device="cuda")
    T = int(case.ctx_len.max())
    ref_out, ref_lse, ref_stats, ws = binding.spec_verify_attn(case.kv, case.q_verify, case.ctx_len, T)
    assert binding.read_status(ws) == 0
    o_out, o_lse, o_stats = oracle.verify_attn(case.kv.cpu(), case.q_verify.cpu(), case.ctx_len.cpu(), 16,
                                               ref_stats.shape[-1])
    for _ in range(2):  # two calls in a row share the built-in scratch
        out, lse, stats = binding.spec_verify_attn_noalloc(case.kv, case.q_verify, case.ctx_len, T)
        assert binding.noalloc_read_status() == 0
        assert (out.cpu().double() - o_out).abs().max().item() <= TOL
        assert (lse.cpu().double() - o_lse).abs().max().item() <= TOL
        for b in range(case.kv.batch):  # entries beyond a sequence's context are not written
            t = int(case.ctx_len[b])
            assert (stats[:, b, :, :t].cpu().double() - o_stats[:, b, :, :t]).abs().max().item() <= TOL
            assert torch.equal(stats[:, b, :, :t], ref_stats[:, b, :, :t])
        assert torch.equal(out, ref_out) and torch.equal(lse, ref_lse)


def test_noalloc_matches_regular_entry_point_twice_in_a_row():
    _compare(inputs.small_config(ctx=(5000, 5000), n_q=9, n_q_heads=32, n_kv_heads=8, planted=50))


def test_noalloc_reuses_the_scratch_for_another_shape():
    _compare(inputs.small_config(ctx=(300, 1100), n_q=7, batch=3, page_size=16, shuffled_pages=True,
                                 planted=0, q_mode="iid", q_std=0.09, n_q_heads=8, n_kv_heads=2))
    _compare(inputs.small_config(ctx=(700, 700), n_q=5, head_dim=64, planted=4))  # head_dim 64


def test_noalloc_refuses_shapes_beyond_the_built_in_scratch():
    cfg = inputs.small_config(ctx=(4096, 4096), n_q=16, n_q_heads=32, n_kv_heads=8, n_layers=24,
                              planted=0, q_mode="iid")
    case = inputs.make_case(cfg, device="cuda")
    need = binding.workspace_bytes(binding.WS_VERIFY, case.kv, cfg.n_q, 4096)
    assert need > binding.noalloc_scratch_bytes()
    before = binding.launch_count()
    with pytest.raises(binding.SpecError) as e:
        binding.spec_verify_attn_noalloc(case.kv, case.q_verify, case.ctx_len, 4096)
    assert e.value.code == -3
    assert binding.launch_count() == before
