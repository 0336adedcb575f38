"""Host-side planning (no GPU): how the library would split the five baseline workloads.  The planner
is pure host arithmetic on the cache description and the SM count (148 assumed without a device), so
its invariants are checked here: every CTA fits one wave, a CTA's share of a head fits the
tensor-memory cache, shares cover the key list, and the shapes the score-cache kernel cannot take
fall back as documented."""
import pytest

from paper_2607_27735_b200 import binding

NSM = 148


def kv_struct(n_layers, batch, hq, hkv, d, max_ctx, page=None):
    page_size = page or max_ctx
    max_pages = (max_ctx + page_size - 1) // page_size
    return binding._KV(1 << 20, 1 << 21, batch * max_pages * hkv * page_size * d, hkv * page_size * d, page_size * d, d,
                       n_layers, page_size, None, max_pages, batch, hq, hkv, d, batch * max_pages, 0.0, 0, None, None)


VERIFY_CASES = [  # (name, kv, n_q, ctx, expected kernel)
    ("cfg1", kv_struct(1, 1, 8, 2, 64, 2048), 5, 2048, 2),            # head_dim 64: lower half of each tile
    ("cfg2", kv_struct(1, 1, 32, 8, 128, 32768 + 128), 9, 32768, 2),
    ("cfg3_k1", kv_struct(1, 1, 32, 8, 128, 131072 + 128), 2, 131072, 2),
    ("cfg3_k8", kv_struct(1, 1, 32, 8, 128, 131072 + 128), 9, 131072, 2),
    ("cfg3_k16", kv_struct(1, 1, 32, 8, 128, 131072 + 128), 17, 131072, 3),  # rows in two passes
    ("cfg4", kv_struct(1, 8, 32, 8, 128, 65536 + 16, page=16), 7, 65536, 2),
    ("cfg5", kv_struct(1, 4, 40, 8, 128, 65536 + 128), 7, 65536, 2),
]


@pytest.mark.parametrize("name,kv,n_q,ctx,kernel", VERIFY_CASES)
def test_verify_plan(name, kv, n_q, ctx, kernel):
    kind, hg, cph, units, n, n_cache, slots, p_bufs = binding.describe_plan(binding.WS_VERIFY, kv, n_q, ctx)
    assert kind == kernel, name
    if kind == 0:
        return
    G = kv.n_q_heads // kv.n_kv_heads
    rows = (n_q + 1) // 2 if kind == 3 else n_q
    assert n % 16 == 0 and n >= rows * G and n - rows * G < 16
    assert kv.n_kv_heads % hg == 0 and hg * cph <= NSM          # one CTA per SM, all co-resident
    assert units == kv.n_layers * kv.batch * (kv.n_kv_heads // hg)
    assert 2 * n + n_cache * n <= 512                            # accumulator + cached score tiles in 512 columns
    tiles = (ctx + 127) // 128
    assert (tiles + cph - 1) // cph <= n_cache                   # a CTA's share of a head fits the cache
    assert slots >= 3 and 1 <= p_bufs <= 4


def test_headline_shape_is_two_units_of_four_heads():
    kv = kv_struct(1, 1, 32, 8, 128, 32768 + 128)
    assert binding.describe_plan(binding.WS_VERIFY, kv, 9, 32768)[:6] == [2, 4, 37, 2, 48, 8]


def test_8bit_cache_plans():
    """The score-cache kernel takes an 8-bit cache at head_dim 128 with three operand slots (its raw stages
    hold the tiles in flight) and as many P buffers as fit; head_dim 64 is not read directly (the entry
    point expands it to bf16 first), so the planner reports no tensor-core kernel for that view."""
    def fp8(kv):
        return binding._KV(kv.k, kv.v, kv.layer_stride, kv.page_stride, kv.head_stride, kv.slot_stride, kv.n_layers,
                           kv.page_size, None, kv.max_pages, kv.batch, kv.n_q_heads, kv.n_kv_heads, kv.head_dim,
                           kv.n_pages, 0.0, binding.KV_FP8_E4M3, None, None)
    kind, hg, cph, units, n, n_cache, slots, p_bufs = binding.describe_plan(
        binding.WS_VERIFY, fp8(kv_struct(1, 1, 32, 8, 128, 32768 + 128)), 9, 32768)
    assert [kind, hg, cph, units, n, n_cache] == [2, 4, 37, 2, 48, 8] and slots == 3 and p_bufs == 3
    # raw stages (2 x 16 KB), Q, P buffers, slots and the small arrays fit the 227 KB of a CTA
    assert 1024 + n * 256 + p_bufs * 2 * n * 256 + 12544 + 2 * 16384 + slots * 32768 <= 227 * 1024
    assert binding.describe_plan(binding.WS_VERIFY, fp8(kv_struct(1, 1, 8, 2, 64, 2048)), 5, 2048)[0] == 0


DRAFT_CASES = [  # (name, kv, keys)
    ("cfg2 per layer", kv_struct(1, 1, 32, 8, 128, 32768 + 128), 2056),
    ("cfg2 folded", kv_struct(32, 1, 32, 8, 128, 32768 + 128), 2056),
    ("cfg3 per layer", kv_struct(1, 1, 32, 8, 128, 131072 + 128), 4104),
    ("cfg4", kv_struct(1, 8, 32, 8, 128, 65536 + 16, page=16), 1030),
    ("cfg5", kv_struct(1, 4, 40, 8, 128, 65536 + 128), 2054),
    ("tiny", kv_struct(1, 1, 8, 2, 64, 2048), 260),
    ("one key", kv_struct(1, 1, 8, 8, 128, 2048), 1),
]


@pytest.mark.parametrize("name,kv,keys", DRAFT_CASES)
def test_draft_plan(name, kv, keys):
    cs, per, nw, st = binding.describe_plan(binding.WS_DRAFT, kv, k_total=keys)[:4]
    G = kv.n_q_heads // kv.n_kv_heads
    assert 1 <= cs <= 8 and per % 16 == 0 and cs * per >= keys   # the shares cover the key list
    assert (nw, st) in {(4, 2), (4, 3), (8, 1), (8, 2), (8, 3), (12, 2)}
    stage = 2 * 16 * (kv.head_dim * 2 + 16)
    smem = nw * st * stage + per * 4 + nw * 64 + 16 + cs * G * (kv.head_dim + 2) * 4
    assert smem <= 227 * 1024
    probs = kv.n_layers * kv.batch * kv.n_kv_heads
    if probs * 8 <= NSM:  # few problems: the CTAs of three consecutive calls fit the GPU together
        assert nw in (8, 12) and probs * cs <= NSM


def test_headline_draft_call_uses_clusters_of_six():
    kv = kv_struct(1, 1, 32, 8, 128, 32768 + 128)
    assert binding.describe_plan(binding.WS_DRAFT, kv, k_total=2056)[:4] == [6, 352, 8, 3]


def test_describe_plan_rejects_bad_arguments():
    kv = kv_struct(1, 1, 32, 8, 128, 4096)
    with pytest.raises(binding.SpecError):
        binding.describe_plan(binding.WS_VERIFY, kv, 0, 4096)
    with pytest.raises(binding.SpecError):
        binding.describe_plan(binding.WS_SELECT, kv, 1, 4096)
