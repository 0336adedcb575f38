"""Seeded synthetic inputs for the SparseSpec-L attention hot path.

This module only draws random tensors and lays them out; it contains none of the method's
arithmetic (no softmax, no scores, no selection), so both the CUDA path and the CPU oracle
can be fed from it.

Workload recipe (stand-in for the long-context benchmarks the paper evaluates on, whose data
and checkpoints are not needed by the attention path): Llama/Qwen-class GQA attention shapes,
bf16 K/V drawn N(0,1) (or Student-t, nu=3) and a small fraction of "planted heavy hitter"
positions per KV head whose key is a multiple of a per-head query direction, so that the
attention mass concentrates on a recallable subset the way retrieval heads do.

Per (layer, sequence, KV head) a direction ``dvec`` with ``|dvec|^2 = 2*sqrt(D)`` is drawn;
queries are ``dvec + N(0, I)``; a planted key is ``c * dvec (+ N(0, I))``, which puts its
logit near ``2c`` at the softmax scale ``1/sqrt(D)`` against background logits of unit order.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import torch


@dataclasses.dataclass
class KVCache:
    """Dense KV cache of one or more layers, paged: storage ``[L, n_phys_pages, Hkv, page, D]``.

    Strides are in elements.  ``page_table`` maps (sequence, logical page) to a physical page;
    ``None`` means ``phys = b * max_pages + page``.
    """

    k: torch.Tensor
    v: torch.Tensor
    layer_stride: int
    page_stride: int
    head_stride: int
    slot_stride: int
    n_layers: int
    page_size: int
    page_table: Optional[torch.Tensor]
    max_pages: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    sm_scale: float = 0.0
    n_pages: int = 0  # physical pages in the pool (0: batch * max_pages)
    fp8: bool = False  # k, v hold e4m3 bytes (uint8) instead of bf16; strides stay in elements
    k_scale: Optional[torch.Tensor] = None  # fp32 [L, Hkv]: dequantised value = e4m3 value * scale
    v_scale: Optional[torch.Tensor] = None

    def to(self, device) -> "KVCache":
        pt = None if self.page_table is None else self.page_table.to(device)
        ks = None if self.k_scale is None else self.k_scale.to(device)
        vs = None if self.v_scale is None else self.v_scale.to(device)
        return dataclasses.replace(self, k=self.k.to(device), v=self.v.to(device), page_table=pt, k_scale=ks, v_scale=vs)

    def cpu(self) -> "KVCache":
        return self.to("cpu")

    def layer_slice(self, lo: int, hi: int) -> "KVCache":
        """View of layers ``[lo, hi)`` (shares storage)."""
        ks = None if self.k_scale is None else self.k_scale[lo:hi].contiguous()
        vs = None if self.v_scale is None else self.v_scale[lo:hi].contiguous()
        return dataclasses.replace(self, k=self.k[lo:hi], v=self.v[lo:hi], n_layers=hi - lo, k_scale=ks, v_scale=vs)

    def phys_page(self, b: int, page: int) -> int:
        if self.page_table is None:
            return b * self.max_pages + page
        return int(self.page_table[b, page])


@dataclasses.dataclass
class SpecConfig:
    name: str
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ctx: tuple  # (lo, hi) inclusive range the per-sequence context is drawn from, lo == hi: fixed
    n_q: int  # k + 1 verification rows
    k_total: int
    k_sink: int
    k_recent: int
    draft_steps: int
    page_size: int = 0  # 0: one page per sequence (contiguous cache)
    shuffled_pages: bool = False
    planted: float = 0.0  # < 1: fraction of the context, >= 1: count per KV head
    planted_mult: float = 0.0
    planted_noise: bool = False
    kv_dist: str = "normal"  # or "student_t3"
    q_mode: str = "direction"  # or "iid": N(0, q_std^2) with no shared direction
    q_std: float = 1.0
    stat_window: int = 16
    seed: int = 0

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads


def baseline_configs(k3: int = 8) -> dict:
    """The five workloads the build is measured on (``k3`` = speculation length of the third)."""
    return {
        "cfg1_tiny": SpecConfig("cfg1_tiny", 1, 1, 8, 2, 64, (2048, 2048), 5, 256, 4, 64, 4,
                                planted=8, planted_mult=4.0, seed=0),
        "cfg2_8b_32k": SpecConfig("cfg2_8b_32k", 32, 1, 32, 8, 128, (32768, 32768), 9, 2048, 4,
                                  64, 8, planted=0.01, planted_mult=3.0, planted_noise=True,
                                  seed=2),
        "cfg3_8b_128k": SpecConfig("cfg3_8b_128k", 32, 1, 32, 8, 128, (131072, 131072), k3 + 1,
                                   4096, 4, 64, k3, planted=0.005, planted_mult=3.0,
                                   planted_noise=True, seed=3),
        "cfg4_ragged_paged": SpecConfig("cfg4_ragged_paged", 32, 8, 32, 8, 128, (8192, 65536), 7,
                                        1024, 4, 64, 6, page_size=16, shuffled_pages=True,
                                        q_mode="iid", q_std=1.0 / math.sqrt(128.0), seed=4),
        "cfg5_32b_64k": SpecConfig("cfg5_32b_64k", 64, 4, 40, 8, 128, (65536, 65536), 7, 2048, 8,
                                   256, 6, planted=0.01, planted_mult=3.0, planted_noise=True,
                                   kv_dist="student_t3", seed=5),
    }


def _draw_kv(shape, dist, gen, device):
    if dist == "normal":
        return torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    if dist == "student_t3":
        z0 = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
        chi = torch.zeros(shape, device=device, dtype=torch.float32)
        for _ in range(3):
            z = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
            chi.addcmul_(z, z)
        return z0 / torch.sqrt(chi / 3.0)
    raise ValueError(dist)


@dataclasses.dataclass
class SpecCase:
    cfg: SpecConfig
    kv: KVCache
    ctx_len: torch.Tensor  # int32 [B], includes the n_q rows under verification
    q_verify: torch.Tensor  # bf16 [L, B, n_q, Hq, D]
    q_draft: torch.Tensor  # bf16 [steps, L, B, Hq, D]
    planted_pos: Optional[torch.Tensor]  # int64 [L, B, Hkv, n_planted] or None
    direction: Optional[torch.Tensor]  # fp32 [L, B, Hkv, D] or None
    capacity: int  # tokens of storage per sequence (>= max ctx + draft_steps)


def make_case(cfg: SpecConfig, device="cpu", n_layers: Optional[int] = None,
              ctx_override: Optional[list] = None, page_round: int = 128) -> SpecCase:
    """Draw one seeded workload.  ``n_layers`` overrides the config's layer count (layers are
    i.i.d., so a subset of layers is the same distribution); ``ctx_override`` fixes the
    per-sequence context lengths."""
    L = cfg.n_layers if n_layers is None else n_layers
    B, Hq, Hkv, D, G = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.group
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(1000003 * cfg.seed + 17)
    cgen = torch.Generator(device="cpu")
    cgen.manual_seed(7919 * cfg.seed + 3)

    if ctx_override is not None:
        ctx = torch.tensor(ctx_override, dtype=torch.int32)
    elif cfg.ctx[0] == cfg.ctx[1]:
        ctx = torch.full((B,), cfg.ctx[0], dtype=torch.int32)
    else:
        ctx = torch.randint(cfg.ctx[0], cfg.ctx[1] + 1, (B,), generator=cgen, dtype=torch.int32)
    assert ctx.numel() == B
    need = int(ctx.max()) + cfg.draft_steps  # room for the tokens drafted after the verify
    if cfg.page_size > 0:
        ps = cfg.page_size
        max_pages = (need + ps - 1) // ps
    else:
        ps = (need + page_round - 1) // page_round * page_round
        max_pages = 1
    n_phys = B * max_pages
    if cfg.shuffled_pages:
        page_table = torch.randperm(n_phys, generator=cgen).to(torch.int32).reshape(B, max_pages)
    else:
        page_table = None

    shape = (L, n_phys, Hkv, ps, D)
    k = torch.empty(shape, device=dev, dtype=torch.bfloat16)
    v = torch.empty(shape, device=dev, dtype=torch.bfloat16)
    for l in range(L):  # layer by layer: bounds the fp32 scratch at the large shapes
        k[l] = _draw_kv(shape[1:], cfg.kv_dist, gen, dev).to(torch.bfloat16)
        v[l] = _draw_kv(shape[1:], cfg.kv_dist, gen, dev).to(torch.bfloat16)

    direction = None
    planted_pos = None
    if cfg.q_mode == "direction":
        g = torch.randn((L, B, Hkv, D), generator=gen, device=dev, dtype=torch.float32)
        direction = g / g.norm(dim=-1, keepdim=True) * math.sqrt(2.0 * math.sqrt(D))
        dq = direction.repeat_interleave(G, dim=2)  # [L, B, Hq, D]: q heads h*G..h*G+G-1 share
        q_verify = dq[:, :, None] + torch.randn((L, B, cfg.n_q, Hq, D), generator=gen,
                                                device=dev, dtype=torch.float32)
        q_draft = dq[None] + torch.randn((cfg.draft_steps, L, B, Hq, D), generator=gen,
                                         device=dev, dtype=torch.float32)
    else:
        q_verify = cfg.q_std * torch.randn((L, B, cfg.n_q, Hq, D), generator=gen, device=dev,
                                           dtype=torch.float32)
        q_draft = cfg.q_std * torch.randn((cfg.draft_steps, L, B, Hq, D), generator=gen,
                                          device=dev, dtype=torch.float32)

    if cfg.planted > 0:
        assert cfg.q_mode == "direction"
        tmin = int(ctx.min())
        n_pl = int(cfg.planted) if cfg.planted >= 1 else max(1, int(round(cfg.planted * tmin)))
        ptab = page_table.to(dev) if page_table is not None else None
        planted_pos = torch.empty((L, B, Hkv, n_pl), dtype=torch.int64, device=dev)
        for l in range(L):
            for b in range(B):
                T = int(ctx[b])
                r = torch.rand((Hkv, T), generator=gen, device=dev)
                pos = r.topk(n_pl, dim=-1).indices.sort(dim=-1).values  # uniform subset of [0, T)
                planted_pos[l, b] = pos
                key = cfg.planted_mult * direction[l, b][:, None, :].expand(Hkv, n_pl, D)
                if cfg.planted_noise:
                    key = key + torch.randn((Hkv, n_pl, D), generator=gen, device=dev,
                                            dtype=torch.float32)
                page = pos // ps
                slot = pos % ps
                phys = (b * max_pages + page) if ptab is None else ptab[b][page].long()
                hh = torch.arange(Hkv, device=dev)[:, None].expand(Hkv, n_pl)
                k[l, phys, hh, slot] = key.to(torch.bfloat16)

    kv = KVCache(
        k=k, v=v, layer_stride=n_phys * Hkv * ps * D, page_stride=Hkv * ps * D,
        head_stride=ps * D, slot_stride=D, n_layers=L, page_size=ps,
        page_table=None if page_table is None else page_table.to(dev), max_pages=max_pages,
        batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, sm_scale=0.0, n_pages=n_phys,
    )
    return SpecCase(cfg=cfg, kv=kv, ctx_len=ctx.to(dev), q_verify=q_verify.to(torch.bfloat16),
                    q_draft=q_draft.to(torch.bfloat16), planted_pos=planted_pos,
                    direction=direction, capacity=ps * max_pages)


def resample_planted(case: SpecCase, prob: float, step: int) -> int:
    """Move each planted heavy-hitter position with probability ``prob`` (third workload: the
    important set drifts between speculation rounds, so the index must be rebuilt from the fresh
    statistic).  The old row gets a fresh background key, the new position (uniform in the
    context, not planted already) gets ``planted_mult`` x the head's direction (+ noise).
    Updates ``case.kv.k`` and ``case.planted_pos`` in place; returns how many positions moved.
    Seeded by (config seed, step)."""
    cfg = case.cfg
    assert case.planted_pos is not None and case.direction is not None
    dev = case.kv.k.device
    gen = torch.Generator(device=dev)
    gen.manual_seed(7368787 * cfg.seed + 104729 * step + 5)
    L, B, Hkv, n_pl = case.planted_pos.shape
    D, ps = cfg.head_dim, case.kv.page_size
    ptab = case.kv.page_table
    moved_total = 0
    for l in range(L):
        for b in range(B):
            T = int(case.ctx_len[b])
            pos = case.planted_pos[l, b]  # [Hkv, n_pl]
            move = torch.rand((Hkv, n_pl), generator=gen, device=dev) < prob
            cand = torch.randint(0, T, (Hkv, n_pl), generator=gen, device=dev)
            taken = torch.zeros((Hkv, T), dtype=torch.bool, device=dev)
            taken.scatter_(1, pos, True)
            move &= ~taken.gather(1, cand)  # a candidate that is planted already: stay
            # two moves of one head to the same candidate: keep the first
            order = torch.where(move, cand, torch.full_like(cand, T)).sort(dim=1)
            dup = torch.zeros_like(move)
            dup.scatter_(1, order.indices[:, 1:], (order.values[:, 1:] == order.values[:, :-1]) &
                         (order.values[:, 1:] < T))
            move &= ~dup
            hh = torch.arange(Hkv, device=dev)[:, None].expand(Hkv, n_pl)

            def rows(p):
                page, slot = p // ps, p % ps
                phys = (b * case.kv.max_pages + page) if ptab is None else ptab[b][page].long()
                return phys, slot

            old_phys, old_slot = rows(pos[move])
            fresh = _draw_kv((int(move.sum()), D), cfg.kv_dist, gen, dev).to(torch.bfloat16)
            kview = case.kv.k.view(L, case.kv.n_pages, Hkv, ps, D)
            kview[l, old_phys, hh[move], old_slot] = fresh
            key = cfg.planted_mult * case.direction[l, b][:, None, :].expand(Hkv, n_pl, D)[move]
            if cfg.planted_noise:
                key = key + torch.randn(key.shape, generator=gen, device=dev, dtype=torch.float32)
            new_phys, new_slot = rows(cand[move])
            kview[l, new_phys, hh[move], new_slot] = key.to(torch.bfloat16)
            pos[move] = cand[move]
            case.planted_pos[l, b] = pos.sort(dim=1).values
            moved_total += int(move.sum())
    return moved_total


def small_config(name="small", **kw) -> SpecConfig:
    """A config sized for element-by-element parity against the oracle; fields overridable."""
    base = dict(name=name, n_layers=1, batch=1, n_q_heads=8, n_kv_heads=2, head_dim=128,
                ctx=(600, 600), n_q=5, k_total=128, k_sink=4, k_recent=16, draft_steps=2,
                planted=6, planted_mult=3.0, planted_noise=True, seed=11)
    base.update(kw)
    return SpecConfig(**base)


def make_logits(rows: int, vocab: int, dtype=torch.bfloat16, seed: int = 0, device="cpu",
                row_stride: Optional[int] = None, offset: int = 0) -> torch.Tensor:
    """Seeded draft-model logits ``[rows, vocab]`` for the speculation-length controller: a
    Gaussian background whose spread differs per row (confident rows to near-uniform rows) plus
    a few boosted tokens per row, the shape of a language model's next-token logits.  Holds no
    arithmetic of the method.  ``row_stride`` > vocab leaves padding between rows and ``offset``
    shifts the first element (to exercise strided and unaligned rows)."""
    gen = torch.Generator().manual_seed(7000 + seed)
    stride = row_stride or vocab
    buf = torch.zeros(rows * stride + offset + 8, dtype=torch.float32)
    view = buf[offset:offset + rows * stride].view(rows, stride)[:, :vocab]
    spread = torch.empty(rows).uniform_(0.2, 4.0, generator=gen)
    view.copy_(torch.randn(rows, vocab, generator=gen) * spread[:, None])
    n_boost = min(4, vocab)
    cols = torch.randint(0, vocab, (rows, n_boost), generator=gen)
    boost = torch.empty(rows, n_boost).uniform_(0.0, 14.0, generator=gen)
    view.scatter_add_(1, cols, boost)
    buf = buf.to(dtype).to(device)
    return buf[offset:offset + rows * stride].view(rows, stride)[:, :vocab]


def quantize_kv_fp8(kv: KVCache) -> KVCache:
    """An 8-bit copy of a bf16 cache: e4m3 bytes (same layout, strides in elements) and a power-of-two
    scale per (layer, KV head) chosen so that the head's largest magnitude lands below 448, the e4m3
    maximum.  Only a cast and a scale: no attention arithmetic."""
    L, Hkv = kv.n_layers, kv.n_kv_heads

    def one(x):
        amax = x.float().abs().amax(dim=(1, 3, 4)).clamp(min=1e-30)            # [L, Hkv] over pages, slots, d
        scale = torch.exp2(torch.ceil(torch.log2(amax / 448.0))).float()
        q = (x.float() / scale.view(L, 1, Hkv, 1, 1)).to(torch.float8_e4m3fn).view(torch.uint8)
        return q.contiguous(), scale.contiguous()

    k8, ks = one(kv.k)
    v8, vs = one(kv.v)
    return dataclasses.replace(kv, k=k8, v=v8, fp8=True, k_scale=ks, v_scale=vs)


def dequantize_kv_fp8(kv: KVCache) -> KVCache:
    """The bf16 cache whose values are exactly the dequantised ones (an e4m3 value times a power of two has
    four significant bits: representable in bf16 without rounding)."""
    L, Hkv = kv.n_layers, kv.n_kv_heads
    k = (kv.k.view(torch.float8_e4m3fn).float() * kv.k_scale.view(L, 1, Hkv, 1, 1)).to(torch.bfloat16)
    v = (kv.v.view(torch.float8_e4m3fn).float() * kv.v_scale.view(L, 1, Hkv, 1, 1)).to(torch.bfloat16)
    return dataclasses.replace(kv, k=k, v=v, fp8=False, k_scale=None, v_scale=None)

