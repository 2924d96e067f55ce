"""Seeded synthetic decode-step inputs shaped like the paper's workloads.

This module only draws random tensors and lays them out as a paged KV cache.  It holds none of the
method's arithmetic (no summaries, scores, selection or attention) and imports neither the CUDA
binding nor the CPU oracle, so both sides can be fed the very same stored values: tensors are
generated once (on whichever torch device is asked for) and handed to each side by copy.

Key structure ("locally low-rank, globally high-rank", Sec. 2 / Table 1 of the paper): the keys of
a page are a page mean plus a few page-specific random directions with large coefficients plus
small isotropic noise; optional per-KV-head global offset; optional "carrier" tokens aligned with
one query head of the group (cosine 0.9, norm 4x the median key norm), the synthetic stand-in for
the answer-bearing tokens the paper's microscope tracks.  Values are N(0,1).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import List, Optional

import torch


@dataclass
class Workload:
    name: str
    seq_lens: List[int]                 # tokens per request, including the one being decoded
    Hq: int = 32
    Hkv: int = 8
    d: int = 128
    B: int = 16
    dtype: str = "bf16"                 # "bf16" | "f32" for K, V and q
    rank: int = 8
    fmt: str = "i4"                     # summary format "i4" | "f32"
    budget: int = 2048                  # tokens per KV head
    n_dirs: int = 6                     # page-specific directions per page (0 = isotropic filler)
    dir_std: float = 3.0
    noise_std: float = 0.1
    offset_std: float = 2.0             # per-KV-head global key offset
    carriers: int = 0                   # carrier tokens per request
    q_scale: float = 1.0
    seed: int = 0
    permute_blocks: bool = True         # physical blocks assigned by a seeded permutation
    layout: str = "HND"                 # [block, head, token, dim] | "NHD" [block, token, head, dim]
    spare_blocks: int = 0
    tail_fill: float = 0.0              # value written to cache slots at or beyond seq_len

    @property
    def n(self) -> int:
        return len(self.seq_lens)

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def k(self) -> int:
        return -(-self.budget // self.B)

    @property
    def max_pages(self) -> int:
        return max(-(-t // self.B) for t in self.seq_lens)

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


def config0(seed: int = 0) -> Workload:
    """Tiny fp32 case: 1 request, 1 KV head x 4 query heads, 4096 tokens, 8 carriers."""
    return Workload("cfg0_tiny", [4096], Hq=4, Hkv=1, dtype="f32", rank=8, fmt="f32", budget=256,
                    n_dirs=4, offset_std=0.0, carriers=8, seed=seed)


def config1(n: int = 8, T: int = 32768, seed: int = 1) -> Workload:
    """Llama-3.1-8B attention shapes: 32 q heads / 8 KV heads, batch 8 x 32K, r8i4, b=2048."""
    return Workload("cfg1_llama_8x32k", [T] * n, Hq=32, Hkv=8, seed=seed)


def config2(n: int = 32, T: int = 16384, rank: int = 8, budget: int = 1024, seed: int = 2) -> Workload:
    """Qwen3-4B shapes: batch 32 x 16K, isotropic N(0,1) filler, 64 carriers per sequence."""
    return Workload(f"cfg2_qwen_{n}x{T // 1024}k_r{rank}_b{budget}", [T] * n, Hq=32, Hkv=8, rank=rank,
                    budget=budget, n_dirs=0, offset_std=0.0, carriers=64, seed=seed)


def config3(T: int = 1 << 20, Hkv: int = 2, seed: int = 3) -> Workload:
    """GLM-4-9B long-context shapes: 32 q heads / 2 KV heads, one request of 128K..1M tokens."""
    return Workload(f"cfg3_glm_1x{T // 1024}k_hkv{Hkv}", [T], Hq=32, Hkv=Hkv, seed=seed)


def config4(batch: int = 8, seed: int = 4, lo: int = 65536, hi: int = 131072) -> Workload:
    """Batched serving sweep, Llama shapes, context lengths uniform in [lo, hi]."""
    g = torch.Generator().manual_seed(1000 + seed)
    lens = torch.randint(lo, hi + 1, (batch,), generator=g).tolist()
    return Workload(f"cfg4_llama_b{batch}", lens, Hq=32, Hkv=8, seed=seed)


@dataclass
class Case:
    w: Workload
    k: torch.Tensor            # paged keys   (layout per w.layout)
    v: torch.Tensor            # paged values
    q: torch.Tensor            # [n, Hq, d]
    block_table: torch.Tensor  # [n, max_pages] int32
    seq_lens: torch.Tensor     # [n] int32
    num_blocks: int
    carrier_pages: List[List[int]] = field(default_factory=list)  # logical page of each carrier

    @property
    def strides(self):
        """(stride_block, stride_head, stride_token) in elements."""
        w = self.w
        if w.layout == "HND":
            return (w.Hkv * w.B * w.d, w.B * w.d, w.d)
        return (w.B * w.Hkv * w.d, w.d, w.Hkv * w.d)


def _tdtype(name: str):
    return torch.bfloat16 if name == "bf16" else torch.float32


def _page_keys(w: Workload, P: int, gen: torch.Generator, dev, offset: Optional[torch.Tensor],
               chunk: int = 4096):
    """Keys of P pages, [P, Hkv, B, d] fp32, generated in page chunks to bound memory."""
    out = torch.empty(P, w.Hkv, w.B, w.d, device=dev, dtype=torch.float32)
    for p0 in range(0, P, chunk):
        p1 = min(P, p0 + chunk)
        m = p1 - p0
        if w.n_dirs > 0:
            mu = torch.randn(m, w.Hkv, 1, w.d, generator=gen, device=dev)
            dirs = torch.randn(m, w.Hkv, w.n_dirs, w.d, generator=gen, device=dev)
            dirs = dirs / dirs.norm(dim=-1, keepdim=True)
            a = torch.randn(m, w.Hkv, w.B, w.n_dirs, generator=gen, device=dev) * w.dir_std
            kk = mu + torch.matmul(a, dirs)
            kk += torch.randn(m, w.Hkv, w.B, w.d, generator=gen, device=dev) * w.noise_std
        else:
            kk = torch.randn(m, w.Hkv, w.B, w.d, generator=gen, device=dev)
        if offset is not None:
            kk += offset[None, :, None, :]
        out[p0:p1] = kk
    return out


def make_case(w: Workload, device="cpu") -> Case:
    dev = torch.device(device)
    gen = torch.Generator(device=dev).manual_seed(w.seed)
    cpu_gen = torch.Generator().manual_seed(w.seed + 7919)
    dt = _tdtype(w.dtype)
    pages = [-(-t // w.B) for t in w.seq_lens]
    num_blocks = sum(pages) + w.spare_blocks
    max_pages = max(pages)
    perm = torch.randperm(num_blocks, generator=cpu_gen) if w.permute_blocks else torch.arange(num_blocks)
    block_table = torch.zeros(w.n, max_pages, dtype=torch.int32)
    q = (torch.randn(w.n, w.Hq, w.d, generator=gen, device=dev) * w.q_scale).to(dt)
    offset = (torch.randn(w.Hkv, w.d, generator=gen, device=dev) * w.offset_std) if w.offset_std > 0 else None
    shape = (num_blocks, w.Hkv, w.B, w.d) if w.layout == "HND" else (num_blocks, w.B, w.Hkv, w.d)
    kc = torch.zeros(shape, device=dev, dtype=dt)
    vc = torch.zeros(shape, device=dev, dtype=dt)
    carrier_pages: List[List[int]] = []
    start = 0
    for b, (T, P) in enumerate(zip(w.seq_lens, pages)):
        ids = perm[start:start + P]
        start += P
        block_table[b, :P] = ids.to(torch.int32)
        kk = _page_keys(w, P, gen, dev, offset)                       # [P, Hkv, B, d]
        vv = torch.randn(P, w.Hkv, w.B, w.d, generator=gen, device=dev)
        cps: List[int] = []
        if w.carriers > 0 and P > 2:
            kappa = kk.norm(dim=-1).permute(1, 0, 2).reshape(w.Hkv, -1).median(dim=1).values   # [Hkv]
            qf = q[b].float().view(w.Hkv, w.G, w.d)
            # carriers sit on complete candidate pages (1 .. P-2), the same positions in every KV head
            cand = torch.randperm(P - 2, generator=cpu_gen)[: w.carriers] + 1
            if cand.numel() < w.carriers:
                extra = torch.randint(1, P - 1, (w.carriers - cand.numel(),), generator=cpu_gen)
                cand = torch.cat([cand, extra])
            slots = torch.randint(0, w.B, (w.carriers,), generator=cpu_gen)
            for c in range(w.carriers):
                g = c % w.G
                qh = qf[:, g, :] / qf[:, g, :].norm(dim=-1, keepdim=True)       # [Hkv, d]
                rnd = torch.randn(w.Hkv, w.d, generator=gen, device=dev)
                rnd = rnd - (rnd * qh).sum(-1, keepdim=True) * qh
                rnd = rnd / rnd.norm(dim=-1, keepdim=True)
                key = 4.0 * kappa[:, None] * (0.9 * qh + math.sqrt(0.19) * rnd)
                kk[int(cand[c]), :, int(slots[c]), :] = key
                cps.append(int(cand[c]))
        carrier_pages.append(cps)
        # slots at or beyond the sequence length hold a fill value nobody may read as data
        tail = P * w.B - T
        if tail > 0:
            kk[P - 1, :, w.B - tail:, :] = w.tail_fill
            vv[P - 1, :, w.B - tail:, :] = w.tail_fill
        idd = ids.to(dev)
        if w.layout == "HND":
            kc[idd] = kk.to(dt)
            vc[idd] = vv.to(dt)
        else:
            kc[idd] = kk.permute(0, 2, 1, 3).to(dt)
            vc[idd] = vv.permute(0, 2, 1, 3).to(dt)
        del kk, vv
    return Case(w, kc, vc, q, block_table.to(dev), torch.tensor(w.seq_lens, dtype=torch.int32, device=dev),
                num_blocks, carrier_pages)


def new_token(w: Workload, step: int, device="cpu"):
    """k_new, v_new [n, Hkv, d] for decode step `step` (seeded, independent of the cache)."""
    dev = torch.device(device)
    gen = torch.Generator(device=dev).manual_seed(w.seed * 100003 + 17 + step)
    dt = _tdtype(w.dtype)
    kn = torch.randn(w.n, w.Hkv, w.d, generator=gen, device=dev) * 2.0
    vn = torch.randn(w.n, w.Hkv, w.d, generator=gen, device=dev)
    qn = torch.randn(w.n, w.Hq, w.d, generator=gen, device=dev) * w.q_scale
    return kn.to(dt), vn.to(dt), qn.to(dt)
