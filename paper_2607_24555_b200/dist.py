"""Host-side plumbing for running the decode path on several GPUs.

The path shards with no exchange: every (request, KV head) problem owns its pages, summaries,
selection and output heads, so each rank simply runs its own slice of the batch (weak scaling
when every rank gets a full batch).  The only collective is the timing reduction of the benchmark
(max over ranks), done with torch.distributed on whichever backend the job was launched with.
"""
from __future__ import annotations

import os
from typing import List, Tuple

import torch
import torch.distributed as dist


def env_rank_world() -> Tuple[int, int, int]:
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def shard_requests(n_requests: int, rank: int, world: int) -> List[int]:
    """Contiguous, balanced split of request indices; the first (n % world) ranks get one more."""
    base, extra = divmod(n_requests, world)
    lo = rank * base + min(rank, extra)
    hi = lo + base + (1 if rank < extra else 0)
    return list(range(lo, hi))


def max_over_ranks(value: float, device="cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device="cpu") -> float:
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def barrier():
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


# ---------------------------------------------------------------------------------------------------------------
# Page-sharded decode of ONE long request: its pages are dealt to the ranks in page order; a step needs three small
# exchanges (per-head log Z, each shard's top-(k-2) candidates, each shard's attention partial).  Everything here
# is index bookkeeping and collectives; the arithmetic runs in the library's kernels behind `ops`.
# ---------------------------------------------------------------------------------------------------------------

def shard_pages(num_pages: int, world: int) -> List[Tuple[int, int]]:
    """Candidate pages 1 .. P-2 of a request of P pages, dealt to `world` shards in page order (contiguous,
    balanced): [(first, end)] global logical pages per shard, end exclusive."""
    ncand = max(num_pages - 2, 0)
    base, extra = divmod(ncand, world)
    out, lo = [], 1
    for r in range(world):
        n = base + (1 if r < extra else 0)
        out.append((lo, lo + n))
        lo += n
    return out


def local_to_global(local_ids: torch.Tensor, first_page: int) -> torch.Tensor:
    """A shard presents itself as [sink or dummy] + its candidate pages + [last page or dummy]: local candidate page
    i (1-based) is global page first_page + i - 1.  -1 stays -1."""
    return torch.where(local_ids >= 0, local_ids - 1 + first_page, local_ids)


def local_attend_table(global_ids: torch.Tensor, counts: torch.Tensor, first_page: int, end_page: int, has_sink: bool,
                       has_tail: bool, local_pages: int, k: int):
    """The shard's page table for attention from the global selection: the selected pages it owns (as local ids),
    plus local page 0 if it holds the request's sink page and its last page if it holds the request's tail.
    global_ids [n, Hkv, kc] ascending, -1 padded -> (table [n, Hkv, k] ascending / -1 padded, count [n, Hkv])."""
    n, Hkv, kc = global_ids.shape
    valid = torch.arange(kc, device=global_ids.device)[None, None, :] < counts[..., None]
    own = valid & (global_ids >= first_page) & (global_ids < end_page)
    big = local_pages + 1                                   # sorts after every real id
    loc = torch.where(own, global_ids - first_page + 1, torch.full_like(global_ids, big))
    cols = [loc]
    if has_sink:
        cols.insert(0, torch.zeros(n, Hkv, 1, dtype=global_ids.dtype, device=global_ids.device))
    if has_tail:
        cols.append(torch.full((n, Hkv, 1), local_pages - 1, dtype=global_ids.dtype, device=global_ids.device))
    allc = torch.cat(cols, dim=-1).sort(dim=-1).values
    cnt = (allc < big).sum(dim=-1).to(torch.int32)
    table = torch.where(allc < big, allc, torch.full_like(allc, -1))
    if table.shape[-1] < k:
        pad = torch.full((n, Hkv, k - table.shape[-1]), -1, dtype=table.dtype, device=table.device)
        table = torch.cat([table, pad], dim=-1)
    return table[..., :k].contiguous().to(torch.int32), cnt.contiguous()


def _all_gather(t: torch.Tensor, group=None) -> torch.Tensor:
    """[...] -> [world, ...] in rank order."""
    if not (dist.is_available() and dist.is_initialized()):
        return t[None].clone()
    parts = [torch.empty_like(t) for _ in range(dist.get_world_size(group))]
    dist.all_gather(parts, t.contiguous(), group=group)
    return torch.stack(parts)


def sharded_decode_step(ops, q, group=None):
    """One decode step of a page-sharded request on this rank.  `ops` runs the shard's kernels:
         ops.scan(q) -> head_logz [n, Hq]
         ops.select_scored(logz_parts [R, n, Hq]) -> (cand_key [n, Hkv, k-2], cand_page [n, Hkv, k-2] GLOBAL pages, -1 pad)
         ops.merge_selection(keys [R, ...], pages [R, ...]) -> (global_ids [n, Hkv, k-2], count [n, Hkv])
         ops.attend(q, global_ids, count) -> (out [n, Hq, d], lse [n, Hq])
         ops.merge_attention(outs [R, ...], lses [R, ...]) -> out [n, Hq, d]
       Returns (out, global_ids, count); every rank ends with the same three."""
    parts = _all_gather(ops.scan(q), group)
    ck, cp = ops.select_scored(parts)
    ids, cnt = ops.merge_selection(_all_gather(ck, group), _all_gather(cp, group))
    o, l = ops.attend(q, ids, cnt)
    return ops.merge_attention(_all_gather(o, group), _all_gather(l, group)), ids, cnt


def emulate_sharded_decode_step(ops_list, q):
    """The same step with every shard in ONE process (one GPU holds all shards, or a CPU test): the phases run in
    lock-step over the shards and a gather is a stack.  No kernel waits for another."""
    parts = torch.stack([o.scan(q) for o in ops_list])
    cands = [o.select_scored(parts) for o in ops_list]
    K, Pg = torch.stack([c[0] for c in cands]), torch.stack([c[1] for c in cands])
    sel = [o.merge_selection(K, Pg) for o in ops_list]
    att = [o.attend(q, ids, cnt) for o, (ids, cnt) in zip(ops_list, sel)]
    O, Ls = torch.stack([a[0] for a in att]), torch.stack([a[1] for a in att])
    return [o.merge_attention(O, Ls) for o in ops_list], sel


class GpuShardOps:
    """A shard of one request on this GPU, driven through the C ABI.  The shard's cache holds, as an ordinary paged
    sequence, [sink or dummy page] + its candidate pages + [the request's last page or a dummy page]."""

    def __init__(self, ctx, kv, summaries, first_page: int, end_page: int, has_sink: bool, has_tail: bool):
        self.ctx, self.kv, self.summ = ctx, kv, summaries
        self.first, self.end, self.has_sink, self.has_tail = first_page, end_page, has_sink, has_tail
        self.n = int(kv.seq_lens.shape[0])
        cfg = ctx.cfg
        self.Hq, self.Hkv, self.k, self.d = cfg.num_q_heads, cfg.num_kv_heads, ctx.k, cfg.head_dim
        self.local_pages = 1 + (end_page - first_page) + 1
        self.dev = kv.seq_lens.device
        self.key = torch.empty(self.n, self.Hkv, cfg.max_pages_per_seq, dtype=torch.float32, device=self.dev)

    def scan(self, q):
        lz = torch.empty(self.n, self.Hq, dtype=torch.float32, device=self.dev)
        self.ctx.locks_scan(q, self.summ, self.kv, self.n, lz)
        return lz

    def select_scored(self, logz_parts):
        ids = torch.empty(self.n, self.Hkv, self.k, dtype=torch.int32, device=self.dev)
        cnt = torch.empty(self.n, self.Hkv, dtype=torch.int32, device=self.dev)
        self.ctx.locks_select_scored(logz_parts.contiguous(), self.kv, self.n, ids, cnt, page_logshare=self.key)
        if int(cnt.min()) < self.k:
            raise ValueError("a shard needs more pages than the page budget k")
        win = ids[..., 1:self.k - 1].to(torch.int64)                       # the shard's k-2 winners, local ids
        keys = torch.gather(self.key, 2, win)
        return keys.contiguous(), local_to_global(win, self.first).to(torch.int32).contiguous()

    def merge_selection(self, keys, pages):
        ids = torch.empty(self.n, self.Hkv, self.k - 2, dtype=torch.int32, device=self.dev)
        cnt = torch.empty(self.n, self.Hkv, dtype=torch.int32, device=self.dev)
        self.ctx.locks_merge_selection(keys.contiguous(), pages.contiguous(), self.n, ids, cnt)
        return ids, cnt

    def attend(self, q, global_ids, count):
        table, cnt = local_attend_table(global_ids, count, self.first, self.end, self.has_sink, self.has_tail,
                                        self.local_pages, self.k)
        out = torch.empty(self.n, self.Hq, self.d, dtype=q.dtype, device=self.dev)
        lse = torch.empty(self.n, self.Hq, dtype=torch.float32, device=self.dev)
        self.ctx.locks_sparse_attend(q, self.kv, self.n, table, cnt, out, lse)
        return out, lse

    def merge_attention(self, outs, lses):
        out = torch.empty(self.n, self.Hq, self.d, dtype=outs.dtype, device=self.dev)
        self.ctx.locks_merge_attention(outs.contiguous(), lses.contiguous(), self.n, out)
        return out
