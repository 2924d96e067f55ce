"""CPU tests of the page-sharded decode step's host logic (world_size 2, gloo): the orchestration and the index
bookkeeping of paper_2607_24555_b200.dist are run for real, with the oracle standing in for the kernels of a shard,
and the result must be the unsharded oracle's."""
import math
import os
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

SM = 1.0 / math.sqrt(128)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _problem(T=16 * 90 + 5, Hq=4, Hkv=2, seed=3):
    g = np.random.default_rng(seed)
    P = -(-T // 16)
    nb = P + 2
    k = g.standard_normal((nb, Hkv, 16, 128)).astype(np.float32)
    v = g.standard_normal((nb, Hkv, 16, 128)).astype(np.float32)
    bt = g.permutation(nb)[:P].astype(np.int32).reshape(1, P)
    q = (g.standard_normal((1, Hq, 128)) * 0.5).astype(np.float32)
    return k, v, bt, T, q, Hq, Hkv


class OracleShardOps:
    """The kernels of one shard, done by the oracle on numpy arrays (a stand-in for GpuShardOps in CPU tests)."""

    def __init__(self, k, v, bt, T, Hq, Hkv, first, end, has_sink, has_tail, kbud, rank_r=8):
        import oracle
        self.o = oracle
        P = bt.shape[1]
        row = [bt[0, 0] if has_sink else bt[0, first]] + list(bt[0, first:end]) + [bt[0, P - 1] if has_tail else bt[0, first]]
        self.first, self.end, self.has_sink, self.has_tail = first, end, has_sink, has_tail
        self.local_pages = len(row)
        T_loc = (self.local_pages - 1) * 16 + ((T - (P - 1) * 16) if has_tail else 16)
        self.cache = oracle.Cache(k, v, np.array([row], np.int32), np.array([T_loc], np.int32), Hq)
        self.summ = oracle.build_summaries(self.cache, rank_r, oracle.FMT_I4)
        self.k, self.Hq, self.Hkv, self.G, self.r = kbud, Hq, Hkv, Hq // Hkv, rank_r

    def scan(self, q):
        self.shat = self.o.page_logmass(self.cache, q.numpy(), self.r, self.o.FMT_I4, self.summ, SM)
        cand = self.shat[:, :, 1:self.local_pages - 1]
        m = cand.max(-1, keepdims=True)
        return torch.from_numpy((m + np.log(np.exp(cand - m).sum(-1, keepdims=True)))[..., 0])

    def select_scored(self, parts):
        lz = torch.logsumexp(parts.double(), dim=0).numpy()                     # [1, Hq]
        keys = np.full((1, self.Hkv, self.k - 2), np.nan)
        pages = np.full((1, self.Hkv, self.k - 2), -1, np.int64)
        for h in range(self.Hkv):
            s = self.shat[0, h * self.G:(h + 1) * self.G, 1:self.local_pages - 1] - lz[0, h * self.G:(h + 1) * self.G, None]
            m = s.max(0)
            key = m + np.log(np.exp(s - m).sum(0)) - math.log(self.G)
            top = np.sort(np.argsort(-key, kind="stable")[: self.k - 2])
            keys[0, h, :len(top)] = key[top]
            pages[0, h, :len(top)] = top + self.first
        return torch.from_numpy(keys), torch.from_numpy(pages)

    def merge_selection(self, keys, pages):
        R, n, Hkv, kc = keys.shape
        ids = torch.full((n, Hkv, kc), -1, dtype=torch.int64)
        cnt = torch.zeros(n, Hkv, dtype=torch.int32)
        for h in range(Hkv):
            kk = keys[:, 0, h].reshape(-1).numpy()
            pp = pages[:, 0, h].reshape(-1).numpy()
            ok = pp >= 0
            order = np.argsort(-kk[ok], kind="stable")[:kc]
            win = np.sort(pp[ok][order])
            ids[0, h, :len(win)] = torch.from_numpy(win)
            cnt[0, h] = len(win)
        return ids, cnt

    def attend(self, q, ids, cnt):
        from paper_2607_24555_b200.dist import local_attend_table
        table, c = local_attend_table(ids, cnt, self.first, self.end, self.has_sink, self.has_tail, self.local_pages, self.k)
        out, lse = self.o.attend(self.cache, q.numpy(), SM, table.numpy(), c.numpy())
        lse = np.where(c.numpy().repeat(self.G, axis=1) > 0, lse, -np.inf)
        return torch.from_numpy(out), torch.from_numpy(lse)

    def merge_attention(self, outs, lses):
        w = torch.softmax(lses, dim=0)[..., None]
        return (torch.nan_to_num(w) * outs).sum(0)


def _reference(k, v, bt, T, q, Hq, Hkv, kbud):
    import oracle
    cache = oracle.Cache(k, v, bt, np.array([T], np.int32), Hq)
    summ = oracle.build_summaries(cache, 8, oracle.FMT_I4)
    ids, cnt, out, lse = oracle.decode_step(cache, q, 8, oracle.FMT_I4, summ, SM, kbud)
    return ids, cnt, out


def _worker(rank, world, port, queue):
    import torch.distributed as dist
    from paper_2607_24555_b200.dist import shard_pages, sharded_decode_step
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    k, v, bt, T, q, Hq, Hkv = _problem()
    P = bt.shape[1]
    lo, hi = shard_pages(P, world)[rank]
    ops = OracleShardOps(k, v, bt, T, Hq, Hkv, lo, hi, rank == 0, rank == world - 1, kbud=12)
    out, ids, cnt = sharded_decode_step(ops, torch.from_numpy(q))
    queue.put((rank, out.numpy(), ids.numpy(), cnt.numpy()))
    dist.destroy_process_group()


def test_two_rank_gloo_sharded_decode_step_equals_unsharded():
    ctx = mp.get_context("spawn")
    queue = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, queue)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted((queue.get(timeout=180) for _ in procs), key=lambda t: t[0])
    for p in procs:
        p.join(60)
    k, v, bt, T, q, Hq, Hkv = _problem()
    rids, rcnt, rout = _reference(k, v, bt, T, q, Hq, Hkv, 12)
    for rank, out, ids, cnt in res:
        assert np.array_equal(ids[0], rids[0, :, 1:11]) and np.all(cnt == 10)     # the k-2 candidates of the unsharded table
        assert np.abs(out - rout).max() < 1e-9


def test_shard_bookkeeping():
    from paper_2607_24555_b200.dist import shard_pages, local_to_global, local_attend_table
    for P in (3, 10, 101, 4096):
        for world in (1, 2, 3, 8):
            sh = shard_pages(P, world)
            assert sh[0][0] == 1 and sh[-1][1] == P - 1 and all(a[1] == b[0] for a, b in zip(sh, sh[1:]))
            assert max(e - s for s, e in sh) - min(e - s for s, e in sh) <= 1
    assert local_to_global(torch.tensor([1, 5, -1]), 40).tolist() == [40, 44, -1]
    ids = torch.tensor([[[3, 40, 41, 77, -1]]])
    cnt = torch.tensor([[4]], dtype=torch.int32)
    t, c = local_attend_table(ids, cnt, 40, 60, False, False, 22, 6)
    assert t.tolist() == [[[1, 2, -1, -1, -1, -1]]] and c.tolist() == [[2]]
    t, c = local_attend_table(ids, cnt, 1, 40, True, False, 41, 6)
    assert t.tolist() == [[[0, 3, -1, -1, -1, -1]]] and c.tolist() == [[2]]
    t, c = local_attend_table(ids, cnt, 60, 99, False, True, 41, 6)
    assert t.tolist() == [[[18, 40, -1, -1, -1, -1]]] and c.tolist() == [[2]]
    t, c = local_attend_table(ids, torch.tensor([[0]], dtype=torch.int32), 40, 60, False, False, 22, 6)
    assert c.tolist() == [[0]] and t.tolist() == [[[-1] * 6]]
