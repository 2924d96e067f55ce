"""Helpers for the GPU parity tests: run the CUDA path through the C-ABI binding on a synthetic
case and hand the same stored values to the oracle."""
from __future__ import annotations

import math

import numpy as np
import torch

import locks_synth
import oracle
import paper_2607_24555_b200 as locks
from paper_2607_24555_b200.binding import KVView, make_config
from common import fmt_code, oracle_cache, t2np

oracle.set_threads(oracle.max_threads())   # the oracle is only a checker here: use every host core


class GpuCase:
    def __init__(self, w: locks_synth.Workload, reserve_pages: int = 0, max_batch=None):
        self.w = w
        self.case = locks_synth.make_case(w, device="cuda:0")
        self.max_pages = self.case.block_table.shape[1]
        self.sm = 1.0 / math.sqrt(w.d)
        self.cfg = make_config(w.Hq, w.Hkv, w.rank, w.fmt, w.dtype, max_batch or w.n, self.max_pages, w.budget, B=w.B)
        self.ctx = locks.Context(self.cfg)
        self.kv = KVView(self.case.k, self.case.v, self.case.strides, self.case.num_blocks, self.case.block_table,
                         self.case.seq_lens)
        self.k = w.k
        self.cache = oracle_cache(self.case)          # CPU copy of the very same stored values
        self.fmt = fmt_code(w)

    # ---- oracle side
    def oracle_summaries(self):
        return oracle.build_summaries(self.cache, self.w.rank, self.fmt)

    # ---- CUDA side (through the C ABI)
    def gpu_build(self):
        summ = self.ctx.new_summaries(self.case.num_blocks)
        self.ctx.locks_build_summaries(self.kv, self.w.n, summ)
        torch.cuda.synchronize()
        return summ

    def gpu_select(self, summ, q=None):
        w = self.w
        q = self.case.q if q is None else q
        ids = torch.full((w.n, w.Hkv, self.k), -7, dtype=torch.int32, device="cuda:0")
        cnt = torch.full((w.n, w.Hkv), -7, dtype=torch.int32, device="cuda:0")
        logmass = torch.full((w.n, w.Hq, self.max_pages), float("nan"), dtype=torch.float32, device="cuda:0")
        logshare = torch.full((w.n, w.Hkv, self.max_pages), float("nan"), dtype=torch.float32, device="cuda:0")
        self.ctx.locks_select(q, summ, self.kv, w.n, ids, cnt, logmass, logshare)
        torch.cuda.synchronize()
        return ids.cpu().numpy(), cnt.cpu().numpy(), logmass.cpu().numpy(), logshare.cpu().numpy()

    def gpu_attend(self, ids=None, cnt=None, q=None):
        w = self.w
        q = self.case.q if q is None else q
        out = torch.full((w.n, w.Hq, w.d), float("nan"), dtype=q.dtype, device="cuda:0")
        lse = torch.full((w.n, w.Hq), float("nan"), dtype=torch.float32, device="cuda:0")
        if ids is not None:
            ids = torch.as_tensor(ids, dtype=torch.int32, device="cuda:0").contiguous()
            cnt = torch.as_tensor(cnt, dtype=torch.int32, device="cuda:0").contiguous()
        self.ctx.locks_sparse_attend(q, self.kv, w.n, ids, cnt, out, lse)
        torch.cuda.synchronize()
        return out.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)

    def status(self):
        return self.ctx.locks_poll_status()


def upload(summ_np):
    return torch.from_numpy(np.ascontiguousarray(summ_np)).to("cuda:0")


def check_select_and_attend(gc: GpuCase, summ_np, out_tol, mass_tol=1e-3, q=None):
    """Full parity of select + attend on identical summary bytes.  Returns #problems whose set differed."""
    from common import check_page_sets
    w = gc.w
    qt = gc.case.q if q is None else q
    qn = t2np(qt)
    ids, cnt, logmass, logshare = gc.gpu_select(upload(summ_np), qt)
    shat = oracle.page_logmass(gc.cache, qn, w.rank, gc.fmt, summ_np, gc.sm)
    oids, ocnt, ologshare = oracle.select(gc.cache, shat, gc.k)
    seq = gc.cache.seq_lens
    for b in range(w.n):
        P = -(-int(seq[b]) // w.B)
        if P <= gc.k:
            continue
        d = np.abs(logmass[b, :, :P - 1] - shat[b, :, :P - 1])
        assert np.nanmax(d) <= mass_tol, ("page log-mass", b, np.nanmax(d))
        assert not np.isnan(logmass[b, :, :P - 1]).any()
        d = np.abs(logshare[b, :, 1:P - 1] - ologshare[b, :, 1:P - 1])
        assert np.nanmax(d) <= mass_tol, ("page log-share", b, np.nanmax(d))
    differed = check_page_sets(ids, cnt, oids, ocnt, ologshare, seq, w.B, gc.k)
    # the oracle attends the GPU's own set (identical to its own unless a tie band was used)
    out, lse = gc.gpu_attend(ids, cnt, qt)
    oout, olse = oracle.attend(gc.cache, qn, gc.sm, ids, cnt)
    assert np.abs(out - oout).max() <= out_tol, ("attend out", np.abs(out - oout).max())
    assert np.abs(lse - olse).max() <= 1e-3 * max(1.0, np.abs(olse).max() / 10), ("attend lse", np.abs(lse - olse).max())
    assert gc.status() == 0
    return differed
