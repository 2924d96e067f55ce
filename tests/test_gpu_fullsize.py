"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration bench.py times.

Summaries are built on the GPU and the very same bytes are handed to the oracle (the builder itself is
compared with the oracle's in test_gpu_parity.py), so page masses, shares, page sets and outputs are
compared on identical inputs.  Tolerances as everywhere: masses and shares 1e-3, sets identical outside a
2e-3 tie band, outputs 2e-2 (bf16 KV), lse 1e-3.
"""
import numpy as np
import pytest
import torch

import locks_synth
import oracle
import paper_2607_24555_b200 as locks
from common import check_page_sets, oracle_cache, t2np

pytestmark = pytest.mark.gpu


def _gc(w, **kw):
    from gpu_util import GpuCase
    return GpuCase(w, **kw)


@pytest.mark.parametrize("rank,budget", [(2, 256), (8, 1024)])
def test_config2_full_size(rank, budget):
    """Qwen shapes, 32 x 16K, isotropic filler with 64 carriers per sequence: 256 (request, KV head) problems,
    one attention CTA per problem, every page mass of every problem checked."""
    from gpu_util import check_select_and_attend
    gc = _gc(locks_synth.config2(rank=rank, budget=budget))
    summ_np = gc.gpu_build().cpu().numpy()
    differed = check_select_and_attend(gc, summ_np, out_tol=2e-2)
    assert differed <= 8, differed                                   # of 256 problems
    # 64 carrier pages per sequence compete for k - 2 < 64 slots: what is kept besides sink and tail are carriers
    ids, _, _, _ = gc.gpu_select(torch.from_numpy(summ_np).cuda())
    kept = hits = 0
    for b in range(gc.w.n):
        cps = set(gc.case.carrier_pages[b])
        for h in range(gc.w.Hkv):
            cand = ids[b, h, 1:gc.k - 1].tolist()
            kept += len(cand)
            hits += sum(1 for j in cand if j in cps)
    assert hits >= 0.9 * kept, (hits, kept)


def test_config3_full_size_1m():
    """GLM shapes, one request of 1M tokens (65 536 pages, G = 16): tens of selector chunks per KV head and the
    CTA-merged scan; every page mass, both page sets and all 32 outputs."""
    from gpu_util import check_select_and_attend
    gc = _gc(locks_synth.config3(T=1 << 20))
    summ_np = gc.gpu_build().cpu().numpy()
    differed = check_select_and_attend(gc, summ_np, out_tol=2e-2)
    assert differed <= 1


def test_config3_512k():
    from gpu_util import check_select_and_attend
    gc = _gc(locks_synth.config3(T=1 << 19))
    summ_np = gc.gpu_build().cpu().numpy()
    differed = check_select_and_attend(gc, summ_np, out_tol=2e-2)
    assert differed <= 1


def test_config4_batch8_graph_replay_against_stepwise_oracle():
    """Batched serving shapes (8 requests, lengths uniform in 64K..128K): locks_decode_step captured once in a CUDA
    graph and replayed 24 times; every replay appends a token per request and builds the summaries of the pages
    that fill.  The oracle steps a 4-request subset on a CPU copy of the cache that the test itself keeps up to
    date (the appended rows are written at the positions the lengths name; the summaries of freshly filled pages
    are the GPU-built bytes), and checks lengths, page sets and outputs after every replay; at the end the whole
    GPU cache must equal the CPU copy bit for bit."""
    steps, sub = 24, [0, 3, 5, 6]
    w0 = locks_synth.config4(batch=8)
    lens0 = list(w0.seq_lens)
    lens0[0] = lens0[0] // 16 * 16 + 9        # a few requests cross a page boundary early and again 16 steps later
    lens0[3] = lens0[3] // 16 * 16 + 15
    lens0[5] = lens0[5] // 16 * 16
    w = w0.with_(seq_lens=[t + 48 for t in lens0])
    gc = _gc(w)
    dev = "cuda:0"
    gc.case.seq_lens.copy_(torch.tensor(lens0, dtype=torch.int32, device=dev))
    summ = gc.ctx.new_summaries(gc.case.num_blocks)
    gc.ctx.locks_build_summaries(gc.kv, w.n, summ)
    out = torch.empty(w.n, w.Hq, w.d, dtype=torch.bfloat16, device=dev)
    ids = torch.empty(w.n, w.Hkv, gc.k, dtype=torch.int32, device=dev)
    cnt = torch.empty(w.n, w.Hkv, dtype=torch.int32, device=dev)
    kn, vn, qn = [t.clone() for t in locks_synth.new_token(w, 0, device=dev)]
    gc.ctx.locks_set_scan_partition(locks.PARTITION_BALANCED)   # what the library picks for these lengths
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        saved = gc.case.seq_lens.clone()
        gc.ctx.locks_decode_step(qn, kn, vn, gc.kv, summ, w.n, out, ids, cnt, stream=s)   # warm-up on scratch lengths
        s.synchronize()
        gc.case.seq_lens.copy_(saved)
        gc.ctx.locks_build_summaries(gc.kv, w.n, summ, stream=s)                          # (undo a warm-up fill)
        s.synchronize()
        with torch.cuda.graph(g, stream=s):
            gc.ctx.locks_decode_step(qn, kn, vn, gc.kv, summ, w.n, out, ids, cnt, stream=s)
    torch.cuda.synchronize()
    # CPU mirror: full K / V / summaries once, then patched by the test
    k_np, v_np = t2np(gc.case.k).copy(), t2np(gc.case.v).copy()
    summ_np = summ.cpu().numpy().copy()
    bt = gc.case.block_table.cpu().numpy()
    lens = np.array(lens0, np.int64)
    sb, sh, st = gc.case.strides
    strides = {"shape": (gc.case.num_blocks, w.Hkv, w.B, w.d), "block": sb, "head": sh, "token": st}
    filled = 0
    for step in range(steps):
        a, b_, c = locks_synth.new_token(w, step, device=dev)
        kn.copy_(a); vn.copy_(b_); qn.copy_(c)
        g.replay()
        torch.cuda.synchronize()
        assert gc.status() == 0
        kn_np, vn_np = t2np(kn), t2np(vn)
        for b in range(w.n):                                           # the append, written out
            page, slot = divmod(int(lens[b]), w.B)
            k_np[bt[b, page], :, slot, :] = kn_np[b]
            v_np[bt[b, page], :, slot, :] = vn_np[b]
        lens += 1
        assert gc.case.seq_lens.cpu().tolist() == lens.tolist()
        sub_cache = oracle.Cache(k_np, v_np, bt[sub], lens[sub].astype(np.int32), w.Hq, strides=strides)
        q_sub = t2np(qn)[sub]
        shat = oracle.page_logmass(sub_cache, q_sub, w.rank, gc.fmt, summ_np, gc.sm)
        oids, ocnt, ols = oracle.select(sub_cache, shat, gc.k)
        gids, gcnt = ids.cpu().numpy()[sub], cnt.cpu().numpy()[sub]
        check_page_sets(gids, gcnt, oids, ocnt, ols, sub_cache.seq_lens, w.B, gc.k)
        oout, _ = oracle.attend(sub_cache, q_sub, gc.sm, gids, gcnt)
        assert np.abs(out.float().cpu().numpy()[sub] - oout).max() <= 2e-2, step
        for b in range(w.n):                                           # pages that filled: GPU-built bytes, checked
            if lens[b] % w.B == 0:
                blk = int(bt[b, lens[b] // w.B - 1])
                got = summ[blk].cpu().numpy()
                assert got.any()
                summ_np[blk] = got
                filled += 1
                if b in sub:
                    one = oracle.Cache(k_np, v_np, bt[b:b + 1], lens[b:b + 1].astype(np.int32), w.Hq, strides=strides)
                    ref = oracle.build_summaries(one, w.rank, gc.fmt, page_begin=[lens[b] // w.B - 1],
                                                 page_end=[lens[b] // w.B])
                    for h in range(w.Hkv):
                        gV, gC, gMu, _, _, _ = oracle.unpack_codes(w.rank, got[h])
                        oV, oC, oMu, _, _, _ = oracle.unpack_codes(w.rank, ref[blk, h])
                        for l in range(w.rank):
                            if int(np.dot(gV[l], oV[l])) < 0:
                                gV[l] = -gV[l]; gC[:, l] = -gC[:, l]
                        assert np.abs(gV - oV).max() <= 1 and np.abs(gC - oC).max() <= 1 and np.abs(gMu - oMu).max() <= 1
    assert filled >= 8                                                 # every request crossed a boundary at least once
    assert np.array_equal(t2np(gc.case.k), k_np) and np.array_equal(t2np(gc.case.v), v_np)
