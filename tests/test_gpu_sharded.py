"""GPU parity of the page-sharded decode step: one long request cut into 2 and 3 page shards that all live on this
one GPU and run in lock-step in one process (a gather is a stack; no kernel waits for another).  The merged
selection and output must be the unsharded ones and the oracle's."""
import numpy as np
import pytest
import torch

import locks_synth
import oracle
import paper_2607_24555_b200 as locks
from common import check_page_sets, t2np
from paper_2607_24555_b200.binding import KVView, make_config
from paper_2607_24555_b200.dist import GpuShardOps, emulate_sharded_decode_step, shard_pages

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("T,Hq,Hkv,budget", [(16 * 3000 + 5, 8, 2, 512), (16 * 9000, 32, 2, 1024)])
def test_sharded_step_equals_unsharded_and_oracle(world, T, Hq, Hkv, budget):
    from gpu_util import GpuCase
    w = locks_synth.Workload("sharded", [T], Hq=Hq, Hkv=Hkv, budget=budget, q_scale=0.5, seed=world + Hq)
    gc = GpuCase(w)
    summ = gc.gpu_build()
    q = gc.case.q
    P = -(-T // 16)
    k = gc.k
    bt = gc.case.block_table[0]
    ops = []
    for r, (lo, hi) in enumerate(shard_pages(P, world)):
        sink, tail = r == 0, r == world - 1
        row = torch.cat([bt[0:1] if sink else bt[lo:lo + 1], bt[lo:hi], bt[P - 1:P] if tail else bt[lo:lo + 1]])
        lp = row.numel()
        T_loc = (lp - 1) * 16 + ((T - (P - 1) * 16) if tail else 16)
        ctx = locks.Context(make_config(Hq, Hkv, w.rank, w.fmt, w.dtype, 1, lp, budget))
        kv = KVView(gc.case.k, gc.case.v, gc.case.strides, gc.case.num_blocks, row.reshape(1, lp).contiguous(),
                    torch.tensor([T_loc], dtype=torch.int32, device="cuda:0"))
        ops.append(GpuShardOps(ctx, kv, summ, lo, hi, sink, tail))
    outs, sels = emulate_sharded_decode_step(ops, q)
    torch.cuda.synchronize()
    for o in ops:
        assert o.ctx.locks_poll_status() == 0
    # every shard ends with the same selection and output
    for (ids, cnt), out in zip(sels[1:], outs[1:]):
        assert torch.equal(ids, sels[0][0]) and torch.equal(cnt, sels[0][1]) and torch.equal(out, outs[0])
    # against the oracle on the whole request (same GPU-built summary bytes)
    summ_np = summ.cpu().numpy()
    shat = oracle.page_logmass(gc.cache, t2np(q), w.rank, gc.fmt, summ_np, gc.sm)
    oids, ocnt, oshare = oracle.select(gc.cache, shat, k)
    full = np.full((1, Hkv, k), -1, np.int32)
    full[:, :, 0] = 0
    full[:, :, 1:k - 1] = sels[0][0].cpu().numpy()
    full[:, :, k - 1] = P - 1
    cnt_full = (sels[0][1].cpu().numpy() + 2).astype(np.int32)
    check_page_sets(full, cnt_full, oids, ocnt, oshare, gc.cache.seq_lens, w.B, k)
    oout, _ = oracle.attend(gc.cache, t2np(q), gc.sm, full, cnt_full)
    assert np.abs(outs[0].float().cpu().numpy() - oout).max() <= 2e-2
    # and against the unsharded library call
    ids_u, cnt_u, _, _ = gc.gpu_select(summ)
    assert np.array_equal(ids_u, full)
