"""The allocation-free sparse-attention entry point against the regular one and against the oracle.

Some callers of the library cannot allocate device memory (a plugin inside an engine that owns the
whole device's memory pool, a path that must not synchronise, a fixed memory budget), so they have no
workspace to give locks_create().  locks_sparse_attend_noalloc keeps its split partials in an array
inside the library instead.  This file is collected last on purpose: if it fails, every other test
has already run.
"""
import numpy as np
import pytest
import torch

import locks_synth

pytestmark = pytest.mark.gpu


def _case(seed):
    from gpu_util import GpuCase
    w = locks_synth.Workload("noalloc", [16 * 300 + 5, 16 * 200, 700], Hq=8, Hkv=2, budget=512, seed=seed)
    return GpuCase(w)


def test_noalloc_entry_point_matches_workspace_entry_point_twice():
    import paper_2607_24555_b200 as locks
    gc = _case(77)
    w = gc.w
    summ = gc.gpu_build()
    ids, cnt, _, _ = gc.gpu_select(summ)
    ref, ref_lse = gc.gpu_attend(ids, cnt)                      # existing entry point (context + workspace)
    import oracle
    from common import t2np
    ora, ora_lse = oracle.attend(gc.cache, t2np(gc.case.q), gc.sm, ids, cnt)   # and the definition itself
    ids_d = torch.as_tensor(ids, device="cuda:0").contiguous()
    cnt_d = torch.as_tensor(cnt, device="cuda:0").contiguous()
    for call in range(2):                                       # two calls in a row share the built-in array
        out = torch.full((w.n, w.Hq, w.d), float("nan"), dtype=torch.bfloat16, device="cuda:0")
        lse = torch.full((w.n, w.Hq), float("nan"), dtype=torch.float32, device="cuda:0")
        locks.locks_sparse_attend_noalloc(gc.cfg, gc.case.q, gc.kv, w.n, ids_d, cnt_d, out, lse)
        torch.cuda.synchronize()
        got = out.float().cpu().numpy().astype(np.float64)
        assert np.abs(got - ref).max() <= 2e-2, (call, np.abs(got - ref).max())
        assert np.abs(lse.cpu().numpy() - ref_lse).max() <= 1e-3, call
        assert np.abs(got - ora).max() <= 2e-2 and np.abs(lse.cpu().numpy() - ora_lse).max() <= 1e-3, call
    # dense mode (no page table) through the same entry point
    dref, dref_lse = gc.gpu_attend()
    out = torch.empty(w.n, w.Hq, w.d, dtype=torch.bfloat16, device="cuda:0")
    lse = torch.empty(w.n, w.Hq, dtype=torch.float32, device="cuda:0")
    locks.locks_sparse_attend_noalloc(gc.cfg, gc.case.q, gc.kv, w.n, None, None, out, lse)
    torch.cuda.synchronize()
    assert np.abs(out.float().cpu().numpy() - dref).max() <= 2e-2
    assert np.abs(lse.cpu().numpy() - dref_lse).max() <= 1e-3


def test_noalloc_entry_point_refuses_problems_beyond_its_scratch():
    import paper_2607_24555_b200 as locks
    from paper_2607_24555_b200.binding import make_config
    gc = _case(78)
    w = gc.w
    big = make_config(512, 128, 8, "i4", "bf16", 1, gc.max_pages, w.budget)     # 512 query heads > 256 rows
    out = torch.empty(1, 512, w.d, dtype=torch.bfloat16, device="cuda:0")
    q = torch.zeros(1, 512, w.d, dtype=torch.bfloat16, device="cuda:0")
    with pytest.raises(locks.LocksError, match="built-in scratch"):
        locks.locks_sparse_attend_noalloc(big, q, gc.kv, 1, None, None, out)
