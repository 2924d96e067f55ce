"""GPU parity of the diagnostics: the exact-LSE selection arm (Lemma 1(ii)) and the selection-fidelity metrics
(App. B) against the oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import locks_synth
import oracle
from common import check_page_sets, t2np

pytestmark = pytest.mark.gpu


def _gc(w, **kw):
    from gpu_util import GpuCase
    return GpuCase(w, **kw)


def _exact(gc):
    w = gc.w
    ids = torch.full((w.n, w.Hkv, gc.k), -7, dtype=torch.int32, device="cuda:0")
    cnt = torch.full((w.n, w.Hkv), -7, dtype=torch.int32, device="cuda:0")
    mass = torch.full((w.n, w.Hq, gc.max_pages), float("nan"), dtype=torch.float32, device="cuda:0")
    share = torch.full((w.n, w.Hkv, gc.max_pages), float("nan"), dtype=torch.float32, device="cuda:0")
    gc.ctx.locks_select_exact(gc.case.q, gc.kv, w.n, ids, cnt, mass, share)
    torch.cuda.synchronize()
    return ids, cnt, mass, share


def _check_exact(gc, tol):
    w = gc.w
    ids, cnt, mass, share = _exact(gc)
    omass = oracle.page_exact_mass_all(gc.cache, t2np(gc.case.q), gc.sm)
    oids, ocnt, oshare = oracle.select(gc.cache, omass, gc.k)
    gm, gs = mass.cpu().numpy(), share.cpu().numpy()
    for b, T in enumerate(gc.cache.seq_lens):
        P = -(-int(T) // w.B)
        assert np.abs(gm[b, :, :P] - omass[b, :, :P]).max() <= tol, b         # every page, the partial tail included
        if P > gc.k:
            assert np.abs(gs[b, :, 1:P - 1] - oshare[b, :, 1:P - 1]).max() <= tol
    check_page_sets(ids.cpu().numpy(), cnt.cpu().numpy(), oids, ocnt, oshare, gc.cache.seq_lens, w.B, gc.k)
    assert gc.status() == 0
    return ids, cnt, mass, omass, oids, ocnt


@pytest.mark.parametrize("Hq,Hkv", [(8, 2), (32, 2), (6, 2), (4, 4)])
def test_exact_selection_matches_oracle(Hq, Hkv):
    gc = _gc(locks_synth.Workload("exact", [16 * 700 + 5, 16 * 64, 300, 16 * 65 + 1], Hq=Hq, Hkv=Hkv, budget=256,
                                  carriers=4, seed=Hq))
    _check_exact(gc, 1e-3)


def test_exact_selection_fp32_config0():
    gc = _gc(locks_synth.config0())
    ids, cnt, mass, omass, oids, ocnt = _check_exact(gc, 1e-4)
    assert np.array_equal(ids.cpu().numpy(), oids)
    for cp in gc.case.carrier_pages[0]:
        assert cp in oids[0, 0].tolist()


def test_selection_quality_matches_oracle_and_estimator_tracks_the_ceiling():
    """gamma, gamma_c, recall and needle of the estimated selection against the exact arm: the kernel's numbers
    equal the oracle's on the same tables, and on locally low-rank keys the rank-8 summary keeps nearly all of
    the mass the exact ranking keeps (the paper's selection-fidelity table: gamma within a point of the ceiling)."""
    w = locks_synth.Workload("quality", [16 * 1500 + 3, 16 * 900], Hq=8, Hkv=2, budget=512, carriers=8, q_scale=0.5, seed=12)
    gc = _gc(w)
    summ = gc.gpu_build()
    ids_e, cnt_e, mass, _ = _exact(gc)
    ids_s, cnt_s, _, _ = gc.gpu_select(summ)
    ids_s = torch.from_numpy(ids_s).cuda(); cnt_s = torch.from_numpy(cnt_s).cuda()
    marked = torch.tensor([cp[:8] for cp in gc.case.carrier_pages], dtype=torch.int32, device="cuda:0")
    qual = torch.full((w.n, w.Hkv, 4), float("nan"), dtype=torch.float32, device="cuda:0")
    ceil_ = torch.full((w.n, w.Hkv, 4), float("nan"), dtype=torch.float32, device="cuda:0")
    gc.ctx.locks_selection_quality(mass, gc.kv, w.n, ids_s, cnt_s, ids_e, cnt_e, qual, marked_pages=marked)
    gc.ctx.locks_selection_quality(mass, gc.kv, w.n, ids_e, cnt_e, ids_e, cnt_e, ceil_, marked_pages=marked)
    torch.cuda.synchronize()
    omass = oracle.page_exact_mass_all(gc.cache, t2np(gc.case.q), gc.sm)
    G = w.Hq // w.Hkv
    for b in range(w.n):
        P = -(-w.seq_lens[b] // w.B)
        for h in range(w.Hkv):
            A = ids_s[b, h, :int(cnt_s[b, h])].cpu().numpy()
            R = ids_e[b, h, :int(cnt_e[b, h])].cpu().numpy()
            want = oracle.selection_quality(omass[b, h * G:(h + 1) * G], P, A, R, marked[b].cpu().numpy())
            assert np.abs(qual[b, h].cpu().numpy() - np.array(want)).max() <= 2e-3, (b, h, qual[b, h], want)
            want_c = oracle.selection_quality(omass[b, h * G:(h + 1) * G], P, R, R, marked[b].cpu().numpy())
            assert np.abs(ceil_[b, h].cpu().numpy() - np.array(want_c)).max() <= 2e-3
    q_, c_ = qual.cpu().numpy(), ceil_.cpu().numpy()
    assert np.all(c_[..., 2] == 1.0) and np.all(c_[..., 3] == 1.0)
    assert np.all(q_[..., 0] >= c_[..., 0] - 0.02)        # total mass within two points of the ceiling
    assert np.all(q_[..., 3] >= 0.99)                     # carriers the exact ranking keeps are kept
    assert gc.status() == 0


@pytest.mark.parametrize("rule", [1, 2])
@pytest.mark.parametrize("lens,Hq,Hkv", [([16 * 700 + 5, 16 * 90], 8, 2), ([16 * 9000 + 3], 32, 2)])
def test_combine_rule_switch_matches_oracle(rule, lens, Hq, Hkv):
    """Group-max and group-mass combine (the rules the paper ablates its share-average against), single- and
    multi-chunk selection: ranking keys and page sets against the oracle's statement of each rule."""
    import paper_2607_24555_b200 as locks
    from paper_2607_24555_b200.binding import make_config
    gc = _gc(locks_synth.Workload("combine", lens, Hq=Hq, Hkv=Hkv, budget=256, q_scale=0.5, seed=rule + Hq))
    w = gc.w
    cfg = make_config(w.Hq, w.Hkv, w.rank, w.fmt, w.dtype, w.n, gc.max_pages, w.budget, combine=rule)
    ctx = locks.Context(cfg)
    summ_np = gc.oracle_summaries()
    summ = torch.from_numpy(summ_np).cuda()
    ids = torch.full((w.n, w.Hkv, gc.k), -7, dtype=torch.int32, device="cuda:0")
    cnt = torch.full((w.n, w.Hkv), -7, dtype=torch.int32, device="cuda:0")
    key = torch.full((w.n, w.Hkv, gc.max_pages), float("nan"), dtype=torch.float32, device="cuda:0")
    ctx.locks_select(gc.case.q, summ, gc.kv, w.n, ids, cnt, None, key)
    torch.cuda.synchronize()
    assert ctx.locks_poll_status() == 0
    shat = oracle.page_logmass(gc.cache, t2np(gc.case.q), w.rank, gc.fmt, summ_np, gc.sm)
    G = w.Hq // w.Hkv
    oids = np.full((w.n, w.Hkv, gc.k), -1, np.int32)
    ocnt = np.zeros((w.n, w.Hkv), np.int32)
    okey = np.full((w.n, w.Hkv, gc.max_pages), np.nan)
    for b in range(w.n):
        P = -(-w.seq_lens[b] // w.B)
        for h in range(w.Hkv):
            oids[b, h], ocnt[b, h], kk = oracle.select_one_rule(shat[b, h * G:(h + 1) * G], P, gc.k, rule)
            okey[b, h, :P] = kk[:P]
            assert np.abs(key[b, h, 1:P - 1].cpu().numpy() - kk[1:P - 1]).max() <= 1e-3
    check_page_sets(ids.cpu().numpy(), cnt.cpu().numpy(), oids, ocnt, okey, gc.cache.seq_lens, w.B, gc.k)


@pytest.mark.parametrize("lens,Hq,Hkv,dtype,fmt,part", [([16 * 700 + 5, 16 * 90, 16 * 300], 8, 2, "bf16", "i4", 1),
                                                        ([16 * 9000 + 3], 32, 2, "bf16", "i4", 1),
                                                        ([16 * 500 + 9, 16 * 64], 4, 1, "f32", "f32", 1),
                                                        ([16 * 2000 + 5, 16 * 90, 16 * 700, 16 * 31], 8, 2, "bf16", "i4", 2)])
def test_per_head_arm_matches_oracle(lens, Hq, Hkv, dtype, fmt, part):
    """The per-head arm of the paper's combine ablation: every query head ranks by its own share, keeps its own k
    pages and attends them (one page table per query head).  Keys, page sets and attention outputs against the
    oracle; single- and multi-chunk selection, both scan partitions, the tensor-core and the plain attention kernels;
    calls that need one table per KV head refuse the configuration."""
    import paper_2607_24555_b200 as locks
    from paper_2607_24555_b200.binding import make_config
    gc = _gc(locks_synth.Workload("perhead", lens, Hq=Hq, Hkv=Hkv, budget=256, q_scale=0.5, dtype=dtype, fmt=fmt, seed=Hq + len(lens)))
    w = gc.w
    cfg = make_config(w.Hq, w.Hkv, w.rank, w.fmt, w.dtype, w.n, gc.max_pages, w.budget, combine=locks.COMBINE_PER_HEAD)
    ctx = locks.Context(cfg)
    ctx.locks_set_scan_partition(part)
    summ_np = gc.oracle_summaries()
    summ = torch.from_numpy(summ_np).cuda()
    ids = torch.full((w.n, w.Hq, gc.k), -7, dtype=torch.int32, device="cuda:0")
    cnt = torch.full((w.n, w.Hq), -7, dtype=torch.int32, device="cuda:0")
    key = torch.full((w.n, w.Hq, gc.max_pages), float("nan"), dtype=torch.float32, device="cuda:0")
    ctx.locks_select(gc.case.q, summ, gc.kv, w.n, ids, cnt, None, key)
    torch.cuda.synchronize()
    assert ctx.locks_poll_status() == 0
    qn = t2np(gc.case.q)
    shat = oracle.page_logmass(gc.cache, qn, w.rank, gc.fmt, summ_np, gc.sm)
    oids, ocnt, okey = oracle.select_per_head(gc.cache, shat, gc.k)
    for b in range(w.n):
        P = -(-w.seq_lens[b] // w.B)
        if P > gc.k:
            assert np.abs(key[b, :, 1:P - 1].cpu().numpy() - okey[b, :, 1:P - 1]).max() <= 1e-3
    # the tie-aware set check treats every (request, query head) as a problem: a view with Hq "KV heads"
    check_page_sets(ids.cpu().numpy(), cnt.cpu().numpy(), oids, ocnt, okey, gc.cache.seq_lens, w.B, gc.k)
    if w.Hq > w.Hkv:
        G = w.Hq // w.Hkv
        assert any(len({tuple(r) for r in ids[b, h * G:(h + 1) * G].cpu().tolist()}) > 1 for b in range(w.n) for h in range(w.Hkv))
    out = torch.full((w.n, w.Hq, w.d), float("nan"), dtype=gc.case.q.dtype, device="cuda:0")
    lse = torch.full((w.n, w.Hq), float("nan"), dtype=torch.float32, device="cuda:0")
    ctx.locks_sparse_attend(gc.case.q, gc.kv, w.n, ids, cnt, out, lse)
    torch.cuda.synchronize()
    assert ctx.locks_poll_status() == 0
    oout, olse = oracle.attend(gc.cache, qn, gc.sm, ids.cpu().numpy(), cnt.cpu().numpy(), per_head=True)
    assert np.abs(out.float().cpu().numpy() - oout).max() <= (2e-2 if dtype == "bf16" else 1e-4)
    assert np.abs(lse.cpu().numpy() - olse).max() <= 1e-3
    # dense mode is unchanged by the rule
    dout = torch.empty_like(out)
    ctx.locks_sparse_attend(gc.case.q, gc.kv, w.n, None, None, dout)
    torch.cuda.synchronize()
    dref, _ = oracle.attend(gc.cache, qn, gc.sm)
    assert np.abs(dout.float().cpu().numpy() - dref).max() <= (2e-2 if dtype == "bf16" else 1e-4)
    kn, vn, q1 = locks_synth.new_token(w, 0, device="cuda:0")
    with pytest.raises(locks.LocksError):
        ctx.locks_decode_step(q1, kn, vn, gc.kv, summ, w.n, out, ids, cnt)


@pytest.mark.parametrize("scorer", [1, 2, 3])
@pytest.mark.parametrize("fmt,dtype,Hq,Hkv", [("i4", "bf16", 8, 2), ("f32", "f32", 4, 1), ("i4", "bf16", 32, 2)])
def test_rival_scorers_match_oracle(scorer, fmt, dtype, Hq, Hkv):
    """Centroid-only, moment-core and envelope scores, and the selections they lead to, against the oracle."""
    import paper_2607_24555_b200 as locks
    w = locks_synth.Workload("rival", [16 * 300 + 5, 16 * 70], Hq=Hq, Hkv=Hkv, budget=256, fmt=fmt, dtype=dtype,
                             carriers=4, q_scale=0.5, seed=scorer + Hq)
    gc = _gc(w)
    summ_np = gc.oracle_summaries()
    summ = torch.from_numpy(summ_np).cuda()
    ids = torch.full((w.n, w.Hkv, gc.k), -7, dtype=torch.int32, device="cuda:0")
    cnt = torch.full((w.n, w.Hkv), -7, dtype=torch.int32, device="cuda:0")
    score = torch.full((w.n, w.Hq, gc.max_pages), float("nan"), dtype=torch.float32, device="cuda:0")
    key = torch.full((w.n, w.Hkv, gc.max_pages), float("nan"), dtype=torch.float32, device="cuda:0")
    gc.ctx.locks_select_rival(scorer, gc.case.q, summ, gc.kv, w.n, ids, cnt, score, key)
    torch.cuda.synchronize()
    assert gc.status() == 0
    oscore = oracle.rival_logmass(gc.cache, t2np(gc.case.q), w.rank, gc.fmt, summ_np, gc.sm, scorer)
    oids, ocnt, okey = oracle.select(gc.cache, oscore, gc.k)
    tol = 1e-3 if dtype == "bf16" else 2e-4
    for b, T in enumerate(w.seq_lens):
        P = -(-T // w.B)
        assert np.abs(score[b, :, :P - 1].cpu().numpy() - oscore[b, :, :P - 1]).max() <= tol
        assert np.abs(key[b, :, 1:P - 1].cpu().numpy() - okey[b, :, 1:P - 1]).max() <= tol
    check_page_sets(ids.cpu().numpy(), cnt.cpu().numpy(), oids, ocnt, okey, gc.cache.seq_lens, w.B, gc.k)
    # the context still runs the summary's own scorer afterwards
    ids2, cnt2, lm, _ = gc.gpu_select(summ)
    shat = oracle.page_logmass(gc.cache, t2np(gc.case.q), w.rank, gc.fmt, summ_np, gc.sm)
    assert np.nanmax(np.abs(lm[0, :, :10] - shat[0, :, :10])) <= 1e-3


@pytest.mark.parametrize("bits,dtype,arm", [(4, "bf16", "post"), (2, "bf16", "pre"), (4, "f32", "pre")])
def test_fake_quantised_cache_composition(bits, dtype, arm):
    """KIVI-style fake quantisation of the complete pages on the GPU against the oracle's, then the paper's two
    compositions: "post" (summaries from the original keys, attention on quantised KV) and "pre" (summaries from
    the quantised keys): page masses, sets and outputs against the oracle on the quantised cache."""
    from common import oracle_cache
    from gpu_util import check_select_and_attend, upload
    fmt = "i4" if dtype == "bf16" else "f32"
    w = locks_synth.Workload("kivi", [16 * 200 + 7, 16 * 90], Hq=8, Hkv=2, budget=256, dtype=dtype, fmt=fmt, q_scale=0.5,
                             layout="NHD" if bits == 2 else "HND", seed=bits)
    gc = _gc(w)
    ref = oracle_cache(gc.case)                                       # CPU copy of the original values
    summ_before = gc.gpu_build() if arm == "post" else None
    gc.ctx.locks_fake_quantize_pages(gc.kv, w.n, bits)
    torch.cuda.synchronize()
    assert gc.status() == 0
    oracle.fake_quantize_pages(ref, bits)
    got = oracle_cache(gc.case)

    def vals(a):
        return ((a.astype(np.uint32) << 16).view(np.float32) if a.dtype == np.uint16 else a).astype(np.float64)

    for a, b_ in ((got.k, ref.k), (got.v, ref.v)):
        d = np.abs(vals(a) - vals(b_))
        # fp32 against fp64 arithmetic: an entry within rounding of a grid midpoint may land on the neighbouring level
        assert (d > 1e-6 * np.abs(vals(b_)).max() + 2.0 ** -8 * np.abs(vals(b_)) * (a.dtype == np.uint16)).mean() <= 2e-3
        assert d.max() <= (vals(b_).max() - vals(b_).min()) / (2 ** bits - 1)
    gc.cache = got                                                    # from here on: the GPU's quantised cache
    summ = summ_before if arm == "post" else gc.gpu_build()
    check_select_and_attend(gc, summ.cpu().numpy(), out_tol=2e-2 if dtype == "bf16" else 1e-4)


@pytest.mark.parametrize("fmt,rank,dtype", [("i8", 8, "bf16"), ("bf16", 8, "bf16"), ("i8", 5, "f32"), ("bf16", 3, "f32")])
def test_wide_basis_formats(fmt, rank, dtype):
    """Int8-basis and bf16-basis ("r8fp") summaries (the precision arms of the paper's ablation): select + attend on
    oracle-built blobs, then the GPU build against the oracle's build through probe scores, stored scales and the
    basis itself (after aligning the sign convention of each mode)."""
    from gpu_util import check_select_and_attend
    w = locks_synth.Workload("widefmt", [16 * 300 + 3, 16 * 80], Hq=8, Hkv=2, budget=256, rank=rank, fmt=fmt, dtype=dtype,
                             q_scale=0.5, seed=rank)
    gc = _gc(w)
    o_summ = gc.oracle_summaries()
    check_select_and_attend(gc, o_summ, out_tol=2e-2 if dtype == "bf16" else 1e-4)
    g_summ = gc.gpu_build().cpu().numpy()
    assert g_summ.shape == o_summ.shape
    rng = np.random.default_rng(2)
    bt = gc.cache.block_table[0]
    worst = 0.0
    for p in range(0, 300, 7):
        for h in range(2):
            mg = oracle.unpack(gc.fmt, rank, g_summ[bt[p], h])
            mo = oracle.unpack(gc.fmt, rank, o_summ[bt[p], h])
            for l in range(rank):
                if float(np.dot(mg[1][l], mo[1][l])) < 0:
                    mg[1][l] *= -1; mg[2][:, l] *= -1
            assert np.abs(mg[0] - mo[0]).max() <= np.abs(mo[0]).max() / 127 + 1e-6            # centroid within one code
            assert np.abs(mg[1] - mo[1]).max() <= 0.02                                        # basis entries (|v| <= 1)
            q = rng.standard_normal(128)
            worst = max(worst, abs(oracle.score(*mg, q, gc.sm) - oracle.score(*mo, q, gc.sm)))
    assert worst <= 5e-3, worst
    assert gc.status() == 0
