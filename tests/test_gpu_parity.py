"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.

Tolerances: page log-masses and log-shares within 1e-3 (fp32 accumulation of exactly represented integer
codes: observed ~1e-5); outputs 2e-2 for bf16 KV because the probabilities enter the PV product as bf16 (8
bits: <= 2^-9 |v|max ~ 1e-2 per output) and the output itself is rounded to bf16 (4e-3);
selected page sets identical except inside a 2e-3 tie band around the oracle's threshold;
attention outputs within 2e-2 (bf16 KV) / 1e-4 (fp32); lse within 1e-3.
"""
import math

import numpy as np
import pytest
import torch

import locks_synth
import oracle
import paper_2607_24555_b200 as locks
from common import t2np

pytestmark = pytest.mark.gpu


def _gc(w, **kw):
    from gpu_util import GpuCase
    return GpuCase(w, **kw)


def small_bf16(seq_lens, Hq=8, Hkv=2, rank=8, budget=256, **kw):
    return locks_synth.Workload("small", list(seq_lens), Hq=Hq, Hkv=Hkv, rank=rank, budget=budget, **kw)


# ----------------------------------------------------------------------------- config 0 (fp32)

def test_config0_tiny_fp32_pipeline():
    from gpu_util import check_select_and_attend
    gc = _gc(locks_synth.config0())
    summ = gc.oracle_summaries()
    differed = check_select_and_attend(gc, summ, out_tol=1e-4, mass_tol=1e-4)
    assert differed == 0
    # planted carriers are all selected
    ids, cnt, _, _ = gc.gpu_select(torch.from_numpy(summ).cuda())
    for cp in gc.case.carrier_pages[0]:
        assert cp in ids[0, 0].tolist()
    # dense attention through the same entry point
    out, lse = gc.gpu_attend()
    oout, olse = oracle.attend(gc.cache, t2np(gc.case.q), gc.sm)
    assert np.abs(out - oout).max() <= 1e-4 and np.abs(lse - olse).max() <= 1e-3


def test_config0_soft_queries_exercise_the_merge():
    """With carriers the softmax is one-hot; a scaled-down query spreads mass over many pages."""
    from gpu_util import check_select_and_attend
    gc = _gc(locks_synth.config0().with_(carriers=0, q_scale=0.25, seq_lens=[4096 - 5]))
    check_select_and_attend(gc, gc.oracle_summaries(), out_tol=1e-4, mass_tol=1e-4)


def test_f32_build_matches_oracle_scores():
    """F32-format build: bases are compared through scores and projectors, never entry by entry."""
    gc = _gc(locks_synth.config0().with_(seq_lens=[1024]))
    w = gc.w
    g_summ = gc.gpu_build().cpu().numpy()
    o_summ = gc.oracle_summaries()
    rng = np.random.default_rng(0)
    bt = gc.cache.block_table[0]
    for p in range(0, 63):
        mu_g, V_g, C_g = oracle.unpack(oracle.FMT_F32, w.rank, g_summ[bt[p], 0])
        mu_o, V_o, C_o = oracle.unpack(oracle.FMT_F32, w.rank, o_summ[bt[p], 0])
        assert np.abs(mu_g - mu_o).max() < 1e-5
        assert np.abs(V_g @ V_g.T - np.eye(w.rank)).max() < 1e-4          # orthonormal
        assert np.abs(C_g.sum(0)).max() < 1e-3                              # centred coefficients
        for _ in range(4):
            q = rng.standard_normal(128)
            assert abs(oracle.score(mu_g, V_g, C_g, q, gc.sm) - oracle.score(mu_o, V_o, C_o, q, gc.sm)) < 1e-4
        assert np.abs(V_g.T @ V_g - V_o.T @ V_o).max() < 2e-3               # same subspace (gap is large here)
    assert gc.status() == 0


@pytest.mark.parametrize("log2_scale", [-40, 30])
def test_f32_build_is_invariant_to_the_scale_of_the_keys(log2_scale):
    """Keys multiplied by a power of two give the same basis, and centroid and coefficients multiplied by it
    (every step of the build is homogeneous in the keys; a power of two is exact in fp32): the eigen-solver
    must not depend on the magnitude of the Gram matrix (2^60 times larger or 2^80 times smaller here)."""
    s = float(2.0 ** log2_scale)
    w = locks_synth.config0().with_(seq_lens=[16 * 40])
    ga, gb = _gc(w), _gc(w)
    gb.case.k.mul_(s)
    sa = ga.gpu_build().cpu().numpy()
    sb = gb.gpu_build().cpu().numpy()
    bt = ga.cache.block_table[0]
    for p in range(40):
        mu_a, V_a, C_a = oracle.unpack(oracle.FMT_F32, w.rank, sa[bt[p], 0])
        mu_b, V_b, C_b = oracle.unpack(oracle.FMT_F32, w.rank, sb[bt[p], 0])
        assert np.array_equal(mu_b, mu_a * s)
        assert np.abs(V_b - V_a).max() < 1e-5
        assert np.abs(C_b / s - C_a).max() < 1e-5 * max(1.0, np.abs(C_a).max())
    assert ga.status() == 0 and gb.status() == 0


def test_full_rank_gpu_summary_is_exact():
    """r = B = 16 in the F32 format reproduces the exact page log-mass (Prop. 3)."""
    gc = _gc(locks_synth.config0().with_(rank=16, seq_lens=[800], n_dirs=0, carriers=0))
    summ = gc.gpu_build()
    ids, cnt, logmass, _ = gc.gpu_select(summ)
    exact = oracle.page_logmass(gc.cache, t2np(gc.case.q), 16, gc.fmt, None, gc.sm, exact=True)
    assert np.abs(logmass[0, :, :49] - exact[0, :, :49]).max() < 1e-3


# ----------------------------------------------------------------------------- bf16 + I4 path

@pytest.mark.parametrize("Hq,Hkv", [(8, 2), (4, 4), (8, 1), (16, 1), (32, 2), (6, 2)])
def test_i4_tensor_path_group_sizes(Hq, Hkv):
    from gpu_util import check_select_and_attend
    gc = _gc(small_bf16([2048 + 37, 4096, 700], Hq=Hq, Hkv=Hkv, budget=256, seed=Hq + Hkv))
    check_select_and_attend(gc, gc.oracle_summaries(), out_tol=2e-2)


@pytest.mark.parametrize("lens,budget", [([16], 64), ([17, 1, 33], 64), ([16 * 5], 64), ([16 * 5 + 1], 64),
                                         ([16 * 6 + 1], 64), ([2000, 48, 640], 512), ([130], 32)])
def test_edge_lengths(lens, budget):
    """Single page, P <= k, P = k + 1, partial tail pages, k = 2."""
    from gpu_util import check_select_and_attend
    gc = _gc(small_bf16(lens, budget=budget, seed=len(lens)))
    check_select_and_attend(gc, gc.oracle_summaries(), out_tol=2e-2)
    out, lse = gc.gpu_attend()                                            # dense
    oout, olse = oracle.attend(gc.cache, t2np(gc.case.q), gc.sm)
    assert np.abs(out - oout).max() <= 2e-2 and np.abs(lse - olse).max() <= 1e-3


def test_carriers_and_nhd_layout():
    from gpu_util import check_select_and_attend
    gc = _gc(small_bf16([3000, 1500], carriers=8, layout="NHD", seed=11))
    differed = check_select_and_attend(gc, gc.oracle_summaries(), out_tol=2e-2)
    ids, _, _, _ = gc.gpu_select(torch.from_numpy(gc.oracle_summaries()).cuda())
    for b in range(2):
        for cp in gc.case.carrier_pages[b]:
            assert all(cp in ids[b, h].tolist() for h in range(gc.w.Hkv))
    assert differed <= 1


@pytest.mark.parametrize("Hq,Hkv,rank,qs", [(8, 2, 8, 6.0), (32, 2, 8, 6.0), (8, 2, 2, 8.0), (12, 2, 4, 8.0), (8, 2, 8, 0.0)])
def test_extreme_logits_take_the_safe_log_sum_exp(Hq, Hkv, rank, qs):
    """Queries scaled up until within-page logit deviations exceed what 2^x holds in fp32 without subtracting a
    maximum (hundreds of log2 units), and a zero query: the scan's page masses must still match the oracle."""
    from gpu_util import check_select_and_attend
    gc = _gc(small_bf16([16 * 300 + 5, 16 * 90], Hq=Hq, Hkv=Hkv, rank=rank, budget=256, q_scale=qs, carriers=4, seed=int(qs) + Hq))
    summ = gc.oracle_summaries()
    shat = oracle.page_logmass(gc.cache, t2np(gc.case.q), rank, gc.fmt, summ, gc.sm)
    if qs > 0:
        assert np.nanmax(shat) - np.nanmedian(shat) > 100          # logits far beyond the fp32 exponent range in log2
    check_select_and_attend(gc, summ, out_tol=2e-2, mass_tol=1e-3 * max(1.0, float(np.nanmax(np.abs(shat))) / 50))


def test_tail_slots_are_never_read_as_data():
    """Cache slots past the sequence end hold NaN: outputs must not change."""
    from gpu_util import check_select_and_attend
    gc = _gc(small_bf16([1000, 333], tail_fill=float("nan"), seed=5))
    check_select_and_attend(gc, gc.oracle_summaries(), out_tol=2e-2)


@pytest.mark.parametrize("rank", [2, 4])
def test_i4_generic_ranks(rank):
    from gpu_util import check_select_and_attend
    gc = _gc(small_bf16([1200, 800], rank=rank, seed=rank))
    check_select_and_attend(gc, gc.oracle_summaries(), out_tol=2e-2)


@pytest.mark.parametrize("rank", [2, 8])
def test_i4_summaries_with_fp32_queries(rank):
    """Quantised summaries with fp32 K, V and q: the plain fp32-arithmetic scan and attention paths."""
    from gpu_util import check_select_and_attend
    gc = _gc(small_bf16([1000, 700], rank=rank, seed=40 + rank, dtype="f32"))
    check_select_and_attend(gc, gc.oracle_summaries(), out_tol=1e-4)


@pytest.mark.parametrize("Hq,Hkv", [(12, 2), (32, 2)])
def test_i4_rank2_group_sizes(Hq, Hkv):
    """Rank-2 summaries through the tensor-core scan at group sizes 6 and 16."""
    from gpu_util import check_select_and_attend
    gc = _gc(small_bf16([1500, 900], Hq=Hq, Hkv=Hkv, rank=2, seed=50 + Hq))
    check_select_and_attend(gc, gc.oracle_summaries(), out_tol=2e-2)


@pytest.mark.parametrize("trial", range(24))
def test_randomized_shapes(trial):
    """Seeded random shapes: group size, rank, budget, request count, lengths (with ragged tails and requests
    shorter than the budget), block layout, carriers, scan partition.  Twice per case: the second call must
    reproduce the first (no state left behind in the workspace)."""
    from gpu_util import check_select_and_attend
    rng = np.random.default_rng(1000 + trial)
    Hkv = int(rng.choice([1, 2, 4]))
    G = int(rng.choice([1, 2, 3, 4, 5, 7, 8, 12, 16]))
    rank = int(rng.choice([2, 4, 8]))
    budget = int(rng.choice([32, 64, 256, 512, 1024]))
    n = int(rng.integers(1, 4))
    lens = [int(rng.integers(1, 6000)) for _ in range(n)]
    if trial % 3 == 0:
        lens[0] = int(rng.integers(9000, 30000))      # one long request
    w = small_bf16(lens, Hq=G * Hkv, Hkv=Hkv, rank=rank, budget=budget, seed=2000 + trial,
                   layout="NHD" if trial % 4 == 1 else "HND", carriers=int(rng.choice([0, 0, 4])),
                   q_scale=float(rng.choice([1.0, 0.25])))
    gc = _gc(w)
    if trial % 2:   # odd trials force the scan's balanced page partition (even ones: strided, the default here)
        gc.ctx.locks_set_scan_partition(locks.PARTITION_BALANCED)
    summ = gc.oracle_summaries()
    check_select_and_attend(gc, summ, out_tol=2e-2)
    ids1, cnt1, lm1, ls1 = gc.gpu_select(torch.from_numpy(summ).cuda())
    ids2, cnt2, lm2, ls2 = gc.gpu_select(torch.from_numpy(summ).cuda())
    assert np.array_equal(ids1, ids2) and np.array_equal(cnt1, cnt2)
    assert gc.status() == 0


@pytest.mark.parametrize("Hq,Hkv,rank", [(8, 2, 8), (16, 2, 8), (32, 2, 8), (8, 2, 2), (8, 2, 4), (12, 2, 2)])
def test_balanced_partition_ragged_batch(Hq, Hkv, rank):
    """The scan's balanced partition (equal page ranges per warp) on a batch of very different lengths:
    warps that start inside a problem, warps that span several problems, requests shorter than the
    budget (no candidates) and a one-page request.  Scores, shares, sets and outputs against the oracle,
    and the same selection as the strided partition."""
    from gpu_util import check_select_and_attend
    lens = [16 * 700 + 5, 40, 16 * 90, 16 * 2300 + 9, 7, 16 * 300 + 1, 16 * 41]
    w = small_bf16(lens, Hq=Hq, Hkv=Hkv, rank=rank, budget=256, seed=300 + Hq + rank)
    gc = _gc(w)
    summ = gc.oracle_summaries()
    dsumm = torch.from_numpy(summ).cuda()
    gc.ctx.locks_set_scan_partition(locks.PARTITION_STRIDED)
    ids_s, cnt_s, lm_s, ls_s = gc.gpu_select(dsumm)
    gc.ctx.locks_set_scan_partition(locks.PARTITION_BALANCED)
    check_select_and_attend(gc, summ, out_tol=2e-2)
    ids_b, cnt_b, lm_b, ls_b = gc.gpu_select(dsumm)
    assert np.array_equal(cnt_s, cnt_b)
    for b, T in enumerate(lens):
        P = -(-T // 16)
        if P > gc.k:   # same scores bit for bit (the partition only changes who computes them)
            assert np.array_equal(lm_s[b, :, :P - 1], lm_b[b, :, :P - 1])
            assert np.abs(ls_s[b, :, 1:P - 1] - ls_b[b, :, 1:P - 1]).max() <= 1e-5
    assert gc.status() == 0


def test_balanced_partition_few_problems_of_very_different_lengths():
    """Two requests, two KV heads, G = 16 (the geometry that otherwise merges partials per CTA), one request
    40 times longer than the other: hundreds of log Z partials per head in the balanced partition."""
    from gpu_util import check_select_and_attend
    w = locks_synth.Workload("few-ragged", [16 * 6000 + 7, 16 * 150], Hq=32, Hkv=2, budget=512, seed=83)
    gc = _gc(w)
    gc.ctx.locks_set_scan_partition(locks.PARTITION_BALANCED)
    check_select_and_attend(gc, gc.oracle_summaries(), out_tol=2e-2)


def test_balanced_partition_more_problems_than_warps_per_problem():
    """Balanced partition with many short problems: most warps cross several problem boundaries."""
    from gpu_util import check_select_and_attend
    rng = np.random.default_rng(77)
    lens = [int(rng.integers(16 * 20, 16 * 60)) for _ in range(48)]
    w = small_bf16(lens, Hq=8, Hkv=4, rank=8, budget=128, seed=78)
    gc = _gc(w)
    gc.ctx.locks_set_scan_partition(locks.PARTITION_BALANCED)
    check_select_and_attend(gc, gc.oracle_summaries(), out_tol=2e-2)


def test_partition_suggestion_follows_lengths():
    """Decode steps leave a suggestion for the scan's partition: ragged lengths turn the balanced one on
    for the following calls, and the step's results do not depend on it."""
    from common import check_page_sets, oracle_cache
    lens = [16 * 9000, 16 * 150, 16 * 200, 16 * 120, 16 * 180]   # 10 problems, one 50 times longer
    w = small_bf16([t + 16 for t in lens], Hq=8, Hkv=2, rank=8, budget=256, seed=91)
    gc = _gc(w)
    gc.case.seq_lens.copy_(torch.tensor(lens, dtype=torch.int32, device="cuda:0"))
    summ = gc.ctx.new_summaries(gc.case.num_blocks)
    gc.ctx.locks_build_summaries(gc.kv, w.n, summ)
    out = torch.empty(w.n, w.Hq, w.d, dtype=torch.bfloat16, device="cuda:0")
    ids = torch.empty(w.n, w.Hkv, gc.k, dtype=torch.int32, device="cuda:0")
    cnt = torch.empty(w.n, w.Hkv, dtype=torch.int32, device="cuda:0")
    for step in range(3):   # step 0 runs strided (no suggestion yet), the later ones balanced
        kn, vn, qn = locks_synth.new_token(w, step, device="cuda:0")
        gc.ctx.locks_decode_step(qn, kn, vn, gc.kv, summ, w.n, out, ids, cnt)
        torch.cuda.synchronize()
        assert gc.status() == 0
        cache = oracle_cache(gc.case)
        shat = oracle.page_logmass(cache, t2np(qn), w.rank, gc.fmt, summ.cpu().numpy(), gc.sm)
        oids, ocnt, ols = oracle.select(cache, shat, gc.k)
        check_page_sets(ids.cpu().numpy(), cnt.cpu().numpy(), oids, ocnt, ols, cache.seq_lens, w.B, gc.k)
        oout, _ = oracle.attend(cache, t2np(qn), gc.sm, ids.cpu().numpy(), cnt.cpu().numpy())
        assert np.abs(out.float().cpu().numpy() - oout).max() <= 2e-2, step


def test_two_level_select_long_context():
    """Several chunks per KV head: per-chunk lists, then the last chunk to arrive ranks the survivors."""
    from gpu_util import check_select_and_attend
    gc = _gc(locks_synth.Workload("long", [16 * 9000 + 3], Hq=32, Hkv=2, budget=2048, seed=9))
    differed = check_select_and_attend(gc, gc.oracle_summaries(), out_tol=2e-2)
    assert differed <= 1


@pytest.mark.parametrize("lens,Hq,Hkv,rank,budget", [([16 * 3000 + 3, 16 * 700], 8, 2, 8, 4096),
                                                     ([16 * 9000], 32, 2, 8, 8192),
                                                     ([16 * 2000, 16 * 2500 + 9, 900], 16, 4, 2, 16384)])
def test_large_budgets(lens, Hq, Hkv, rank, budget):
    """Budgets of 256 to 1024 pages: long candidate lists per chunk, many winners to compact, long attention."""
    from gpu_util import check_select_and_attend
    gc = _gc(locks_synth.Workload("big-budget", lens, Hq=Hq, Hkv=Hkv, rank=rank, budget=budget, seed=5))
    check_select_and_attend(gc, gc.oracle_summaries(), out_tol=2e-2)


def test_ties_resolve_to_lower_index():
    """All keys identical and a zero query: every candidate ties, the lowest indices win."""
    gc = _gc(small_bf16([16 * 40], Hq=4, Hkv=1, budget=128))
    gc.case.k.fill_(0.5)
    gc.case.q.zero_()
    from gpu_util import GpuCase
    gc.cache = __import__("common").oracle_cache(gc.case)
    summ = gc.oracle_summaries()
    ids, cnt, _, _ = gc.gpu_select(torch.from_numpy(summ).cuda())
    assert cnt[0, 0] == 8 and ids[0, 0].tolist() == [0, 1, 2, 3, 4, 5, 6, 39]


@pytest.mark.parametrize("pages", [5000, 18500])
def test_ties_across_chunks(pages):
    """Every candidate ties and the problem spans several chunks: all list entries survive the
    threshold (at 18500 pages more than the final round holds in shared memory, so it ranks them in
    place); the lowest page indices must still win."""
    gc = _gc(small_bf16([16 * pages + 5], Hq=4, Hkv=1, budget=2048))
    gc.case.k.fill_(0.5)
    gc.case.q.zero_()
    gc.cache = __import__("common").oracle_cache(gc.case)
    summ = gc.oracle_summaries()
    ids, cnt, _, _ = gc.gpu_select(torch.from_numpy(summ).cuda())
    assert cnt[0, 0] == 128 and ids[0, 0].tolist() == list(range(127)) + [pages]


@pytest.mark.parametrize("rank", [2, 4, 8])
def test_gpu_i4_build_decoupled_parity(rank):
    """I4 build (ranks 2, 4 and 8): codes agree with the oracle's on >= 99.9 % of entries (|diff| <= 1 elsewhere) after sign
    alignment, the stored scales are the fp16 abs-max scales of the blob's own values, probe scores stay
    close.  The sign of a mode (largest-magnitude basis entry positive) is a determinism convention: the score
    only sees the products of a basis vector with its coefficients, and the rule is decided by a comparison
    of two magnitudes that fp32 and fp64 can order differently when they are within a code of each other.
    Such a joint flip of (basis row, coefficient column) is accepted only at a near-tie and must stay rare."""
    gc = _gc(small_bf16([16 * 600], Hq=8, Hkv=2, rank=rank, seed=21))
    w = gc.w
    g_summ = gc.gpu_build().cpu().numpy()
    o_summ = gc.oracle_summaries()
    rng = np.random.default_rng(1)
    bt = gc.cache.block_table[0]
    tot = diff = flips = 0
    worst = 0.0
    for p in range(600):
        for h in range(2):
            gV, gC, gMu, gsV, gsC, gsMu = oracle.unpack_codes(rank, g_summ[bt[p], h])
            oV, oC, oMu, osV, osC, osMu = oracle.unpack_codes(rank, o_summ[bt[p], h])
            for l in range(rank):
                if int(np.dot(gV[l], oV[l])) < 0:
                    top = np.sort(np.abs(oV[l]))[-2:]
                    assert top[1] - top[0] <= 1, (p, h, l, top)
                    gV[l] = -gV[l]
                    gC[:, l] = -gC[:, l]
                    flips += 1
            for a, b_ in ((gV, oV), (gC, oC), (gMu, oMu)):
                d = np.abs(a - b_)
                assert d.max() <= 1
                tot += d.size; diff += int((d > 0).sum())
            assert np.all(np.abs(gsV - osV) <= np.spacing(np.float16(osV)).astype(np.float64) + 0)
            assert np.all(np.abs(gsC - osC) <= np.spacing(np.float16(osC)).astype(np.float64) + 0)
            assert abs(gsMu - osMu) <= float(np.spacing(np.float16(osMu)))
            if p % 10 == 0:
                mg = oracle.unpack(oracle.FMT_I4, rank, g_summ[bt[p], h])
                mo = oracle.unpack(oracle.FMT_I4, rank, o_summ[bt[p], h])
                q = rng.standard_normal(128)
                worst = max(worst, abs(oracle.score(*mg, q, gc.sm) - oracle.score(*mo, q, gc.sm)))
    assert diff / tot <= 1e-3, diff / tot
    assert flips <= 2, flips   # of 1200 * rank modes
    assert worst <= 5e-3, worst
    assert gc.status() == 0


def test_multi_layer_build_in_one_launch():
    """locks_build_summaries_layers: three layers with different keys (same block table and lengths) in one launch.
    Every layer's blobs equal, byte for byte, what the single-layer call writes for that layer, and one layer's codes
    are checked against the oracle's build of that layer's keys (sign-aligned code agreement, as in the decoupled
    test); pages outside the requested range and the blocks of other layers are not touched."""
    gc = _gc(small_bf16([16 * 70 + 3, 16 * 33], Hq=8, Hkv=2, seed=91))
    w = gc.w
    g = torch.Generator(device="cuda:0").manual_seed(5)
    k_layers = [gc.case.k] + [(gc.case.k.float() * s + torch.randn(gc.case.k.shape, generator=g, device="cuda:0") * 0.5)
                              .to(gc.case.k.dtype) for s in (0.5, -1.25)]
    singles = []
    from paper_2607_24555_b200.binding import KVView
    for kl in k_layers:
        kv = KVView(kl, gc.case.v, gc.case.strides, gc.case.num_blocks, gc.case.block_table, gc.case.seq_lens)
        summ = gc.ctx.new_summaries(gc.case.num_blocks)
        summ.fill_(0x5A)
        gc.ctx.locks_build_summaries(kv, w.n, summ)
        singles.append(summ)
    multi = [gc.ctx.new_summaries(gc.case.num_blocks) for _ in k_layers]
    for m in multi:
        m.fill_(0x5A)
    keep = gc.ctx.locks_build_summaries_layers(gc.kv, k_layers, multi, w.n)
    torch.cuda.synchronize()
    assert keep is not None and gc.status() == 0
    for l in range(len(k_layers)):
        assert torch.equal(multi[l], singles[l]), l
    # layer 2 against the oracle's build of the same keys
    import copy
    from common import oracle_cache
    case2 = copy.copy(gc.case)
    case2.k = k_layers[2]
    o_summ = oracle.build_summaries(oracle_cache(case2), w.rank, gc.fmt)
    g_summ = multi[2].cpu().numpy()
    tot = diff = 0
    for b in range(w.n):
        bt = gc.cache.block_table[b]
        for p in range(w.seq_lens[b] // 16):
            for h in range(w.Hkv):
                gV, gC, gMu, _, _, _ = oracle.unpack_codes(w.rank, g_summ[bt[p], h])
                oV, oC, oMu, _, _, _ = oracle.unpack_codes(w.rank, o_summ[bt[p], h])
                for l in range(w.rank):
                    if int(np.dot(gV[l], oV[l])) < 0:
                        gV[l] = -gV[l]; gC[:, l] = -gC[:, l]
                for a_, b_ in ((gV, oV), (gC, oC), (gMu, oMu)):
                    d = np.abs(a_ - b_)
                    assert d.max() <= 1
                    tot += d.size; diff += int((d > 0).sum())
    assert diff / tot <= 1e-3, diff / tot
    # a page range: only pages 2..4 of every request are rebuilt
    pb = torch.full((w.n,), 2, dtype=torch.int32, device="cuda:0")
    pe = torch.full((w.n,), 5, dtype=torch.int32, device="cuda:0")
    part = [torch.full_like(m, 0x5A) for m in multi]
    keep2 = gc.ctx.locks_build_summaries_layers(gc.kv, k_layers, part, w.n, pb, pe)
    torch.cuda.synchronize()
    assert keep2 is not None
    bt_all = gc.case.block_table.cpu().numpy()
    touched = sorted({int(bt_all[b, p]) for b in range(w.n) for p in range(2, 5)})
    for l in range(len(k_layers)):
        pl, ml = part[l].cpu().numpy(), multi[l].cpu().numpy()
        for blk in range(gc.case.num_blocks):
            if blk in touched:
                assert np.array_equal(pl[blk], ml[blk]), (l, blk)
            else:
                assert (pl[blk] == 0x5A).all(), (l, blk)


def test_decode_step_matches_stepwise_oracle():
    """locks_decode_step with appends across page boundaries; summaries of freshly filled pages
    are built on the device and handed to the oracle (identical bytes) for the next steps."""
    from common import check_page_sets, oracle_cache
    w = small_bf16([16 * 130 - 3, 16 * 90 + 14, 500], Hq=8, Hkv=2, budget=256, spare_blocks=0, seed=33)
    reserve = 3
    w = w.with_(seq_lens=[t + 16 * reserve for t in w.seq_lens])     # room to grow
    gc = _gc(w)
    start = torch.tensor([t - 16 * reserve for t in w.seq_lens], dtype=torch.int32, device="cuda:0")
    gc.case.seq_lens.copy_(start)
    summ = gc.ctx.new_summaries(gc.case.num_blocks)
    gc.ctx.locks_build_summaries(gc.kv, w.n, summ)
    out = torch.empty(w.n, w.Hq, w.d, dtype=torch.bfloat16, device="cuda:0")
    ids = torch.empty(w.n, w.Hkv, gc.k, dtype=torch.int32, device="cuda:0")
    cnt = torch.empty(w.n, w.Hkv, dtype=torch.int32, device="cuda:0")
    for step in range(36):
        kn, vn, qn = locks_synth.new_token(w, step, device="cuda:0")
        gc.ctx.locks_decode_step(qn, kn, vn, gc.kv, summ, w.n, out, ids, cnt)
        torch.cuda.synchronize()
        assert gc.status() == 0
        assert gc.case.seq_lens.cpu().tolist() == [int(s) + step + 1 for s in start.cpu()]
        cache = oracle_cache(gc.case)                               # cache now holds the new token
        summ_np = summ.cpu().numpy()
        shat = oracle.page_logmass(cache, t2np(qn), w.rank, gc.fmt, summ_np, gc.sm)
        oids, ocnt, ols = oracle.select(cache, shat, gc.k)
        check_page_sets(ids.cpu().numpy(), cnt.cpu().numpy(), oids, ocnt, ols, cache.seq_lens, w.B, gc.k)
        oout, _ = oracle.attend(cache, t2np(qn), gc.sm, ids.cpu().numpy(), cnt.cpu().numpy())
        assert np.abs(out.float().cpu().numpy() - oout).max() <= 2e-2, step
        # a page that just filled has a summary now, equal in quality to the bulk build
        for b in range(w.n):
            T = int(cache.seq_lens[b])
            if T % 16 == 0:
                blk = cache.block_table[b, T // 16 - 1]
                ref = oracle.build_summaries(cache, w.rank, gc.fmt, page_begin=[T // 16 - 1 if i == b else 0 for i in range(w.n)],
                                             page_end=[T // 16 if i == b else 0 for i in range(w.n)])
                for h in range(w.Hkv):
                    gV, gC, gMu, _, _, _ = oracle.unpack_codes(8, summ_np[blk, h])
                    oV, oC, oMu, _, _, _ = oracle.unpack_codes(8, ref[blk, h])
                    for l in range(8):   # a mode's joint sign is a convention decided at a near-tie (see the build test)
                        if int(np.dot(gV[l], oV[l])) < 0:
                            gV[l] = -gV[l]; gC[:, l] = -gC[:, l]
                    assert np.abs(gV - oV).max() <= 1 and np.abs(gC - oC).max() <= 1 and np.abs(gMu - oMu).max() <= 1


def test_decode_step_long_context_few_problems():
    """Decode steps on one long request (several selector chunks per KV head, cluster-merged attention,
    G = 16): the token is appended by the selector's first chunk, and a page fills on the way."""
    from common import check_page_sets, oracle_cache
    T0 = 16 * 4000 + 14
    w = locks_synth.Workload("long-step", [T0 + 16], Hq=32, Hkv=2, budget=1024, seed=61)
    gc = _gc(w)
    gc.case.seq_lens.fill_(T0)
    summ = gc.ctx.new_summaries(gc.case.num_blocks)
    gc.ctx.locks_build_summaries(gc.kv, w.n, summ)
    out = torch.empty(w.n, w.Hq, w.d, dtype=torch.bfloat16, device="cuda:0")
    ids = torch.empty(w.n, w.Hkv, gc.k, dtype=torch.int32, device="cuda:0")
    cnt = torch.empty(w.n, w.Hkv, dtype=torch.int32, device="cuda:0")
    for step in range(3):
        kn, vn, qn = locks_synth.new_token(w, step, device="cuda:0")
        gc.ctx.locks_decode_step(qn, kn, vn, gc.kv, summ, w.n, out, ids, cnt)
        torch.cuda.synchronize()
        assert gc.status() == 0
        assert gc.case.seq_lens.cpu().tolist() == [T0 + step + 1]
        cache = oracle_cache(gc.case)
        shat = oracle.page_logmass(cache, t2np(qn), w.rank, gc.fmt, summ.cpu().numpy(), gc.sm)
        oids, ocnt, ols = oracle.select(cache, shat, gc.k)
        check_page_sets(ids.cpu().numpy(), cnt.cpu().numpy(), oids, ocnt, ols, cache.seq_lens, w.B, gc.k)
        oout, _ = oracle.attend(cache, t2np(qn), gc.sm, ids.cpu().numpy(), cnt.cpu().numpy())
        assert np.abs(out.float().cpu().numpy() - oout).max() <= 2e-2, step


def test_decode_step_graph_replay_against_stepwise_oracle():
    """The whole step captured ONCE in a CUDA graph and replayed 56 times on three ragged requests (every one
    crosses three or four page boundaries; one starts shorter than the budget and outgrows it on the way): after
    every replay the lengths, the page sets and the outputs are checked against the oracle stepping the same
    state, and the summaries of freshly filled pages (built inside the graph) against the oracle's build."""
    from common import check_page_sets, oracle_cache
    steps, reserve = 56, 5
    start_lens = [16 * 130 - 3, 16 * 90 + 14, 16 * 15 + 9]          # k = 16 pages: the last request starts dense
    w = small_bf16([t + 16 * reserve for t in start_lens], Hq=8, Hkv=2, budget=256, seed=35)
    gc = _gc(w)
    start = torch.tensor(start_lens, dtype=torch.int32, device="cuda:0")
    gc.case.seq_lens.copy_(start)
    summ = gc.ctx.new_summaries(gc.case.num_blocks)
    gc.ctx.locks_build_summaries(gc.kv, w.n, summ)
    out = torch.empty(w.n, w.Hq, w.d, dtype=torch.bfloat16, device="cuda:0")
    ids = torch.empty(w.n, w.Hkv, gc.k, dtype=torch.int32, device="cuda:0")
    cnt = torch.empty(w.n, w.Hkv, dtype=torch.int32, device="cuda:0")
    kn, vn, qn = [t.clone() for t in locks_synth.new_token(w, 0, device="cuda:0")]
    s = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        gc.ctx.locks_decode_step(qn, kn, vn, gc.kv, summ, w.n, out, ids, cnt, stream=s)   # warm-up, then rewind
        s.synchronize()
        gc.case.seq_lens.copy_(start)
        with torch.cuda.graph(g, stream=s):
            gc.ctx.locks_decode_step(qn, kn, vn, gc.kv, summ, w.n, out, ids, cnt, stream=s)
    torch.cuda.synchronize()
    crossings = [0] * w.n
    for step in range(steps):
        a, b_, c = locks_synth.new_token(w, step, device="cuda:0")
        kn.copy_(a); vn.copy_(b_); qn.copy_(c)
        g.replay()
        torch.cuda.synchronize()
        assert gc.status() == 0
        assert gc.case.seq_lens.cpu().tolist() == [t + step + 1 for t in start_lens]
        cache = oracle_cache(gc.case)
        summ_np = summ.cpu().numpy()
        shat = oracle.page_logmass(cache, t2np(qn), w.rank, gc.fmt, summ_np, gc.sm)
        oids, ocnt, ols = oracle.select(cache, shat, gc.k)
        check_page_sets(ids.cpu().numpy(), cnt.cpu().numpy(), oids, ocnt, ols, cache.seq_lens, w.B, gc.k)
        oout, _ = oracle.attend(cache, t2np(qn), gc.sm, ids.cpu().numpy(), cnt.cpu().numpy())
        assert np.abs(out.float().cpu().numpy() - oout).max() <= 2e-2, step
        for b in range(w.n):
            T = int(cache.seq_lens[b])
            if T % 16 == 0:
                crossings[b] += 1
                blk = cache.block_table[b, T // 16 - 1]
                ref = oracle.build_summaries(cache, w.rank, gc.fmt, page_begin=[T // 16 - 1 if i == b else 0 for i in range(w.n)],
                                             page_end=[T // 16 if i == b else 0 for i in range(w.n)])
                for h in range(w.Hkv):
                    gV, gC, gMu, _, _, _ = oracle.unpack_codes(8, summ_np[blk, h])
                    oV, oC, oMu, _, _, _ = oracle.unpack_codes(8, ref[blk, h])
                    for l in range(8):
                        if int(np.dot(gV[l], oV[l])) < 0:
                            gV[l] = -gV[l]; gC[:, l] = -gC[:, l]
                    assert np.abs(gV - oV).max() <= 1 and np.abs(gC - oC).max() <= 1 and np.abs(gMu - oMu).max() <= 1
    assert min(crossings) >= 3, crossings


def test_decode_step_graph_replay_equals_eager():
    """The step is captured once in a CUDA graph and replayed as the sequences grow."""
    w = small_bf16([16 * 100 + 9, 16 * 70], Hq=8, Hkv=2, budget=256, seed=44)
    w = w.with_(seq_lens=[t + 64 for t in w.seq_lens])
    res = []
    for mode in ("eager", "graph"):
        gc = _gc(w)
        gc.case.seq_lens.copy_(torch.tensor([t - 64 for t in w.seq_lens], dtype=torch.int32, device="cuda:0"))
        summ = gc.ctx.new_summaries(gc.case.num_blocks)
        gc.ctx.locks_build_summaries(gc.kv, w.n, summ)
        out = torch.empty(w.n, w.Hq, w.d, dtype=torch.bfloat16, device="cuda:0")
        kn, vn, qn = [t.clone() for t in locks_synth.new_token(w, 0, device="cuda:0")]
        outs = []
        if mode == "graph":
            s = torch.cuda.Stream()
            g = torch.cuda.CUDAGraph()
            s.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(s):
                # warm up outside capture on a scratch copy of the lengths
                saved = gc.case.seq_lens.clone()
                gc.ctx.locks_decode_step(qn, kn, vn, gc.kv, summ, w.n, out, stream=s)
                s.synchronize()
                gc.case.seq_lens.copy_(saved)
                with torch.cuda.graph(g, stream=s):
                    gc.ctx.locks_decode_step(qn, kn, vn, gc.kv, summ, w.n, out, stream=s)
            torch.cuda.synchronize()
        for step in range(20):
            a, b_, c = locks_synth.new_token(w, step, device="cuda:0")
            kn.copy_(a); vn.copy_(b_); qn.copy_(c)
            if mode == "graph":
                g.replay()
            else:
                gc.ctx.locks_decode_step(qn, kn, vn, gc.kv, summ, w.n, out)
            torch.cuda.synchronize()
            outs.append(out.float().cpu().numpy().copy())
        assert gc.status() == 0
        res.append((outs, gc.case.seq_lens.cpu().tolist()))
    assert res[0][1] == res[1][1]
    for a, b_ in zip(res[0][0], res[1][0]):
        assert np.array_equal(a, b_)


def test_decode_step_host_entry_point():
    w = small_bf16([16 * 50 + 5, 900], Hq=8, Hkv=2, budget=128, seed=55)
    gc = _gc(w)
    summ = gc.gpu_build()
    q_host = gc.case.q.cpu().pin_memory()
    out_host = torch.empty(w.n, w.Hq, w.d, dtype=torch.bfloat16).pin_memory()
    ids_host = torch.empty(w.n, w.Hkv, gc.k, dtype=torch.int32).pin_memory()
    cnt_host = torch.empty(w.n, w.Hkv, dtype=torch.int32).pin_memory()
    gc.ctx.locks_decode_step_host(q_host, None, None, gc.kv, summ, w.n, out_host, ids_host, cnt_host)
    out = torch.empty(w.n, w.Hq, w.d, dtype=torch.bfloat16, device="cuda:0")
    ids = torch.empty(w.n, w.Hkv, gc.k, dtype=torch.int32, device="cuda:0")
    cnt = torch.empty(w.n, w.Hkv, dtype=torch.int32, device="cuda:0")
    gc.ctx.locks_decode_step(gc.case.q, None, None, gc.kv, summ, w.n, out, ids, cnt)
    torch.cuda.synchronize()
    assert torch.equal(out.cpu(), out_host) and torch.equal(ids.cpu(), ids_host) and torch.equal(cnt.cpu(), cnt_host)


def test_decode_step_host_repeated_calls_match_device_steps():
    """Repeated host-buffer steps with fixed buffers (from the second repetition on the library replays a
    cached graph): each call appends its token and returns what the device entry point returns on a twin."""
    w = small_bf16([16 * 60 + 13, 700], Hq=8, Hkv=2, budget=128, seed=57)
    reserve = 2
    w = w.with_(seq_lens=[t + 16 * reserve for t in w.seq_lens])
    gc_h, gc_d = _gc(w), _gc(w)
    start = torch.tensor([t - 16 * reserve for t in w.seq_lens], dtype=torch.int32, device="cuda:0")
    outs = []
    for gc in (gc_h, gc_d):
        gc.case.seq_lens.copy_(start)
    summ_h = gc_h.ctx.new_summaries(gc_h.case.num_blocks)
    summ_d = gc_d.ctx.new_summaries(gc_d.case.num_blocks)
    gc_h.ctx.locks_build_summaries(gc_h.kv, w.n, summ_h)
    gc_d.ctx.locks_build_summaries(gc_d.kv, w.n, summ_d)
    qh = torch.empty(w.n, w.Hq, w.d, dtype=torch.bfloat16).pin_memory()
    kh = torch.empty(w.n, w.Hkv, w.d, dtype=torch.bfloat16).pin_memory()
    vh = torch.empty(w.n, w.Hkv, w.d, dtype=torch.bfloat16).pin_memory()
    out_host = torch.empty(w.n, w.Hq, w.d, dtype=torch.bfloat16).pin_memory()
    ids_host = torch.empty(w.n, w.Hkv, gc_h.k, dtype=torch.int32).pin_memory()
    cnt_host = torch.empty(w.n, w.Hkv, dtype=torch.int32).pin_memory()
    out = torch.empty(w.n, w.Hq, w.d, dtype=torch.bfloat16, device="cuda:0")
    ids = torch.empty(w.n, w.Hkv, gc_d.k, dtype=torch.int32, device="cuda:0")
    cnt = torch.empty(w.n, w.Hkv, dtype=torch.int32, device="cuda:0")
    for step in range(20):   # crosses a page boundary of both requests
        kn, vn, qn = locks_synth.new_token(w, step, device="cuda:0")
        qh.copy_(qn.cpu()); kh.copy_(kn.cpu()); vh.copy_(vn.cpu())
        gc_h.ctx.locks_decode_step_host(qh, kh, vh, gc_h.kv, summ_h, w.n, out_host, ids_host, cnt_host)
        gc_d.ctx.locks_decode_step(qn, kn, vn, gc_d.kv, summ_d, w.n, out, ids, cnt)
        torch.cuda.synchronize()
        assert torch.equal(gc_h.case.seq_lens, gc_d.case.seq_lens)
        assert torch.equal(ids.cpu(), ids_host) and torch.equal(cnt.cpu(), cnt_host), step
        assert torch.equal(out.cpu(), out_host), step
    assert torch.equal(summ_h, summ_d)
    assert gc_h.status() == 0 and gc_d.status() == 0


def test_decode_step_host_pageable_buffers_take_the_copy_path():
    """Host buffers that are not page-locked cannot be read by the staging kernel or written by the attention
    kernel: the call falls back to plain copies and returns the same results as with page-locked buffers."""
    w = small_bf16([16 * 40 + 5, 300], Hq=8, Hkv=2, budget=128, seed=58)
    w = w.with_(seq_lens=[t + 32 for t in w.seq_lens])
    res = []
    for pinned in (True, False):
        gc = _gc(w)
        gc.case.seq_lens.copy_(torch.tensor([t - 32 for t in w.seq_lens], dtype=torch.int32, device="cuda:0"))
        summ = gc.ctx.new_summaries(gc.case.num_blocks)
        gc.ctx.locks_build_summaries(gc.kv, w.n, summ)
        mk = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
        out_host = mk(torch.empty(w.n, w.Hq, w.d, dtype=torch.bfloat16))
        ids_host = mk(torch.empty(w.n, w.Hkv, gc.k, dtype=torch.int32))
        cnt_host = mk(torch.empty(w.n, w.Hkv, dtype=torch.int32))
        got = []
        for step in range(4):
            kn, vn, qn = locks_synth.new_token(w, step, device="cuda:0")
            gc.ctx.locks_decode_step_host(mk(qn.cpu()), mk(kn.cpu()), mk(vn.cpu()), gc.kv, summ, w.n, out_host, ids_host,
                                          cnt_host)
            got.append((out_host.clone(), ids_host.clone(), cnt_host.clone()))
        assert gc.status() == 0
        res.append(got)
    for (o1, i1, c1), (o2, i2, c2) in zip(*res):
        assert torch.equal(o1, o2) and torch.equal(i1, i2) and torch.equal(c1, c2)


def test_scan_partition_setter_rejects_unknown_modes():
    gc = _gc(small_bf16([16 * 20], Hq=8, Hkv=2, budget=128))
    for mode in (locks.PARTITION_AUTO, locks.PARTITION_STRIDED, locks.PARTITION_BALANCED):
        gc.ctx.locks_set_scan_partition(mode)
    for mode in (-1, 3):
        with pytest.raises(locks.LocksError):
            gc.ctx.locks_set_scan_partition(mode)


def test_bounded_wait_runs_out_and_reports():
    """Host-visible outcome of a device-side wait that nothing completes: the kernel gives up after its limit,
    the status word says LOCKS_ERR_TIMEOUT (-5), and the context keeps working."""
    import time
    gc = _gc(small_bf16([16 * 40], Hq=8, Hkv=2, budget=128, seed=67))
    summ = gc.gpu_build()
    ids0, cnt0, _, _ = gc.gpu_select(summ)
    t0 = time.perf_counter()
    gc.ctx.locks_selftest_wait_timeout(50)
    assert gc.status() == -5                      # polling synchronises and clears
    assert time.perf_counter() - t0 < 2.0        # 50 ms limit, not the one-second default nor the poll count
    assert gc.status() == 0
    ids1, cnt1, _, _ = gc.gpu_select(summ)       # the context is as usable as before
    assert np.array_equal(ids0, ids1) and np.array_equal(cnt0, cnt1)
    with pytest.raises(locks.LocksError):
        gc.ctx.locks_selftest_wait_timeout(0)


def test_bad_block_id_sets_status_without_faulting():
    """Host-injected fault: a block id outside the cache is skipped and reported, nothing traps."""
    gc = _gc(small_bf16([16 * 60], Hq=8, Hkv=2, budget=128, seed=66))
    summ = gc.gpu_build()
    gc.case.block_table[0, 7] = gc.case.num_blocks + 5
    gc.gpu_select(summ)
    assert gc.status() == -6
    assert gc.status() == 0                                          # polling clears it


def test_page_count_beyond_the_table_row_is_clamped_and_reported():
    """Host-injected fault: a page_count larger than k would index past the row of page ids; the kernels use
    the row's k entries, skip nothing else, and report LOCKS_ERR_BAD_BLOCK."""
    gc = _gc(small_bf16([16 * 200, 16 * 120], Hq=8, Hkv=2, budget=128, seed=68))
    summ = gc.gpu_build()
    ids, cnt, _, _ = gc.gpu_select(summ)
    ref, ref_lse = gc.gpu_attend(ids, cnt)
    assert gc.status() == 0
    bad = cnt.copy()
    bad[1, 1] = gc.k + 3
    bad[0, 0] = -2                                    # a negative count attends nothing: rows of that head are zero
    out, lse = gc.gpu_attend(ids, bad)
    assert gc.status() == -6
    assert np.array_equal(out[1], ref[1]) and np.array_equal(out[0, 4:], ref[0, 4:])
    assert not np.isnan(out).any()


def test_host_cache_clear_and_partition_report():
    """The host entry point caches a graph per argument set; locks_host_cache_clear drops them (a caller does
    that before freeing its pinned buffers) and later calls still give the same results.  The partition the
    scan used is reported, and pinning another mode drops the cached graphs too."""
    w = small_bf16([16 * 80 + 5, 900], Hq=8, Hkv=2, budget=128, seed=59)
    gc = _gc(w)
    summ = gc.gpu_build()
    q_host = gc.case.q.cpu().pin_memory()
    outs = []
    for rep in range(8):
        if rep == 4:
            gc.ctx.locks_host_cache_clear()
        if rep == 6:
            gc.ctx.locks_set_scan_partition(locks.PARTITION_BALANCED)
        out_host = torch.empty(w.n, w.Hq, w.d, dtype=torch.bfloat16).pin_memory() if rep in (0, 4) else out_host
        gc.ctx.locks_decode_step_host(q_host, None, None, gc.kv, summ, w.n, out_host)
        outs.append(out_host.clone())
        assert gc.ctx.locks_last_scan_partition() == (locks.PARTITION_BALANCED if rep >= 6 else locks.PARTITION_STRIDED)
    for o in outs[1:]:
        assert torch.equal(o, outs[0])
    assert gc.status() == 0


def test_fresh_context_after_set_device():
    """Kernel attributes are kept per device: a second context, created after the device has been selected
    again, launches every kernel with its attributes in place (large dynamic shared memory, clusters)."""
    from gpu_util import check_select_and_attend
    torch.cuda.set_device(0)
    a = _gc(small_bf16([16 * 300 + 3], Hq=8, Hkv=2, budget=256, seed=70))
    check_select_and_attend(a, a.oracle_summaries(), out_tol=2e-2)
    torch.cuda.set_device(0)
    b = _gc(small_bf16([16 * 500 + 3, 16 * 20], Hq=32, Hkv=2, budget=256, seed=71))
    check_select_and_attend(b, b.oracle_summaries(), out_tol=2e-2)


def test_argument_errors_are_reported_on_the_host():
    import ctypes as C
    import paper_2607_24555_b200 as locks
    from paper_2607_24555_b200.binding import make_config, lib
    gc = _gc(small_bf16([16 * 20], Hq=8, Hkv=2, budget=128))
    with pytest.raises(locks.LocksError):
        gc.ctx.locks_select(gc.case.q, None, gc.kv, 1, None, None)
    with pytest.raises(locks.LocksError):
        gc.ctx.locks_sparse_attend(gc.case.q, gc.kv, 99, None, None, gc.case.q)
    assert locks.locks_workspace_bytes(make_config(8, 3, 8, "i4", "bf16", 1, 16, 64)) == 0      # Hq % Hkv
    assert locks.locks_workspace_bytes(make_config(8, 2, 3, "i4", "bf16", 1, 16, 64)) == 0      # rank
    assert locks.locks_workspace_bytes(make_config(8, 2, 8, "i4", "bf16", 1, 16, 16)) == 0      # k < 2


# ----------------------------------------------------------------------------- full-size configs

def test_config1_full_size_sampled():
    """Llama shapes at full size (8 x 32K, r8i4, b = 2048) in the launch configuration bench.py
    times; the oracle checks every page mass of sampled (request, head) problems and the outputs."""
    from gpu_util import check_select_and_attend
    gc = _gc(locks_synth.config1())
    w = gc.w
    summ_gpu = gc.gpu_build()
    summ_np = summ_gpu.cpu().numpy()                                  # GPU-built bytes handed to the oracle
    differed = check_select_and_attend(gc, summ_np, out_tol=2e-2)
    assert differed <= 2, differed                                    # of 64 problems
    out, lse = gc.gpu_attend()                                        # dense flash-decode baseline
    sub = slice(0, 2)
    oout, olse = oracle.attend(gc.cache, t2np(gc.case.q), gc.sm)
    assert np.abs(out - oout).max() <= 2e-2 and np.abs(lse - olse).max() <= 1e-3


def test_config3_long_context_128k():
    from gpu_util import check_select_and_attend
    gc = _gc(locks_synth.config3(T=131072))
    summ_np = gc.gpu_build().cpu().numpy()
    differed = check_select_and_attend(gc, summ_np, out_tol=2e-2)
    assert differed <= 1
