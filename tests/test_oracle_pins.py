"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU, no CUDA code).

Each test names the passage of the LOCKS paper it rests on.  A plausible mistake in the oracle
(dropped term, wrong sign, wrong index, transposed operand, wrong normalisation set) fails at
least one of them.
"""
import itertools
import math

import numpy as np
import pytest

import oracle
from common import read_golden

SM = 1.0 / math.sqrt(128.0)
rng = np.random.default_rng(1234)


def low_rank_page(rank, B=16, d=128, noise=0.0, seed=0):
    g = np.random.default_rng(seed)
    mu = g.standard_normal(d)
    dirs = g.standard_normal((rank, d))
    a = g.standard_normal((B, rank)) * 3.0
    return mu + a @ dirs + noise * g.standard_normal((B, d))


# ------------------------------------------------------------------ eigensolver (library cross-check)

@pytest.mark.parametrize("n", [2, 5, 16])
def test_jacobi_matches_numpy_eigh(n):
    A = rng.standard_normal((n, n))
    A = A @ A.T
    lam, U = oracle.eigh_jacobi(A)
    ref = np.linalg.eigvalsh(A)[::-1]
    assert np.allclose(lam, ref, rtol=1e-12, atol=1e-12 * abs(ref).max())
    assert np.allclose(U.T @ U, np.eye(n), atol=1e-12)
    assert np.allclose(U @ np.diag(lam) @ U.T, A, atol=1e-10 * abs(A).max())
    w, Q = np.linalg.eigh(A)
    for l in range(n):  # projectors onto each (simple) eigenvector agree
        pr = np.outer(U[:, l], U[:, l])
        qr = np.outer(Q[:, n - 1 - l], Q[:, n - 1 - l])
        assert np.abs(pr - qr).max() < 1e-9


def test_jacobi_degenerate_and_zero():
    lam, U = oracle.eigh_jacobi(np.zeros((4, 4)))
    assert np.all(lam == 0) and np.allclose(U, np.eye(4))
    lam, U = oracle.eigh_jacobi(np.diag([1.0, 3.0, 3.0, 2.0]))
    assert np.allclose(lam, [3, 3, 2, 1])


# ------------------------------------------------------------------ build invariants (Sec. 4 Build; Cor. 2)

@pytest.mark.parametrize("r", [1, 2, 4, 8, 15])
def test_build_invariants(r):
    keys = low_rank_page(6, noise=0.1, seed=r)
    mu, V, C, lam, r_eff = oracle.build_page(keys, r)
    D = keys - keys.mean(0)
    assert r_eff == r
    assert np.allclose(mu, keys.mean(0), atol=1e-13)
    assert np.allclose(V @ V.T, np.eye(r), atol=1e-9)               # orthonormal basis
    assert np.allclose(C.sum(0), 0, atol=1e-9)                      # centred coefficients
    assert np.allclose(C.T @ C, np.diag(lam[:r]), atol=1e-8 * lam[0])   # C^T C = Sigma_r^2
    assert np.allclose(C, D @ V.T, atol=1e-9 * np.sqrt(lam[0]))         # c_i = V^T delta_i
    assert np.isclose(lam.sum(), (D * D).sum(), rtol=1e-12)             # trace
    resid = ((D - C @ V) ** 2).sum()
    assert np.isclose(resid, lam[r:].sum(), rtol=1e-8, atol=1e-9 * lam[0])  # Eckart-Young tail
    sv = np.linalg.svd(D, compute_uv=False)
    assert np.allclose(np.sqrt(np.maximum(lam[:15], 0)), sv[:15], rtol=1e-9, atol=1e-9 * sv[0])
    for l in range(r):  # sign convention
        assert V[l, np.argmax(np.abs(V[l]))] > 0


def test_build_drops_zero_modes():
    keys = low_rank_page(3, noise=0.0, seed=5)                      # rank(D) = 3
    mu, V, C, lam, r_eff = oracle.build_page(keys, 8)
    assert r_eff == 3
    assert np.all(V[3:] == 0) and np.all(C[:, 3:] == 0)
    # a centred page never has more than B-1 modes
    keys = np.random.default_rng(0).standard_normal((16, 128))
    _, V, C, lam, r_eff = oracle.build_page(keys, 16)
    assert r_eff == 15 and np.all(V[15] == 0) and np.all(C[:, 15] == 0)
    # all keys identical: D = 0, nothing kept
    _, V, C, lam, r_eff = oracle.build_page(np.tile(keys[:1], (16, 1)), 8)
    assert r_eff == 0 and np.all(V == 0) and np.all(C == 0)


# ------------------------------------------------------------------ Eq. (1) against the exact log-mass

def test_full_rank_summary_is_exact():
    """Prop. 3 / Sec. 4: r >= rank(D_j) reproduces the exact page log-mass."""
    g = np.random.default_rng(7)
    keys = g.standard_normal((16, 128)) * 2.0
    q = g.standard_normal(128) * 1.5
    mu, V, C, lam, _ = oracle.build_page(keys, 16)
    assert abs(oracle.score(mu, V, C, q, SM) - oracle.exact_lse(keys, q, SM)) < 1e-10
    keys = low_rank_page(5, noise=0.0, seed=3)                      # planted rank 5 <= r = 8
    mu, V, C, lam, _ = oracle.build_page(keys, 8)
    assert abs(oracle.score(mu, V, C, q, SM) - oracle.exact_lse(keys, q, SM)) < 1e-10
    mu, V, C, lam, _ = oracle.build_page(keys, 4)                   # r < rank: no longer exact
    assert abs(oracle.score(mu, V, C, q, SM) - oracle.exact_lse(keys, q, SM)) > 1e-4


def test_exact_lse_matches_definition():
    g = np.random.default_rng(8)
    keys, q = g.standard_normal((16, 128)), g.standard_normal(128)
    ref = np.log(np.exp(keys @ q * SM).sum())
    assert abs(oracle.exact_lse(keys, q, SM) - ref) < 1e-12
    assert abs(oracle.exact_lse(keys[:5], q, SM) - np.log(np.exp(keys[:5] @ q * SM).sum())) < 1e-12


def test_score_error_bounds():
    """Prop. 3: |s^ - s| <= max_i |q_perp . delta_perp_i|/sqrt(d) <= |q_perp| sigma_{r+1}/sqrt(d)
    <= |q_perp| sqrt(tau_r)/sqrt(d), on every page and query tried."""
    g = np.random.default_rng(9)
    for trial in range(40):
        r = [2, 4, 8][trial % 3]
        keys = low_rank_page(6, noise=0.3, seed=100 + trial)
        q = g.standard_normal(128) * (1 + trial % 4)
        mu, V, C, lam, _ = oracle.build_page(keys, r)
        err = abs(oracle.score(mu, V, C, q, SM) - oracle.exact_lse(keys, q, SM))
        D = keys - mu
        dperp = D - C @ V
        qperp = q - V.T @ (V @ q)
        b1 = np.abs(dperp @ qperp).max() * SM
        b2 = np.linalg.norm(qperp) * math.sqrt(lam[r]) * SM
        b3 = np.linalg.norm(qperp) * math.sqrt(lam[r:].sum()) * SM
        assert err <= b1 * (1 + 1e-9) + 1e-12
        assert b1 <= b2 * (1 + 1e-9) and b2 <= b3 * (1 + 1e-9)
        assert err > 0  # the bound is not vacuous: truncation does perturb the score


def test_score_closed_forms():
    g = np.random.default_rng(10)
    q = g.standard_normal(128)
    key = g.standard_normal(128)
    # identical keys: s^ = q.mu/sqrt(d) + log B
    mu, V, C, _, _ = oracle.build_page(np.tile(key, (16, 1)), 8)
    assert abs(oracle.score(mu, V, C, q, SM) - (SM * q @ key + math.log(16))) < 1e-12
    # rank-1 deviations: r = 1 is exact
    keys = key + np.outer(g.standard_normal(16), g.standard_normal(128))
    mu, V, C, _, _ = oracle.build_page(keys, 1)
    assert abs(oracle.score(mu, V, C, q, SM) - oracle.exact_lse(keys, q, SM)) < 1e-10
    # a single rank-r score by hand: mu = 0, V = e_0, c_i = i  ->  log sum_i exp(q_0 i / sqrt d)
    V = np.zeros((1, 128)); V[0, 0] = 1.0
    C = np.arange(16, dtype=float).reshape(16, 1)
    ref = np.log(np.exp(q[0] * np.arange(16) * SM).sum())
    assert abs(oracle.score(np.zeros(128), V, C, q, SM) - ref) < 1e-12
    # the centroid term enters once, inside the scale
    assert abs(oracle.score(key, V, C, q, SM) - (ref + SM * q @ key)) < 1e-12


def test_score_symmetries():
    """Token permutation and a common rotation of keys and query leave s^ unchanged."""
    g = np.random.default_rng(11)
    keys = low_rank_page(6, noise=0.2, seed=21)
    q = g.standard_normal(128)
    mu, V, C, _, _ = oracle.build_page(keys, 4)
    s0 = oracle.score(mu, V, C, q, SM)
    perm = g.permutation(16)
    mu, V, C, _, _ = oracle.build_page(keys[perm], 4)
    assert abs(oracle.score(mu, V, C, q, SM) - s0) < 1e-10
    Q, _ = np.linalg.qr(g.standard_normal((128, 128)))
    mu, V, C, _, _ = oracle.build_page(keys @ Q, 4)
    assert abs(oracle.score(mu, V, C, q @ Q, SM) - s0) < 1e-9


# ------------------------------------------------------------------ isotropic null (paper-printed numbers)

def test_isotropic_null_matches_paper():
    med, mean, std = read_golden("isotropic_null.txt")[0]
    g = np.random.default_rng(2024)
    frac = np.empty(20000)
    for i in range(20000):
        keys = g.standard_normal((16, 128))
        D = keys - keys.mean(0)
        lam, _ = oracle.eigh_jacobi(D @ D.T)
        frac[i] = lam[:8].sum() / lam.sum()
    assert abs(np.median(frac) - med) < 0.002
    assert abs(frac.mean() - mean) < 0.002
    assert abs(frac.std() - std) < 0.001


# ------------------------------------------------------------------ storage formats

def test_payload_bytes_match_paper_table():
    for r, stored, alpha, ceil_, red, share in read_golden("payload_table.txt"):
        r = int(r)
        nbytes = oracle.summary_payload_bytes(oracle.FMT_I4, r)
        assert nbytes == int(stored)
        assert round(nbytes / 8192, 3) == alpha
        assert round(8192 / nbytes) == int(ceil_)
        N, b = 1 << 20, 2048
        dense = N * 512
        ours = (N // 16) * nbytes + b * 512
        assert round(dense / ours, 1) == red
        assert round(100 * (N // 16) * nbytes / ours) == int(share)
        assert oracle.summary_stride_bytes(oracle.FMT_I4, r) % 16 == 0
        assert 0 <= oracle.summary_stride_bytes(oracle.FMT_I4, r) - nbytes < 16
    for B, pct in read_golden("pagesize_payload.txt"):
        B = int(B)
        logical = 128 * 8 // 2 + B * 8 + 128
        assert round(100 * logical / (B * 512), 1) == pct
    assert oracle.summary_payload_bytes(oracle.FMT_F32, 8) == 5120


def test_half_conversion_matches_numpy():
    g = np.random.default_rng(3)
    xs = np.concatenate([g.standard_normal(2000) * 10.0 ** g.integers(-9, 5, 2000),
                         [0.0, 1.0, 65504.0, 65519.9, 65520.0, 1e-8, 5.96e-8, 2.98e-8, 2.99e-8, 6.1e-5]])
    for x in xs:
        bits = oracle.double_to_half(float(x))
        ref = np.float16(x)
        assert bits == int(ref.view(np.uint16)), (x, bits, ref)
        if np.isfinite(ref):
            assert oracle.half_to_double(bits) == float(ref)


@pytest.mark.parametrize("B", [16, 32, 64])
@pytest.mark.parametrize("r", [2, 4, 8])
def test_i4_pack_roundtrip_and_quantiser(r, B):
    """(B = 32, 64: the page sizes of the paper's App. D ablation; same quantiser, coefficients stored row-major.)"""
    g = np.random.default_rng(40 + r + B)
    keys = (low_rank_page(6, noise=0.2, seed=40 + r) + 3.0) if B == 16 else \
        (g.standard_normal((B, 6)) @ g.standard_normal((6, 128)) * 2.0 + 0.2 * g.standard_normal((B, 128)) + 3.0)
    mu, V, C, _, _ = oracle.build_page(keys, r)
    assert C.shape == (B, r)
    blob = oracle.pack(oracle.FMT_I4, mu, V, C)
    assert blob.size == oracle.summary_stride_bytes(oracle.FMT_I4, r, B)
    assert oracle.summary_payload_bytes(oracle.FMT_I4, r, B) == 128 * r // 2 + B * r + 128 + 2 * (r + B + 1)
    assert np.all(blob[oracle.summary_payload_bytes(oracle.FMT_I4, r, B):] == 0)
    cV, cC, cMu, sV, sC, sMu = oracle.unpack_codes(r, blob, B)
    mu2, V2, C2 = oracle.unpack(oracle.FMT_I4, r, blob, B)
    assert np.abs(cV).max() <= 7 and np.abs(cC).max() <= 127 and np.abs(cMu).max() <= 127
    for l in range(r):   # one fp16 scale per basis column, abs-max symmetric, round-half-even codes
        assert sV[l] == float(np.float16(np.abs(V[l]).max() / 7))
        assert np.array_equal(cV[l], np.clip(np.rint(V[l] / sV[l]), -7, 7))
        assert np.allclose(V2[l], cV[l] * sV[l], rtol=0, atol=0)
        assert np.abs(V2[l] - V[l]).max() <= 0.5 * sV[l] * (1 + 1e-3) + 1e-12
    for i in range(B):  # one scale per coefficient row
        assert sC[i] == float(np.float16(np.abs(C[i]).max() / 127))
        assert np.array_equal(cC[i], np.clip(np.rint(C[i] / sC[i]), -127, 127))
        assert np.array_equal(C2[i], cC[i] * sC[i])
    assert sMu == float(np.float16(np.abs(mu).max() / 127))
    assert np.array_equal(cMu, np.clip(np.rint(mu / sMu), -127, 127))
    assert np.array_equal(mu2, cMu * sMu)


@pytest.mark.parametrize("r,B", [(2, 16), (4, 16), (8, 16), (8, 32), (4, 64)])
def test_i4_layout_is_a_bijection(r, B):
    """Every payload byte/nibble is owned by exactly one entry: flipping one entry changes exactly
    one nibble (basis) or one byte (coefficients, centroid) and nothing else."""
    V = np.zeros((r, 128)); C = np.zeros((B, r)); mu = np.zeros(128)
    V[:, 0] = 7.0; C[:, 0] = 127.0; mu[0] = 127.0       # fixes every scale at 1.0
    base = oracle.pack(oracle.FMT_I4, mu, V, C)
    seen = set()
    for l in range(r):
        for c in range(1, 128):
            V2 = V.copy(); V2[l, c] = 3.0
            diff = np.nonzero(oracle.pack(oracle.FMT_I4, mu, V2, C) != base)[0]
            assert diff.size == 1
            b = oracle.pack(oracle.FMT_I4, mu, V2, C)[diff[0]] ^ base[diff[0]]
            key = (int(diff[0]), "lo" if b < 16 else "hi")
            assert key not in seen
            seen.add(key)
    for i in range(B):
        for l in range(1, r):
            C2 = C.copy(); C2[i, l] = 5.0
            diff = np.nonzero(oracle.pack(oracle.FMT_I4, mu, V, C2) != base)[0]
            assert diff.size == 1 and ("c", int(diff[0])) not in seen
            seen.add(("c", int(diff[0])))
    for c in range(1, 128):
        mu2 = mu.copy(); mu2[c] = 9.0
        diff = np.nonzero(oracle.pack(oracle.FMT_I4, mu2, V, C) != base)[0]
        assert diff.size == 1 and ("m", int(diff[0])) not in seen
        seen.add(("m", int(diff[0])))


def test_zero_scale_gives_zero_codes():
    blob = oracle.pack(oracle.FMT_I4, np.zeros(128), np.zeros((8, 128)), np.zeros((16, 8)))
    mu, V, C = oracle.unpack(oracle.FMT_I4, 8, blob)
    assert not mu.any() and not V.any() and not C.any()
    assert abs(oracle.score(mu, V, C, np.ones(128), SM) - math.log(16)) < 1e-12


def test_f32_format_roundtrip():
    keys = low_rank_page(6, noise=0.2, seed=77)
    mu, V, C, _, _ = oracle.build_page(keys, 8)
    mu2, V2, C2 = oracle.unpack(oracle.FMT_F32, 8, oracle.pack(oracle.FMT_F32, mu, V, C))
    assert np.array_equal(mu2, mu.astype(np.float32)) and np.array_equal(V2, V.astype(np.float32))
    assert np.array_equal(C2, C.astype(np.float32))


# ------------------------------------------------------------------ combine + selection (Cor. 4, Thm. 1)

def shares(s):
    e = np.exp(s - s.max(axis=1, keepdims=True))
    return e / e.sum(axis=1, keepdims=True)


def test_select_brute_force_maximises_group_coverage():
    """Cor. 4: among k-sets containing sink and most recent page, the selected set maximises the
    group-mean coverage sum_{j in S} m_bar_j (shares normalised over the candidates)."""
    g = np.random.default_rng(12)
    for trial in range(30):
        P = int(g.integers(4, 12)); G = int(g.integers(1, 5)); k = int(g.integers(2, min(6, P)))
        s = g.standard_normal((G, P)) * 3
        ids, cnt, logm = oracle.select_one(s, P, k)
        assert cnt == k and ids[0] == 0 and ids[k - 1] == P - 1 and np.all(np.diff(ids[:k]) > 0)
        mbar = shares(s[:, 1:P - 1]).mean(0)                       # candidate pages 1..P-2
        assert np.allclose(np.exp(logm[1:P - 1]), mbar, rtol=1e-12)
        best = max(sum(mbar[j - 1] for j in comb)
                   for comb in itertools.combinations(range(1, P - 1), k - 2))
        got = sum(mbar[j - 1] for j in ids[1:k - 1])
        assert abs(got - best) < 1e-13


def test_select_edge_cases_and_ties():
    s = np.zeros((2, 10))
    ids, cnt, _ = oracle.select_one(s, 10, 4)                      # all tied: lower indices win
    assert cnt == 4 and ids.tolist() == [0, 1, 2, 9]
    ids, cnt, _ = oracle.select_one(s, 3, 4)                       # P <= k: every page
    assert cnt == 3 and ids.tolist() == [0, 1, 2, -1]
    ids, cnt, _ = oracle.select_one(s, 1, 4)
    assert cnt == 1 and ids.tolist() == [0, -1, -1, -1]
    ids, cnt, _ = oracle.select_one(s, 10, 2)                      # k = 2: sink + recent only
    assert cnt == 2 and ids.tolist() == [0, 9]
    # a head-wise constant shift changes no share and no set (Eq. 2 factorisation remark)
    g = np.random.default_rng(13)
    s = g.standard_normal((4, 40)) * 2
    a, _, la = oracle.select_one(s, 40, 8)
    b, _, lb = oracle.select_one(s + g.standard_normal((4, 1)) * 50, 40, 8)
    assert np.array_equal(a, b) and np.allclose(la[1:39], lb[1:39], atol=1e-10)
    # the sink and last page's own scores are never read
    s2 = s.copy(); s2[:, 0] = 1e9; s2[:, 39] = -1e9
    c, _, _ = oracle.select_one(s2, 40, 8)
    assert np.array_equal(a, c)


def test_share_sandwich_and_retention():
    """Thm. 1 steps 2-3: |log m^bar - log m_bar| <= 2 eta and the estimated-share set keeps at least
    e^{-4 eta} of the candidate coverage of the exact-share set."""
    g = np.random.default_rng(14)
    for trial in range(20):
        G, P, k = 4, 60, 10
        s = g.standard_normal((G, P)) * 4
        eta = 0.05 * (1 + trial % 5)
        shat = s + g.uniform(-eta, eta, size=s.shape)
        ia, _, la = oracle.select_one(s, P, k)
        ib, _, lb = oracle.select_one(shat, P, k)
        assert np.abs(la[1:P - 1] - lb[1:P - 1]).max() <= 2 * eta + 1e-12
        m = np.exp(la)
        cov_exact = m[ia[1:k - 1]].sum()
        cov_est = m[ib[1:k - 1]].sum()
        assert cov_est >= math.exp(-4 * eta) * cov_exact - 1e-12


# ------------------------------------------------------------------ attention (Sec. 3, Lemma 1)

def tiny_cache(T=70, Hq=4, Hkv=2, B=16, d=128, seed=0, nb_extra=3):
    g = np.random.default_rng(seed)
    P = -(-T // B)
    nb = P + nb_extra
    k = g.standard_normal((nb, Hkv, B, d)).astype(np.float32)
    v = g.standard_normal((nb, Hkv, B, d)).astype(np.float32)
    bt = g.permutation(nb)[:P].astype(np.int32).reshape(1, P)
    return oracle.Cache(k, v, bt, np.array([T], np.int32), Hq), g


def dense_reference(cache, q, pages):
    """Textbook softmax attention over the tokens of the given pages, straight from numpy."""
    B, d, G = cache.B, cache.d, cache.Hq // cache.Hkv
    T = int(cache.seq_lens[0])
    out = np.zeros((cache.Hq, d)); lse = np.zeros(cache.Hq)
    for gq in range(cache.Hq):
        h = gq // G
        ks, vs = [], []
        for p in pages:
            blk = cache.block_table[0, p]
            n = min(B, T - p * B)
            ks.append(cache.k[blk, h, :n]); vs.append(cache.v[blk, h, :n])
        ks, vs = np.concatenate(ks).astype(np.float64), np.concatenate(vs).astype(np.float64)
        x = ks @ q[0, gq].astype(np.float64) / math.sqrt(d)
        w = np.exp(x - x.max())
        out[gq] = (w / w.sum()) @ vs
        lse[gq] = x.max() + math.log(w.sum())
    return out, lse


def test_attend_matches_textbook_softmax():
    cache, g = tiny_cache(T=70)
    q = g.standard_normal((1, 4, 128)).astype(np.float32)
    out, lse = oracle.attend(cache, q, SM)                          # dense: all 5 pages, 70 tokens
    ref, rl = dense_reference(cache, q, range(5))
    assert np.allclose(out[0], ref, atol=1e-12) and np.allclose(lse[0], rl, atol=1e-12)
    ids = np.array([[[0, 2, 4, -1], [1, 4, -1, -1]]], np.int32)
    cnt = np.array([[3, 2]], np.int32)
    out, lse = oracle.attend(cache, q, SM, ids, cnt)
    for h, pages in enumerate([[0, 2, 4], [1, 4]]):
        ref, rl = dense_reference(cache, q, pages)
        assert np.allclose(out[0, 2 * h:2 * h + 2], ref[2 * h:2 * h + 2], atol=1e-12)
        assert np.allclose(lse[0, 2 * h:2 * h + 2], rl[2 * h:2 * h + 2], atol=1e-12)


def test_attend_special_cases():
    # a single token: the output is that token's value
    cache, g = tiny_cache(T=1)
    q = g.standard_normal((1, 4, 128)).astype(np.float32)
    out, lse = oracle.attend(cache, q, SM)
    blk = cache.block_table[0, 0]
    for gq in range(4):
        assert np.allclose(out[0, gq], cache.v[blk, gq // 2, 0], atol=1e-12)
        assert abs(lse[0, gq] - SM * float(cache.k[blk, gq // 2, 0].astype(np.float64) @ q[0, gq])) < 1e-9
    # zero query: uniform weights, output is the mean value, lse = log T
    cache, g = tiny_cache(T=37)
    out, lse = oracle.attend(cache, np.zeros((1, 4, 128), np.float32), SM)
    ref, _ = dense_reference(cache, np.zeros((1, 4, 128), np.float32), range(3))
    assert np.allclose(out[0], ref, atol=1e-12) and np.allclose(lse, math.log(37), atol=1e-12)


def test_coverage_identity_and_bound():
    """Lemma 1(i): o - o_S = eps (vbar_Sc - vbar_S) exactly, and |o - o_S| <= 2R(1 - gamma_S)."""
    cache, g = tiny_cache(T=160, Hq=2, Hkv=2)
    q = g.standard_normal((1, 2, 128)).astype(np.float32) * 3
    P = 10
    full, lse_full = oracle.attend(cache, q, SM)
    for trial in range(5):
        S = sorted(g.choice(P, size=4, replace=False).tolist())
        Sc = [p for p in range(P) if p not in S]
        ids = np.array([[S, S]], np.int32); cnt = np.array([[4, 4]], np.int32)
        oS, lS = oracle.attend(cache, q, SM, ids, cnt)
        idc = np.array([[Sc, Sc]], np.int32); cnc = np.array([[6, 6]], np.int32)
        oC, lC = oracle.attend(cache, q, SM, idc, cnc)
        gamma = np.exp(lS - lse_full)                               # coverage of S
        assert np.allclose(np.exp(lS - lse_full) + np.exp(lC - lse_full), 1, atol=1e-12)
        eps = 1 - gamma
        assert np.allclose(full - oS, eps[..., None] * (oC - oS), atol=1e-12)
        R = np.linalg.norm(cache.v.astype(np.float64), axis=-1).max()
        assert np.all(np.linalg.norm(full - oS, axis=-1) <= 2 * R * eps + 1e-12)


def test_full_budget_equals_dense_and_pipeline_runs():
    """Budget >= all pages selects everything, so the sparse output is the dense one; with a small
    budget the pipeline returns sink + recent + top pages."""
    import torch
    import locks_synth
    from common import oracle_cache, fmt_code
    w = locks_synth.config0().with_(seq_lens=[300], budget=4096, carriers=2)
    case = locks_synth.make_case(w)
    cache = oracle_cache(case)
    q = case.q.numpy()
    summ = oracle.build_summaries(cache, w.rank, fmt_code(w))
    ids, cnt, out, lse = oracle.decode_step(cache, q, w.rank, fmt_code(w), summ, SM, w.k)
    P = 19
    assert cnt[0, 0] == P and ids[0, 0, :P].tolist() == list(range(P))
    dense, dl = oracle.attend(cache, q, SM)
    assert np.allclose(out, dense, atol=1e-13) and np.allclose(lse, dl, atol=1e-13)
    ids, cnt, out, lse = oracle.decode_step(cache, q, w.rank, fmt_code(w), summ, SM, 6)
    assert cnt[0, 0] == 6 and ids[0, 0, 0] == 0 and ids[0, 0, 5] == P - 1
    for cp in case.carrier_pages[0]:                                # planted carriers are found
        assert cp in ids[0, 0].tolist()
    # the estimated masses follow the exact ones within the proven bound on this data
    shat = oracle.page_logmass(cache, q, w.rank, fmt_code(w), summ, SM)
    sex = oracle.page_logmass(cache, q, w.rank, fmt_code(w), None, SM, exact=True)
    assert np.nanmax(np.abs(shat - sex)[:, :, :P - 1]) < 0.5
    assert np.all(np.isnan(shat[:, :, P - 1:]))


# ------------------------------------------------------------------ batch / head indexing of the wrappers

def ragged_batch_cache(layout="HND", bf16=False, seed=5):
    """3 requests of different lengths (one with a partial tail page), 2 KV heads x 3 query heads each,
    physical blocks dealt by a permutation that interleaves the requests, spare blocks in between."""
    g = np.random.default_rng(seed)
    B, d, Hkv, Hq = 16, 128, 2, 6
    lens = [16 * 9 + 5, 16 * 7, 16 * 12 + 1]
    pages = [-(-t // B) for t in lens]
    nb = sum(pages) + 4
    shape = (nb, Hkv, B, d) if layout == "HND" else (nb, B, Hkv, d)
    k = g.standard_normal(shape).astype(np.float32)
    v = g.standard_normal(shape).astype(np.float32)
    if bf16:   # stored as raw bfloat16 bits; `vals` are the values those bits stand for
        k = (k.view(np.uint32) >> 16).astype(np.uint16)
        v = (v.view(np.uint32) >> 16).astype(np.uint16)
    perm = g.permutation(nb)
    bt = np.full((3, max(pages)), -12345, np.int32)      # slots past a request's pages hold a poison id
    at = 0
    for b, P in enumerate(pages):
        bt[b, :P] = perm[at:at + P]
        at += P
    if layout == "HND":
        strides = {"shape": (nb, Hkv, B, d), "block": Hkv * B * d, "head": B * d, "token": d}
    else:
        strides = {"shape": (nb, Hkv, B, d), "block": B * Hkv * d, "head": d, "token": Hkv * d}
    cache = oracle.Cache(k, v, bt, np.array(lens, np.int32), Hq, strides=strides)

    def vals(a):
        f = (a.astype(np.uint32) << 16).view(np.float32) if bf16 else a
        return f.astype(np.float64)

    def page(a, blk, h):   # [B, d] values of (block, head), whatever the layout
        return vals(a[blk, h]) if layout == "HND" else vals(a[blk, :, h])

    q = g.standard_normal((3, Hq, d)).astype(np.float32)
    if bf16:
        q = (q.view(np.uint32) >> 16).astype(np.uint16)
    return cache, q, vals(q), page, lens, pages


@pytest.mark.parametrize("layout,bf16,fmt,r", [("HND", False, oracle.FMT_I4, 8), ("NHD", True, oracle.FMT_I4, 4),
                                               ("HND", True, oracle.FMT_F32, 3)])
def test_batch_wrappers_index_requests_heads_and_blocks(layout, bf16, fmt, r):
    """build_summaries, page_logmass, select, attend and decode_step on a ragged batch of 3 requests, 2 KV heads,
    G = 3, permuted blocks: every entry equals what the per-page functions (pinned above one by one) give when
    they are composed with the index arithmetic written out here."""
    cache, q_raw, q, page, lens, pages = ragged_batch_cache(layout, bf16)
    B, d, Hkv, Hq, G = 16, 128, 2, 6, 3
    k = 5
    summ = oracle.build_summaries(cache, r, fmt)
    stride = oracle.summary_stride_bytes(fmt, r)
    assert summ.shape == (cache.num_blocks, Hkv, stride)
    used = set()
    shat_ref = np.full((3, Hq, max(pages)), np.nan)
    sex_ref = np.full((3, Hq, max(pages)), np.nan)
    for b in range(3):
        for h in range(Hkv):
            for p in range(lens[b] // B):                              # complete pages only
                blk = int(cache.block_table[b, p])
                used.add((blk, h))
                mu, V, Cc, _, _ = oracle.build_page(page(cache.k, blk, h), r)
                assert np.array_equal(summ[blk, h], oracle.pack(fmt, mu, V, Cc)), (b, h, p)
            for p in range(pages[b] - 1):                              # pages 0 .. P-2 are scored
                blk = int(cache.block_table[b, p])
                m = oracle.unpack(fmt, r, summ[blk, h])
                for gi in range(G):
                    shat_ref[b, h * G + gi, p] = oracle.score(*m, q[b, h * G + gi], SM)
                    sex_ref[b, h * G + gi, p] = oracle.exact_lse(page(cache.k, blk, h), q[b, h * G + gi], SM)
    for blk in range(cache.num_blocks):                                # nothing else was written
        for h in range(Hkv):
            if (blk, h) not in used:
                assert not summ[blk, h].any()
    shat = oracle.page_logmass(cache, q_raw, r, fmt, summ, SM)
    sex = oracle.page_logmass(cache, q_raw, r, fmt, None, SM, exact=True)
    assert np.array_equal(np.isnan(shat), np.isnan(shat_ref)) and np.array_equal(np.isnan(sex), np.isnan(sex_ref))
    assert np.nanmax(np.abs(shat - shat_ref)) == 0.0 and np.nanmax(np.abs(sex - sex_ref)) == 0.0
    ids, cnt, ls = oracle.select(cache, shat, k)
    ids_ref = np.full((3, Hkv, k), -1, np.int32)
    for b in range(3):
        for h in range(Hkv):
            i1, c1, l1 = oracle.select_one(shat[b, h * G:(h + 1) * G], pages[b], k)
            ids_ref[b, h] = i1
            assert cnt[b, h] == c1 == k and np.array_equal(ids[b, h], i1)
            assert np.array_equal(ls[b, h, 1:pages[b] - 1], l1[1:pages[b] - 1])
            assert np.all(np.isnan(ls[b, h, pages[b] - 1:])) and np.isnan(ls[b, h, 0])
    # the two heads and the three requests do select different pages here, so a swapped index would show
    assert len({tuple(ids[b, h]) for b in range(3) for h in range(Hkv)}) == 3 * Hkv

    def attend_ref(b, gq, plist):
        h = gq // G
        ks, vs = [], []
        for p in plist:
            blk = int(cache.block_table[b, p])
            n = min(B, lens[b] - p * B)
            ks.append(page(cache.k, blk, h)[:n]); vs.append(page(cache.v, blk, h)[:n])
        ks, vs = np.concatenate(ks), np.concatenate(vs)
        x = ks @ q[b, gq] / math.sqrt(d)
        wgt = np.exp(x - x.max())
        return (wgt / wgt.sum()) @ vs, x.max() + math.log(wgt.sum())

    out, lse = oracle.attend(cache, q_raw, SM, ids, cnt)
    dense, dlse = oracle.attend(cache, q_raw, SM)
    sids, scnt, sout, slse = oracle.decode_step(cache, q_raw, r, fmt, summ, SM, k)
    assert np.array_equal(sids, ids) and np.array_equal(scnt, cnt)
    assert np.array_equal(sout, out) and np.array_equal(slse, lse)
    for b in range(3):
        for gq in range(Hq):
            o, l = attend_ref(b, gq, ids[b, gq // G, :k].tolist())
            assert np.allclose(out[b, gq], o, atol=1e-12) and abs(lse[b, gq] - l) < 1e-12
            o, l = attend_ref(b, gq, range(pages[b]))
            assert np.allclose(dense[b, gq], o, atol=1e-12) and abs(dlse[b, gq] - l) < 1e-12


def test_per_head_arm_selects_and_attends_head_by_head():
    """The per-head arm of the combine ablation (App. D): every query head keeps the pages of its own largest shares
    and attends them.  select_per_head equals select_one on a group of one, head by head; attend with per-head tables
    equals a numpy softmax over exactly that head's pages, and equals the grouped call when the heads of a group are
    handed the same table; heads of one group do end up with different pages here."""
    cache, q_raw, q, page, lens, pages = ragged_batch_cache("NHD", True, seed=9)
    B, d, Hkv, Hq, G, k, r, fmt = 16, 128, 2, 6, 3, 5, 8, oracle.FMT_I4
    summ = oracle.build_summaries(cache, r, fmt)
    shat = oracle.page_logmass(cache, q_raw, r, fmt, summ, SM)
    ids, cnt, ls = oracle.select_per_head(cache, shat, k)
    assert ids.shape == (3, Hq, k) and cnt.shape == (3, Hq) and ls.shape == (3, Hq, max(pages))
    for b in range(3):
        for gq in range(Hq):
            i1, c1, l1 = oracle.select_one(shat[b, gq:gq + 1], pages[b], k)
            assert cnt[b, gq] == c1 and np.array_equal(ids[b, gq], i1)
            assert np.array_equal(ls[b, gq, 1:pages[b] - 1], l1[1:pages[b] - 1])
            # a group of one: the key is the head's own log share
            cand = shat[b, gq, 1:pages[b] - 1]
            assert np.allclose(l1[1:pages[b] - 1], cand - (cand.max() + np.log(np.exp(cand - cand.max()).sum())), atol=1e-12)
    assert any(len({tuple(ids[b, h * G + gi]) for gi in range(G)}) > 1 for b in range(3) for h in range(Hkv))
    out, lse = oracle.attend(cache, q_raw, SM, ids, cnt, per_head=True)
    for b in range(3):
        for gq in range(Hq):
            h = gq // G
            ks, vs = [], []
            for pg in ids[b, gq, :cnt[b, gq]]:
                blk = int(cache.block_table[b, pg])
                n = min(B, lens[b] - pg * B)
                ks.append(page(cache.k, blk, h)[:n]); vs.append(page(cache.v, blk, h)[:n])
            ks, vs = np.concatenate(ks), np.concatenate(vs)
            x = ks @ q[b, gq] / math.sqrt(d)
            wgt = np.exp(x - x.max())
            assert np.allclose(out[b, gq], (wgt / wgt.sum()) @ vs, atol=1e-12)
            assert abs(lse[b, gq] - (x.max() + math.log(wgt.sum()))) < 1e-12
    gids, gcnt, _ = oracle.select(cache, shat, k)
    rep_ids = np.repeat(gids, G, axis=1)
    rep_cnt = np.repeat(gcnt, G, axis=1)
    o1, l1 = oracle.attend(cache, q_raw, SM, gids, gcnt)
    o2, l2 = oracle.attend(cache, q_raw, SM, rep_ids, rep_cnt, per_head=True)
    assert np.array_equal(o1, o2) and np.array_equal(l1, l2)


def test_build_summaries_page_ranges_per_request():
    """page_begin / page_end are per request: only the named complete pages are written."""
    cache, _, _, page, lens, pages = ragged_batch_cache()
    r, fmt = 8, oracle.FMT_I4
    full = oracle.build_summaries(cache, r, fmt)
    part = oracle.build_summaries(cache, r, fmt, page_begin=[2, 0, 11], page_end=[4, 0, 99])
    want = {(0, 2), (0, 3), (2, 11)}                                   # request 2 has 12 complete pages: 11 is the last
    for b in range(3):
        for p in range(pages[b]):
            blk = int(cache.block_table[b, p])
            if (b, p) in want:
                assert np.array_equal(part[blk], full[blk]) and part[blk].any()
            else:
                assert not part[blk].any()


# ------------------------------------------------------------------ selection fidelity metrics (App. B)

def test_selection_quality_closed_forms_and_token_level_softmax():
    """gamma, gamma_c, recall, needle: hand-computable cases, and gamma against the token-level softmax mass of the
    selected pages computed straight from numpy (the quantity Lemma 1 calls gamma_S)."""
    P = 6
    s = np.log(np.array([[1.0, 2.0, 3.0, 4.0, 5.0, 5.0], [6.0, 1.0, 1.0, 1.0, 1.0, 10.0]]))
    A, R = [0, 2, 3, 5], [0, 3, 4, 5]
    gam, gamc, rec, ndl = oracle.selection_quality(s, P, A, R, marked=[3, 4, 1, 0, 99])
    assert abs(gam - 0.5 * ((1 + 3 + 4 + 5) / 20.0 + (6 + 1 + 1 + 10) / 20.0)) < 1e-14
    assert abs(gamc - 0.5 * ((3 + 4) / 14.0 + (1 + 1) / 4.0)) < 1e-14
    assert rec == 0.5                      # candidates of R: {3, 4}; A keeps 3
    assert ndl == 0.5                      # marked candidates R keeps: {3, 4}; A keeps 3 (1 is not in R; 0, 99 ignored)
    assert oracle.selection_quality(s, P, list(range(P)), R)[:3] == (1.0, 1.0, 1.0)
    g2 = oracle.selection_quality(s, P, [0, 5], [0, 5])
    assert g2[1] == 0.0 and g2[2] == 1.0 and g2[3] == 1.0
    # against the definition at token level on a random cache (partial last page)
    cache, g = tiny_cache(T=93, Hq=4, Hkv=2)
    q = g.standard_normal((1, 4, 128)).astype(np.float32)
    mass = oracle.page_exact_mass_all(cache, q, SM)
    Pn, Bsz = 6, 16
    assert np.all(np.isfinite(mass[0, :, :Pn]))
    sel = [0, 2, 5]
    for h in range(2):
        want = 0.0
        for gq in (2 * h, 2 * h + 1):
            ks = np.concatenate([cache.k[cache.block_table[0, p], h, :min(Bsz, 93 - p * Bsz)] for p in range(Pn)])
            x = ks.astype(np.float64) @ q[0, gq].astype(np.float64) / math.sqrt(128)
            wgt = np.exp(x - x.max()); wgt /= wgt.sum()
            want += sum(wgt[p * Bsz:min((p + 1) * Bsz, 93)].sum() for p in sel) / 2
            # a page's exact log-mass is the log of its tokens' summed exponentials
            assert abs(mass[0, gq, 5] - math.log(np.exp(x[80:93]).sum())) < 1e-12
        got = oracle.selection_quality(mass[0, 2 * h:2 * h + 2], Pn, sel, sel)[0]
        assert abs(got - want) < 1e-13
    # pages 0..P-2 agree with the candidate-only exact arm
    part = oracle.page_logmass(cache, q, 8, oracle.FMT_F32, None, SM, exact=True)
    assert np.array_equal(part[0, :, :Pn - 1], mass[0, :, :Pn - 1])


def test_combine_rules_differ_where_they_should():
    """Share-average, group-max and group-mass on a hand-made group of two heads with very different partition
    functions: head 0 has huge raw masses spread evenly, head 1 small raw masses with one page holding nearly all
    of its share.  Group-max and group-mass follow head 0's raw scores; the share-average keeps head 1's page."""
    P, k = 8, 3                                                   # one free slot
    s = np.zeros((2, P))
    s[0, 1:7] = [10.0, 10.1, 10.2, 10.05, 10.0, 10.0]             # head 0: flat, page 3 barely the largest
    s[1, 1:7] = [-5.0, -5.0, -5.0, -5.0, 1.0, -5.0]               # head 1: page 5 carries ~99 % of its mass
    ids0, c0, key0 = oracle.select_one_rule(s, P, k, oracle.RULE_SHARE_AVG)
    ids1, c1, key1 = oracle.select_one_rule(s, P, k, oracle.RULE_GROUP_MAX)
    ids2, c2, key2 = oracle.select_one_rule(s, P, k, oracle.RULE_GROUP_MASS)
    assert ids0.tolist() == [0, 5, 7] and ids1.tolist() == [0, 3, 7] and ids2.tolist() == [0, 3, 7]
    assert np.array_equal(ids0, oracle.select_one(s, P, k)[0])
    assert np.allclose(key1[1:7], s[:, 1:7].max(0)) and np.allclose(key2[1:7], np.log(np.exp(s[:, 1:7]).sum(0)))
    # one head: every rule ranks by the raw score
    s1 = np.random.default_rng(3).standard_normal((1, 40))
    want = sorted([0, 39] + (np.argsort(-s1[0, 1:39])[:6] + 1).tolist())
    for rule in (0, 1, 2):
        assert oracle.select_one_rule(s1, 40, 8, rule)[0].tolist() == want


# ------------------------------------------------------------------ rival scorers (App. A / B)

def test_rival_scorers_against_the_paper_s_statements():
    """Moment core: s - log B = s^q + R_cum + R_rank with |R_cum| <= L^3 / 3 and 0 <= R_rank <= sigma_{r+1}^2 |q|^2 /
    (2 B d) (Prop. 4), on random pages and queries, unquantised summaries.  Centroid: the score of a summary
    whose coefficients vanish.  Envelope: an upper bound of every logit of the page, tight for a page of one
    repeated key (Lemma 2)."""
    rng = np.random.default_rng(11)
    B, d = 16, 128
    for trial in range(30):
        r = int(rng.integers(1, 15))
        keys = low_rank_page(int(rng.integers(2, 9)), noise=0.3, seed=100 + trial) * float(rng.choice([0.2, 1.0]))
        q = rng.standard_normal(d) * float(rng.choice([0.3, 1.0]))
        mu, V, Cc, lam, r_eff = oracle.build_page(keys, r)
        s_exact = oracle.exact_lse(keys, q, SM)
        s_mom = oracle.rival_score(oracle.SCORER_MOMENT, mu, V, Cc, q, SM)
        s_cen = oracle.rival_score(oracle.SCORER_CENTROID, mu, V, Cc, q, SM)
        z = (keys - keys.mean(0)) @ q * SM                         # centred per-key logits
        kappa2 = float((z ** 2).mean())
        a = float(keys.mean(0) @ q) * SM
        assert abs(s_cen - (a + math.log(B))) < 1e-12
        assert abs(s_cen - oracle.score(mu, V, np.zeros_like(Cc), q, SM)) < 1e-12
        r_rank = 0.5 * kappa2 - (s_mom - s_cen)                    # what the rank truncation leaves out
        assert -1e-12 <= r_rank <= lam[r] * (q @ q) / (2 * B * d) + 1e-12 if r < B else abs(r_rank) < 1e-12
        r_cum = s_exact - math.log(B) - a - 0.5 * kappa2
        assert abs(r_cum) <= np.abs(z).max() ** 3 / 3 + 1e-12
        env = oracle.envelope_score(keys, q, SM)
        assert env >= (keys @ q * SM).max() - 1e-12
    one = np.tile(rng.standard_normal(d), (B, 1))
    q = rng.standard_normal(d)
    assert abs(oracle.envelope_score(one, q, SM) - float(one[0] @ q) * SM) < 1e-12
    # full rank: the moment core is a + log B + kappa_2 / 2 exactly
    keys = rng.standard_normal((B, d))
    mu, V, Cc, lam, _ = oracle.build_page(keys, 15)
    z = (keys - keys.mean(0)) @ q * SM
    assert abs(oracle.rival_score(oracle.SCORER_MOMENT, mu, V, Cc, q, SM) - (float(keys.mean(0) @ q) * SM + math.log(B) + 0.5 * float((z ** 2).mean()))) < 1e-10


# ------------------------------------------------------------------ KV-cache fake quantisation (Sec. 5, KIVI grid)

@pytest.mark.parametrize("bits,bf16", [(4, True), (2, True), (4, False), (8, False)])
def test_fake_quantisation_groups_levels_and_bounds(bits, bf16):
    """Keys: per channel over the page's 16 tokens; values: per token over groups of 32 dims.  Every group keeps its
    minimum and maximum, takes at most 2^bits distinct values, moves no entry by more than half a step (plus the
    storage rounding), and nothing outside the complete pages changes."""
    cache, _, _, page, lens, pages = ragged_batch_cache("HND", bf16, seed=9)
    k0, v0 = cache.k.copy(), cache.v.copy()

    def vals(a):
        return ((a.astype(np.uint32) << 16).view(np.float32) if bf16 else a).astype(np.float64)

    oracle.fake_quantize_pages(cache, bits)
    ulp = 2.0 ** -8 if bf16 else 2.0 ** -23
    touched = set()
    for b in range(3):
        for p in range(lens[b] // 16):
            blk = int(cache.block_table[b, p])
            touched.add(blk)
            for h in range(2):
                K0, K1 = vals(k0[blk, h]), vals(cache.k[blk, h])          # [16, 128]
                lo, hi = K0.min(0), K0.max(0)
                step = (hi - lo) / (2 ** bits - 1)
                assert np.array_equal(K1.min(0), lo) and np.allclose(K1.max(0), hi, rtol=ulp, atol=0)
                assert np.all(np.abs(K1 - K0) <= step / 2 + np.maximum(np.abs(K0), np.abs(K1)) * ulp + 1e-12)
                assert max(len(np.unique(K1[:, c])) for c in range(128)) <= 2 ** bits
                V0, V1 = vals(v0[blk, h]).reshape(16, 4, 32), vals(cache.v[blk, h]).reshape(16, 4, 32)
                lo, hi = V0.min(-1, keepdims=True), V0.max(-1, keepdims=True)
                step = (hi - lo) / (2 ** bits - 1)
                assert np.array_equal(V1.min(-1, keepdims=True), lo)
                assert np.all(np.abs(V1 - V0) <= step / 2 + np.maximum(np.abs(V0), np.abs(V1)) * ulp + 1e-12)
                assert max(len(np.unique(V1[i, g])) for i in range(16) for g in range(4)) <= 2 ** bits
    for blk in range(cache.num_blocks):
        if blk not in touched:
            assert np.array_equal(cache.k[blk], k0[blk]) and np.array_equal(cache.v[blk], v0[blk])
    # a constant group is kept as it is; a two-valued group is a fixed point at any width
    c2, _ = tiny_cache(T=32)
    c2.k[:] = 1.25
    c2.v[:] = np.where(np.arange(128) % 2 == 0, -3.0, 5.0).astype(np.float32)
    kk, vv = c2.k.copy(), c2.v.copy()
    oracle.fake_quantize_pages(c2, 2)
    assert np.array_equal(c2.k, kk) and np.array_equal(c2.v, vv)
    # page ranges are per request
    c3, _, _, _, _, _ = ragged_batch_cache("HND", False, seed=9)
    before = c3.k.copy()
    oracle.fake_quantize_pages(c3, 4, page_begin=[1, 0, 0], page_end=[2, 0, 0])
    changed = {blk for blk in range(c3.num_blocks) if not np.array_equal(c3.k[blk], before[blk])}
    assert changed == {int(c3.block_table[0, 1])}


# ------------------------------------------------------------------ int8-basis and bf16-basis formats (App. B ablation)

@pytest.mark.parametrize("fmt,r", [(oracle.FMT_I8, 8), (oracle.FMT_I8, 3), (oracle.FMT_BF16, 8), (oracle.FMT_BF16, 5)])
def test_wide_basis_formats_roundtrip_and_sizes(fmt, r):
    """The int8-basis and the bf16-basis ("r8fp") summaries: payload arithmetic, quantiser identities against numpy,
    and the ordering of the three basis precisions on the same page (the score error shrinks with the basis width,
    as in the paper's rank x precision ablation)."""
    B, d = 16, 128
    want = (d * r + B * r + d + 2 * (r + B + 1)) if fmt == oracle.FMT_I8 else (2 * d * r + B * r + d + 2 * (B + 1))
    assert oracle.summary_payload_bytes(fmt, r) == want
    assert oracle.summary_stride_bytes(fmt, r) == (want + 15) // 16 * 16
    keys = low_rank_page(6, noise=0.1, seed=41)
    mu, V, Cc, lam, r_eff = oracle.build_page(keys, r)
    blob = oracle.pack(fmt, mu, V, Cc)
    mu2, V2, C2 = oracle.unpack(fmt, r, blob)
    if fmt == oracle.FMT_I8:
        sV = np.float16(np.abs(V).max(1) / 127).astype(np.float64)
        codes = np.clip(np.rint(V / sV[:, None]), -127, 127)
        assert np.array_equal(V2, codes * sV[:, None])
    else:
        import torch
        assert np.array_equal(V2, torch.from_numpy(V).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy())
    sC = np.float16(np.abs(Cc).max(1) / 127).astype(np.float64)
    assert np.array_equal(C2, np.clip(np.rint(Cc / np.where(sC > 0, sC, 1)[:, None]), -127, 127) * sC[:, None])
    sMu = float(np.float16(np.abs(mu).max() / 127))
    assert np.array_equal(mu2, np.clip(np.rint(mu / sMu), -127, 127) * sMu)
    # every byte of the payload is used, padding stays zero
    assert not blob[want:].any()
    if r == 8:
        rng = np.random.default_rng(5)
        errs = {}
        for f in (oracle.FMT_I4, oracle.FMT_I8, oracle.FMT_BF16):
            m = oracle.unpack(f, r, oracle.pack(f, mu, V, Cc))
            errs[f] = np.mean([abs(oracle.score(*m, q, SM) - oracle.score(mu, V, Cc, q, SM))
                               for q in rng.standard_normal((40, d))])
        assert errs[oracle.FMT_I4] > errs[oracle.FMT_I8] and errs[oracle.FMT_I4] > errs[oracle.FMT_BF16]
