"""ctypes front end of the fp64 CPU oracle (``locks_oracle.c``).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the tests, the smoke check and the benchmark's
CPU-baseline leg import this package.  It shares nothing with the CUDA library and never imports
it.  The C file is compiled with gcc on first use (``build()``); all arithmetic lives in C, this
module only marshals numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "locks_oracle.c")
_LIB = os.path.join(_HERE, "liblocks_oracle.so")

F32, BF16, F64 = 0, 1, 2
FMT_F32, FMT_I4, FMT_I8, FMT_BF16 = 0, 1, 2, 3

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


class KV(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("dtype", C.c_int32),
                ("stride_block", C.c_int64), ("stride_head", C.c_int64), ("stride_token", C.c_int64),
                ("num_blocks", C.c_int32), ("block_table", C.c_void_p), ("max_pages", C.c_int32),
                ("seq_lens", C.c_void_p), ("B", C.c_int32), ("d", C.c_int32), ("Hq", C.c_int32),
                ("Hkv", C.c_int32)]


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_LIB)
        L.ora_half_to_double.restype = C.c_double
        L.ora_half_to_double.argtypes = [C.c_uint16]
        L.ora_double_to_half.restype = C.c_uint16
        L.ora_double_to_half.argtypes = [C.c_double]
        L.ora_summary_payload_bytes.restype = C.c_int64
        L.ora_summary_stride_bytes.restype = C.c_int64
        L.ora_score.restype = C.c_double
        L.ora_exact_lse.restype = C.c_double
        L.ora_rival_score.restype = C.c_double
        L.ora_envelope_score.restype = C.c_double
        L.ora_build_page.restype = C.c_int
        L.ora_select_one.restype = C.c_int
        L.ora_select_one_rule.restype = C.c_int
        L.ora_get_max_threads.restype = C.c_int
        _lib = L
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def set_threads(n: int) -> None:
    lib().ora_set_threads(C.c_int(int(n)))


def max_threads() -> int:
    return int(lib().ora_get_max_threads())


def half_to_double(bits: int) -> float:
    return float(lib().ora_half_to_double(C.c_uint16(bits)))


def double_to_half(x: float) -> int:
    return int(lib().ora_double_to_half(C.c_double(x)))


def summary_payload_bytes(fmt: int, r: int, B: int = 16, d: int = 128) -> int:
    return int(lib().ora_summary_payload_bytes(C.c_int(fmt), C.c_int(r), C.c_int(B), C.c_int(d)))


def summary_stride_bytes(fmt: int, r: int, B: int = 16, d: int = 128) -> int:
    return int(lib().ora_summary_stride_bytes(C.c_int(fmt), C.c_int(r), C.c_int(B), C.c_int(d)))


def eigh_jacobi(A):
    """Eigenvalues (descending) and eigenvectors (columns) of a symmetric matrix."""
    A = _f64(A).copy()
    n = A.shape[0]
    U = np.empty((n, n))
    lam = np.empty(n)
    lib().ora_eigh_jacobi(C.c_int(n), _p(A), _p(U), _p(lam))
    return lam, U


def build_page(keys, r: int):
    """keys [B, d] -> (mu [d], V [r, d], C [B, r], lam [B], r_eff)."""
    keys = _f64(keys)
    B, d = keys.shape
    mu, V, Cc, lam = np.empty(d), np.empty((r, d)), np.empty((B, r)), np.empty(B)
    r_eff = lib().ora_build_page(_p(keys), C.c_int(B), C.c_int(d), C.c_int(r), _p(mu), _p(V), _p(Cc), _p(lam))
    return mu, V, Cc, lam, int(r_eff)


def pack(fmt: int, mu, V, Cc) -> np.ndarray:
    mu, V, Cc = _f64(mu), _f64(V), _f64(Cc)
    r, d = V.shape
    B = Cc.shape[0]
    blob = np.zeros(summary_stride_bytes(fmt, r, B, d), dtype=np.uint8)
    lib().ora_pack(C.c_int(fmt), C.c_int(r), C.c_int(B), C.c_int(d), _p(mu), _p(V), _p(Cc), _p(blob))
    return blob


def unpack(fmt: int, r: int, blob, B: int = 16, d: int = 128):
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    mu, V, Cc = np.empty(d), np.empty((r, d)), np.empty((B, r))
    lib().ora_unpack(C.c_int(fmt), C.c_int(r), C.c_int(B), C.c_int(d), _p(blob), _p(mu), _p(V), _p(Cc))
    return mu, V, Cc


def unpack_codes(r: int, blob, B: int = 16, d: int = 128):
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    cV, cC, cMu = np.empty((r, d), np.int32), np.empty((B, r), np.int32), np.empty(d, np.int32)
    sV, sC, sMu = np.empty(r), np.empty(B), np.empty(1)
    lib().ora_unpack_codes(C.c_int(r), C.c_int(B), C.c_int(d), _p(blob), _p(cV), _p(cC), _p(cMu),
                           _p(sV), _p(sC), _p(sMu))
    return cV, cC, cMu, sV, sC, float(sMu[0])


def score(mu, V, Cc, q, sm_scale: float) -> float:
    mu, V, Cc, q = _f64(mu), _f64(V), _f64(Cc), _f64(q)
    r, d = V.shape
    B = Cc.shape[0]
    return float(lib().ora_score(C.c_int(B), C.c_int(d), C.c_int(r), _p(mu), _p(V), _p(Cc), _p(q),
                                 C.c_double(sm_scale)))


def exact_lse(keys, q, sm_scale: float) -> float:
    keys, q = _f64(keys), _f64(q)
    n, d = keys.shape
    return float(lib().ora_exact_lse(C.c_int(n), C.c_int(d), _p(keys), _p(q), C.c_double(sm_scale)))


SCORER_CENTROID, SCORER_MOMENT, SCORER_ENVELOPE = 1, 2, 3


def rival_score(scorer: int, mu, V, Cc, q, sm_scale: float) -> float:
    """Centroid-only (1) or rank-r moment-core (2) score of one page from its summary."""
    mu, V, Cc, q = _f64(mu), _f64(V), _f64(Cc), _f64(q)
    r, d = V.shape
    B = Cc.shape[0]
    return float(lib().ora_rival_score(C.c_int(scorer), C.c_int(B), C.c_int(d), C.c_int(r), _p(mu), _p(V), _p(Cc), _p(q),
                                       C.c_double(sm_scale)))


def envelope_score(keys, q, sm_scale: float) -> float:
    keys, q = _f64(keys), _f64(q)
    n, d = keys.shape
    return float(lib().ora_envelope_score(C.c_int(n), C.c_int(d), _p(keys), _p(q), C.c_double(sm_scale)))


def select_one(s, P: int, k: int):
    """s [G, >=P] page scores of one KV head -> (ids [k] ascending/-1 padded, count, log m_bar [P])."""
    s = _f64(s)
    G, ld = s.shape
    ids = np.full(k, -1, np.int32)
    logshare = np.full(max(P, 1), np.nan)
    cnt = lib().ora_select_one(C.c_int(P), C.c_int(G), C.c_int(k), _p(s), C.c_int64(ld), _p(ids), _p(logshare))
    return ids, int(cnt), logshare


RULE_SHARE_AVG, RULE_GROUP_MAX, RULE_GROUP_MASS = 0, 1, 2


def select_one_rule(s, P: int, k: int, rule: int):
    """select_one under one of the ablated combine rules -> (ids, count, ranking key [P])."""
    s = _f64(s)
    G, ld = s.shape
    ids = np.full(k, -1, np.int32)
    key = np.full(max(P, 1), np.nan)
    cnt = lib().ora_select_one_rule(C.c_int(P), C.c_int(G), C.c_int(k), _p(s), C.c_int64(ld), C.c_int(rule), _p(ids),
                                    _p(key))
    return ids, int(cnt), key


# ----------------------------------------------------------------------------- batch level

def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.float64:
        return F64
    if a.dtype in (np.uint16, np.int16):
        return BF16  # raw bfloat16 bit patterns
    raise TypeError(f"unsupported dtype {a.dtype}")


class Cache:
    """A paged KV cache view held as numpy arrays.

    k, v: [num_blocks, Hkv, B, d] or any layout given by element strides; float32, or uint16
    holding bfloat16 bits.  block_table [batch, max_pages] int32, seq_lens [batch] int32.
    """

    def __init__(self, k, v, block_table, seq_lens, Hq: int, strides=None):
        self.k = np.ascontiguousarray(k)
        self.v = np.ascontiguousarray(v)
        self.block_table = np.ascontiguousarray(block_table, dtype=np.int32)
        self.seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
        nb, Hkv, B, d = self.k.shape if strides is None else strides["shape"]
        self.num_blocks, self.Hkv, self.B, self.d, self.Hq = nb, Hkv, B, d, Hq
        if strides is None:
            sb, sh, st = Hkv * B * d, B * d, d
        else:
            sb, sh, st = strides["block"], strides["head"], strides["token"]
        self.struct = KV(_p(self.k), _p(self.v), _dtype_code(self.k), sb, sh, st, nb,
                         _p(self.block_table), self.block_table.shape[1], _p(self.seq_lens), B, d, Hq, Hkv)
        self.batch = self.block_table.shape[0]
        self.max_pages = self.block_table.shape[1]

    def ref(self):
        return C.byref(self.struct)


def build_summaries(cache: Cache, r: int, fmt: int, summaries=None, page_begin=None, page_end=None):
    stride = summary_stride_bytes(fmt, r, cache.B, cache.d)
    if summaries is None:
        summaries = np.zeros((cache.num_blocks, cache.Hkv, stride), dtype=np.uint8)
    pb = np.ascontiguousarray(page_begin, dtype=np.int32) if page_begin is not None else None
    pe = np.ascontiguousarray(page_end, dtype=np.int32) if page_end is not None else None
    lib().ora_build_summaries(cache.ref(), C.c_int(cache.batch), C.c_int(r), C.c_int(fmt), _p(pb), _p(pe),
                              _p(summaries))
    return summaries


def fake_quantize_pages(cache: Cache, bits: int, page_begin=None, page_end=None):
    """KIVI-style fake quantisation of the complete pages of `cache`, IN PLACE (cache.k / cache.v are overwritten)."""
    pb = np.ascontiguousarray(page_begin, dtype=np.int32) if page_begin is not None else None
    pe = np.ascontiguousarray(page_end, dtype=np.int32) if page_end is not None else None
    lib().ora_fake_quantize_pages(cache.ref(), C.c_int(cache.batch), _p(pb), _p(pe), C.c_int(int(bits)))


def _q_arg(q):
    q = np.ascontiguousarray(q)
    return q, _dtype_code(q)


def page_logmass(cache: Cache, q, r: int, fmt: int, summaries, sm_scale: float, exact: bool = False):
    """s^ (or exact s) for pages 0..P-2 of each request: [batch, Hq, max_pages] (NaN elsewhere)."""
    q, qd = _q_arg(q)
    shat = np.full((cache.batch, cache.Hq, cache.max_pages), np.nan)
    summ = np.ascontiguousarray(summaries, dtype=np.uint8) if summaries is not None else None
    lib().ora_page_logmass(cache.ref(), C.c_int(cache.batch), _p(q), C.c_int(qd), C.c_int(r), C.c_int(fmt),
                           _p(summ), C.c_double(sm_scale), C.c_int(1 if exact else 0), _p(shat))
    return shat


def rival_logmass(cache: Cache, q, r: int, fmt: int, summaries, sm_scale: float, scorer: int):
    """Rival scores of every page: [batch, Hq, max_pages] (NaN where a scorer has no value)."""
    q, qd = _q_arg(q)
    out = np.full((cache.batch, cache.Hq, cache.max_pages), np.nan)
    summ = np.ascontiguousarray(summaries, dtype=np.uint8) if summaries is not None else None
    lib().ora_rival_logmass(cache.ref(), C.c_int(cache.batch), _p(q), C.c_int(qd), C.c_int(r), C.c_int(fmt), _p(summ),
                            C.c_double(sm_scale), C.c_int(scorer), _p(out))
    return out


def select(cache: Cache, shat, k: int):
    shat = _f64(shat)
    ids = np.full((cache.batch, cache.Hkv, k), -1, np.int32)
    cnt = np.zeros((cache.batch, cache.Hkv), np.int32)
    logshare = np.full((cache.batch, cache.Hkv, cache.max_pages), np.nan)
    lib().ora_select(cache.ref(), C.c_int(cache.batch), C.c_int(k), _p(shat), _p(ids), _p(cnt), _p(logshare))
    return ids, cnt, logshare


def select_per_head(cache: Cache, shat, k: int):
    """Per-head arm of the combine ablation: ids [batch, Hq, k], count [batch, Hq], log share [batch, Hq, max_pages]."""
    shat = _f64(shat)
    ids = np.full((cache.batch, cache.Hq, k), -1, np.int32)
    cnt = np.zeros((cache.batch, cache.Hq), np.int32)
    logshare = np.full((cache.batch, cache.Hq, cache.max_pages), np.nan)
    lib().ora_select_per_head(cache.ref(), C.c_int(cache.batch), C.c_int(k), _p(shat), _p(ids), _p(cnt), _p(logshare))
    return ids, cnt, logshare


def page_exact_mass_all(cache: Cache, q, sm_scale: float):
    """Exact log-mass of every page 0..P-1 (last page over its valid tokens): [batch, Hq, max_pages]."""
    q, qd = _q_arg(q)
    mass = np.full((cache.batch, cache.Hq, cache.max_pages), np.nan)
    lib().ora_page_exact_mass_all(cache.ref(), C.c_int(cache.batch), _p(q), C.c_int(qd), C.c_double(sm_scale), _p(mass))
    return mass


def selection_quality(s, P: int, A, R, marked=()):
    """s [G, >=P] exact page log-masses of one KV head; A, R page lists -> (gamma, gamma_c, recall, needle)."""
    s = _f64(s)
    G, ld = s.shape
    A = np.ascontiguousarray(A, dtype=np.int32)
    R = np.ascontiguousarray(R, dtype=np.int32)
    M = np.ascontiguousarray(marked, dtype=np.int32)
    out = np.zeros(4)
    lib().ora_selection_quality(C.c_int(P), C.c_int(G), _p(s), C.c_int64(ld), _p(A), C.c_int(A.size), _p(R),
                                C.c_int(R.size), _p(M) if M.size else None, C.c_int(M.size), _p(out))
    return tuple(float(x) for x in out)


def attend(cache: Cache, q, sm_scale: float, page_ids=None, page_count=None, per_head: bool = False):
    """per_head: page_ids [batch, Hq, k] / page_count [batch, Hq] (one table per query head) instead of per KV head."""
    q, qd = _q_arg(q)
    out = np.zeros((cache.batch, cache.Hq, cache.d))
    lse = np.zeros((cache.batch, cache.Hq))
    k = 0
    if page_ids is not None:
        page_ids = np.ascontiguousarray(page_ids, dtype=np.int32)
        page_count = np.ascontiguousarray(page_count, dtype=np.int32)
        k = page_ids.shape[-1]
    fn = lib().ora_attend_per_head if (per_head and page_ids is not None) else lib().ora_attend
    fn(cache.ref(), C.c_int(cache.batch), _p(q), C.c_int(qd), C.c_double(sm_scale), C.c_int(k),
       _p(page_ids), _p(page_count), _p(out), _p(lse))
    return out, lse


def decode_step(cache: Cache, q, r: int, fmt: int, summaries, sm_scale: float, k: int):
    """score -> select -> attend on resident summaries; returns (ids, count, out, lse)."""
    q, qd = _q_arg(q)
    summ = np.ascontiguousarray(summaries, dtype=np.uint8)
    shat = np.full((cache.batch, cache.Hq, cache.max_pages), np.nan)
    ids = np.full((cache.batch, cache.Hkv, k), -1, np.int32)
    cnt = np.zeros((cache.batch, cache.Hkv), np.int32)
    out = np.zeros((cache.batch, cache.Hq, cache.d))
    lse = np.zeros((cache.batch, cache.Hq))
    lib().ora_decode_step(cache.ref(), C.c_int(cache.batch), _p(q), C.c_int(qd), C.c_int(r), C.c_int(fmt),
                          _p(summ), C.c_double(sm_scale), C.c_int(k), _p(shat), _p(ids), _p(cnt), _p(out),
                          _p(lse))
    return ids, cnt, out, lse
