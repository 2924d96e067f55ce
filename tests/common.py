"""Glue shared by the tests: turn a synthetic case into the oracle's numpy cache view and compare
page sets with the tie band.  No method arithmetic lives here."""
from __future__ import annotations

import os

import numpy as np
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_golden(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append([float(x) for x in line.split()])
    return rows


def t2np(t: torch.Tensor) -> np.ndarray:
    """Stored values as numpy: float32 stays float32, bfloat16 becomes its raw uint16 bits."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def bf16_bits_to_f64(a: np.ndarray) -> np.ndarray:
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def np_values(t: torch.Tensor) -> np.ndarray:
    """Stored values as float64."""
    return t.detach().cpu().to(torch.float64).numpy()


def oracle_cache(case) -> oracle.Cache:
    w = case.w
    sb, sh, st = case.strides
    strides = {"shape": (case.num_blocks, w.Hkv, w.B, w.d), "block": sb, "head": sh, "token": st}
    return oracle.Cache(t2np(case.k), t2np(case.v), t2np(case.block_table), t2np(case.seq_lens), w.Hq,
                        strides=strides)


def fmt_code(w) -> int:
    return {"i4": oracle.FMT_I4, "f32": oracle.FMT_F32, "i8": oracle.FMT_I8, "bf16": oracle.FMT_BF16}[w.fmt]


def check_page_sets(ids_gpu, cnt_gpu, ids_ora, cnt_ora, logshare_ora, seq_lens, B, k, band=2e-3):
    """Tie-aware comparison of selected page sets.

    For every (request, KV head): same count; sink and most recent page present; every candidate
    whose oracle log-share is above theta + band is selected, none below theta - band, where theta
    is the oracle's (k-2)-th largest candidate log-share.  Returns the number of problems whose set
    differs from the oracle's at all.
    """
    n, Hkv = cnt_ora.shape
    differed = 0
    for b in range(n):
        P = -(-int(seq_lens[b]) // B)
        for h in range(Hkv):
            assert int(cnt_gpu[b, h]) == int(cnt_ora[b, h]), (b, h, cnt_gpu[b, h], cnt_ora[b, h])
            c = int(cnt_ora[b, h])
            g = ids_gpu[b, h, :c]
            o = ids_ora[b, h, :c]
            assert np.all(ids_gpu[b, h, c:] == -1)
            assert np.all(np.diff(g) > 0), "page ids must be strictly ascending"
            if np.array_equal(g, o):
                continue
            differed += 1
            assert P > k
            gs, os_ = set(g.tolist()), set(o.tolist())
            assert 0 in gs and (P - 1) in gs
            ls = logshare_ora[b, h]
            theta = min(ls[j] for j in os_ if j not in (0, P - 1))
            for j in gs - os_:
                assert ls[j] >= theta - band, (b, h, j, ls[j], theta)
            for j in os_ - gs:
                assert ls[j] <= theta + band, (b, h, j, ls[j], theta)
    return differed
