"""ctypes binding of liblocks.so.  Names mirror include/locks.h; tensors are torch CUDA tensors."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "liblocks.so")

F32, BF16 = 0, 1
FMT_F32, FMT_I4, FMT_I8, FMT_BF16 = 0, 1, 2, 3

SYMBOLS = ["locks_summary_bytes", "locks_workspace_bytes", "locks_create", "locks_destroy",
           "locks_build_summaries", "locks_select", "locks_sparse_attend", "locks_decode_step",
           "locks_decode_step_host", "locks_poll_status", "locks_last_launch_count", "locks_strerror",
           "locks_profile_begin", "locks_profile_end", "locks_profile_read", "locks_sparse_attend_noalloc",
           "locks_set_scan_partition", "locks_selftest_wait_timeout", "locks_last_scan_partition",
           "locks_host_cache_clear", "locks_select_exact", "locks_selection_quality",
           "locks_select_rival", "locks_fake_quantize_pages", "locks_scan",
           "locks_select_scored", "locks_merge_selection", "locks_merge_attention",
           "locks_build_summaries_layers"]


PARTITION_AUTO, PARTITION_STRIDED, PARTITION_BALANCED = 0, 1, 2   # LOCKS_PARTITION_* of include/locks.h
SCORER_SUMMARY, SCORER_CENTROID, SCORER_MOMENT, SCORER_ENVELOPE = 0, 1, 2, 3   # LOCKS_SCORER_*


class LocksError(RuntimeError):
    pass


class Config(C.Structure):
    _fields_ = [("head_dim", C.c_int32), ("page_size", C.c_int32), ("num_q_heads", C.c_int32),
                ("num_kv_heads", C.c_int32), ("rank", C.c_int32), ("summary_fmt", C.c_int32),
                ("kv_dtype", C.c_int32), ("q_dtype", C.c_int32), ("max_batch", C.c_int32),
                ("max_pages_per_seq", C.c_int32), ("budget_tokens", C.c_int32), ("sm_scale", C.c_float),
                ("combine", C.c_int32)]


class KV(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("stride_block", C.c_int64), ("stride_head", C.c_int64),
                ("stride_token", C.c_int64), ("num_blocks", C.c_int32), ("block_table", C.c_void_p),
                ("seq_lens", C.c_void_p)]


_lib = None


def library_path() -> str:
    return _LIB_PATH


def lib():
    """Load liblocks.so (built in-tree by paper_2607_24555_b200.build).  Raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise LocksError(f"{_LIB_PATH} is missing: run `python -m paper_2607_24555_b200.build` "
                             "(there is no CPU or PyTorch fallback)")
        L = C.CDLL(_LIB_PATH)
        vp, i32p = C.c_void_p, C.c_void_p
        L.locks_summary_bytes.restype = C.c_size_t
        L.locks_summary_bytes.argtypes = [C.POINTER(Config)]
        L.locks_workspace_bytes.restype = C.c_size_t
        L.locks_workspace_bytes.argtypes = [C.POINTER(Config)]
        L.locks_create.argtypes = [C.POINTER(Config), vp, C.c_size_t, C.POINTER(vp)]
        L.locks_destroy.argtypes = [vp]
        L.locks_build_summaries.argtypes = [vp, C.POINTER(KV), C.c_int, i32p, i32p, vp, vp]
        L.locks_select.argtypes = [vp, vp, vp, C.POINTER(KV), C.c_int, i32p, i32p, vp, vp, vp]
        L.locks_build_summaries_layers.argtypes = [vp, C.POINTER(KV), vp, vp, C.c_int, C.c_int, i32p, i32p, vp]
        L.locks_build_summaries_layers.restype = C.c_int
        L.locks_sparse_attend.argtypes = [vp, vp, C.POINTER(KV), C.c_int, i32p, i32p, vp, vp, vp]
        L.locks_decode_step.argtypes = [vp, vp, vp, vp, C.POINTER(KV), vp, C.c_int, vp, i32p, i32p, vp]
        L.locks_decode_step_host.argtypes = [vp, vp, vp, vp, C.POINTER(KV), vp, C.c_int, vp, i32p, i32p, vp]
        L.locks_poll_status.argtypes = [vp, C.POINTER(C.c_int32), vp]
        L.locks_last_launch_count.argtypes = [vp]
        L.locks_profile_begin.argtypes = [vp, C.c_int]
        L.locks_profile_end.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(C.c_int)]
        L.locks_profile_read.argtypes = [vp, C.POINTER(C.c_float), vp]
        L.locks_profile_read.restype = C.c_int
        L.locks_profile_begin.restype = C.c_int
        L.locks_profile_end.restype = C.c_int
        L.locks_sparse_attend_noalloc.argtypes = [C.POINTER(Config), vp, C.POINTER(KV), C.c_int, i32p, i32p, vp, vp, vp]
        L.locks_sparse_attend_noalloc.restype = C.c_int
        L.locks_set_scan_partition.argtypes = [vp, C.c_int]
        L.locks_selftest_wait_timeout.argtypes = [vp, C.c_int, vp]
        L.locks_selftest_wait_timeout.restype = C.c_int
        L.locks_set_scan_partition.restype = C.c_int
        L.locks_last_scan_partition.argtypes = [vp]
        L.locks_last_scan_partition.restype = C.c_int
        L.locks_host_cache_clear.argtypes = [vp]
        L.locks_host_cache_clear.restype = C.c_int
        L.locks_select_rival.argtypes = [vp, C.c_int, vp, vp, C.POINTER(KV), C.c_int, i32p, i32p, vp, vp, vp]
        L.locks_select_rival.restype = C.c_int
        L.locks_fake_quantize_pages.argtypes = [vp, C.POINTER(KV), C.c_int, i32p, i32p, C.c_int, vp]
        L.locks_fake_quantize_pages.restype = C.c_int
        L.locks_scan.argtypes = [vp, vp, vp, C.POINTER(KV), C.c_int, vp, vp, vp]
        L.locks_select_scored.argtypes = [vp, vp, vp, C.c_int, C.POINTER(KV), C.c_int, i32p, i32p, vp, vp]
        L.locks_merge_selection.argtypes = [vp, vp, i32p, C.c_int, C.c_int, i32p, i32p, vp]
        L.locks_merge_attention.argtypes = [vp, vp, vp, C.c_int, C.c_int, vp, vp, vp]
        for fn in ("locks_scan", "locks_select_scored", "locks_merge_selection", "locks_merge_attention"):
            getattr(L, fn).restype = C.c_int
        L.locks_select_exact.argtypes = [vp, vp, C.POINTER(KV), C.c_int, i32p, i32p, vp, vp, vp]
        L.locks_select_exact.restype = C.c_int
        L.locks_selection_quality.argtypes = [vp, vp, C.POINTER(KV), C.c_int, i32p, i32p, i32p, i32p, i32p, C.c_int, vp, vp]
        L.locks_selection_quality.restype = C.c_int
        L.locks_strerror.restype = C.c_char_p
        L.locks_strerror.argtypes = [C.c_int]
        for fn in ("locks_create", "locks_destroy", "locks_build_summaries", "locks_select", "locks_sparse_attend",
                   "locks_decode_step", "locks_decode_step_host", "locks_poll_status", "locks_last_launch_count"):
            getattr(L, fn).restype = C.c_int
        _lib = L
    return _lib


def locks_strerror(code: int) -> str:
    return lib().locks_strerror(code).decode()


def locks_summary_bytes(cfg: Config) -> int:
    return int(lib().locks_summary_bytes(C.byref(cfg)))


def locks_workspace_bytes(cfg: Config) -> int:
    return int(lib().locks_workspace_bytes(C.byref(cfg)))


def _check(rc: int, what: str):
    if rc != 0:
        raise LocksError(f"{what} failed: {locks_strerror(rc)} ({rc})")


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


COMBINE_SHARE_AVG, COMBINE_GROUP_MAX, COMBINE_GROUP_MASS, COMBINE_PER_HEAD = 0, 1, 2, 3   # LOCKS_COMBINE_* of include/locks.h


def make_config(Hq, Hkv, rank, fmt, dtype, max_batch, max_pages, budget, sm_scale=None, d=128, B=16,
                combine=COMBINE_SHARE_AVG) -> Config:
    if sm_scale is None:
        sm_scale = d ** -0.5
    dt = BF16 if dtype in ("bf16", torch.bfloat16) else F32
    f = {"i4": FMT_I4, "f32": FMT_F32, "i8": FMT_I8, "bf16": FMT_BF16}[fmt]
    return Config(d, B, Hq, Hkv, rank, f, dt, dt, max_batch, max_pages, budget, sm_scale, combine)


@dataclass
class KVView:
    """A paged cache: torch tensors plus element strides (block, head, token)."""
    k: torch.Tensor
    v: torch.Tensor
    strides: tuple
    num_blocks: int
    block_table: torch.Tensor   # [max_batch, max_pages] int32, device
    seq_lens: torch.Tensor      # [max_batch] int32, device

    def struct(self) -> KV:
        sb, sh, st = self.strides
        return KV(self.k.data_ptr(), self.v.data_ptr(), sb, sh, st, self.num_blocks, self.block_table.data_ptr(),
                  self.seq_lens.data_ptr())


class Context:
    """Owns a locks_ctx and its torch-allocated workspace.  Methods mirror the C entry points."""

    def __init__(self, cfg: Config, device="cuda:0"):
        self.cfg = cfg
        self.device = torch.device(device)
        L = lib()
        nbytes = locks_workspace_bytes(cfg)
        if nbytes == 0:
            raise LocksError("invalid or unsupported configuration")
        self.summary_bytes = locks_summary_bytes(cfg)
        self.k = -(-cfg.budget_tokens // cfg.page_size)
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            base = (self.workspace.data_ptr() + 255) // 256 * 256
            h = C.c_void_p()
            _check(L.locks_create(C.byref(cfg), base, nbytes, C.byref(h)), "locks_create")
        self.handle = h

    def close(self):
        if self.handle:
            lib().locks_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def new_summaries(self, num_blocks: int) -> torch.Tensor:
        return torch.zeros(num_blocks, self.cfg.num_kv_heads, self.summary_bytes, dtype=torch.uint8, device=self.device)

    def locks_build_summaries(self, kv: KVView, batch, summaries, page_begin=None, page_end=None, stream=None):
        s = kv.struct()
        _check(lib().locks_build_summaries(self.handle, C.byref(s), batch, _ptr(page_begin), _ptr(page_end),
                                           _ptr(summaries), _stream(stream)), "locks_build_summaries")

    def locks_build_summaries_layers(self, kv: KVView, k_layers, summaries_layers, batch, page_begin=None, page_end=None,
                                     stream=None):
        """k_layers / summaries_layers: lists of tensors (one per layer).  Returns the two device pointer arrays, which
        the caller keeps alive until the launch has run."""
        import torch
        dev = summaries_layers[0].device
        kp = torch.tensor([t.data_ptr() for t in k_layers], dtype=torch.int64, device=dev)
        sp = torch.tensor([t.data_ptr() for t in summaries_layers], dtype=torch.int64, device=dev)
        s = kv.struct()
        _check(lib().locks_build_summaries_layers(self.handle, C.byref(s), _ptr(kp), _ptr(sp), len(k_layers), batch,
                                                  _ptr(page_begin), _ptr(page_end), _stream(stream)),
               "locks_build_summaries_layers")
        return kp, sp

    def locks_fake_quantize_pages(self, kv: KVView, batch, bits, page_begin=None, page_end=None, stream=None):
        s = kv.struct()
        _check(lib().locks_fake_quantize_pages(self.handle, C.byref(s), batch, _ptr(page_begin), _ptr(page_end), int(bits),
                                               _stream(stream)), "locks_fake_quantize_pages")

    def locks_scan(self, q, summaries, kv: KVView, batch, head_logz, page_logmass=None, stream=None):
        s = kv.struct()
        _check(lib().locks_scan(self.handle, _ptr(q), _ptr(summaries), C.byref(s), batch, _ptr(page_logmass), _ptr(head_logz),
                                _stream(stream)), "locks_scan")

    def locks_select_scored(self, head_logz_parts, kv: KVView, batch, page_ids, page_count, page_logshare=None,
                            page_logmass=None, stream=None):
        s = kv.struct()
        _check(lib().locks_select_scored(self.handle, _ptr(page_logmass), _ptr(head_logz_parts), int(head_logz_parts.shape[0]),
                                         C.byref(s), batch, _ptr(page_ids), _ptr(page_count), _ptr(page_logshare),
                                         _stream(stream)), "locks_select_scored")

    def locks_merge_selection(self, cand_key, cand_page, batch, page_ids, page_count, stream=None):
        _check(lib().locks_merge_selection(self.handle, _ptr(cand_key), _ptr(cand_page), int(cand_key.shape[0]), batch,
                                           _ptr(page_ids), _ptr(page_count), _stream(stream)), "locks_merge_selection")

    def locks_merge_attention(self, part_out, part_lse, batch, out, lse=None, stream=None):
        _check(lib().locks_merge_attention(self.handle, _ptr(part_out), _ptr(part_lse), int(part_out.shape[0]), batch,
                                           _ptr(out), _ptr(lse), _stream(stream)), "locks_merge_attention")

    def locks_select(self, q, summaries, kv: KVView, batch, page_ids, page_count, page_logmass=None,
                     page_logshare=None, stream=None):
        s = kv.struct()
        _check(lib().locks_select(self.handle, _ptr(q), _ptr(summaries), C.byref(s), batch, _ptr(page_ids),
                                  _ptr(page_count), _ptr(page_logmass), _ptr(page_logshare), _stream(stream)),
               "locks_select")

    def locks_select_exact(self, q, kv: KVView, batch, page_ids, page_count, page_logmass=None, page_logshare=None,
                           stream=None):
        s = kv.struct()
        _check(lib().locks_select_exact(self.handle, _ptr(q), C.byref(s), batch, _ptr(page_ids), _ptr(page_count),
                                        _ptr(page_logmass), _ptr(page_logshare), _stream(stream)), "locks_select_exact")

    def locks_select_rival(self, scorer, q, summaries, kv: KVView, batch, page_ids, page_count, page_score=None,
                           page_logshare=None, stream=None):
        s = kv.struct()
        _check(lib().locks_select_rival(self.handle, int(scorer), _ptr(q), _ptr(summaries), C.byref(s), batch,
                                        _ptr(page_ids), _ptr(page_count), _ptr(page_score), _ptr(page_logshare),
                                        _stream(stream)), "locks_select_rival")

    def locks_selection_quality(self, exact_logmass, kv: KVView, batch, page_ids, page_count, ref_ids, ref_count,
                                quality, marked_pages=None, stream=None):
        s = kv.struct()
        n_marked = 0 if marked_pages is None else int(marked_pages.shape[-1])
        _check(lib().locks_selection_quality(self.handle, _ptr(exact_logmass), C.byref(s), batch, _ptr(page_ids),
                                             _ptr(page_count), _ptr(ref_ids), _ptr(ref_count), _ptr(marked_pages),
                                             n_marked, _ptr(quality), _stream(stream)), "locks_selection_quality")

    def locks_sparse_attend(self, q, kv: KVView, batch, page_ids, page_count, out, lse=None, stream=None):
        s = kv.struct()
        _check(lib().locks_sparse_attend(self.handle, _ptr(q), C.byref(s), batch, _ptr(page_ids), _ptr(page_count),
                                         _ptr(out), _ptr(lse), _stream(stream)), "locks_sparse_attend")

    def locks_decode_step(self, q, k_new, v_new, kv: KVView, summaries, batch, out, page_ids=None, page_count=None,
                          stream=None):
        s = kv.struct()
        _check(lib().locks_decode_step(self.handle, _ptr(q), _ptr(k_new), _ptr(v_new), C.byref(s), _ptr(summaries),
                                       batch, _ptr(out), _ptr(page_ids), _ptr(page_count), _stream(stream)),
               "locks_decode_step")

    def locks_decode_step_host(self, q_host, k_new_host, v_new_host, kv: KVView, summaries, batch, out_host,
                               page_ids_host=None, page_count_host=None, stream=None):
        s = kv.struct()
        _check(lib().locks_decode_step_host(self.handle, _ptr(q_host), _ptr(k_new_host), _ptr(v_new_host), C.byref(s),
                                            _ptr(summaries), batch, _ptr(out_host), _ptr(page_ids_host),
                                            _ptr(page_count_host), _stream(stream)), "locks_decode_step_host")

    def locks_poll_status(self, stream=None) -> int:
        st = C.c_int32(0)
        _check(lib().locks_poll_status(self.handle, C.byref(st), _stream(stream)), "locks_poll_status")
        return int(st.value)

    def locks_selftest_wait_timeout(self, limit_ms: int, stream=None):
        _check(lib().locks_selftest_wait_timeout(self.handle, int(limit_ms), _stream(stream)), "locks_selftest_wait_timeout")

    def locks_set_scan_partition(self, mode: int):
        _check(lib().locks_set_scan_partition(self.handle, int(mode)), "locks_set_scan_partition")

    def locks_last_scan_partition(self) -> int:
        return int(lib().locks_last_scan_partition(self.handle))

    def locks_host_cache_clear(self):
        _check(lib().locks_host_cache_clear(self.handle), "locks_host_cache_clear")

    def locks_profile_begin(self, max_steps: int):
        _check(lib().locks_profile_begin(self.handle, max_steps), "locks_profile_begin")

    def locks_profile_end(self):
        ms = (C.c_float * 3)()
        n = C.c_int(0)
        _check(lib().locks_profile_end(self.handle, ms, C.byref(n)), "locks_profile_end")
        return {"scan": ms[0], "select": ms[1], "attend": ms[2]}, int(n.value)

    def locks_profile_read(self, stream=None):
        ms = (C.c_float * 3)()
        _check(lib().locks_profile_read(self.handle, ms, _stream(stream)), "locks_profile_read")
        return {"scan": ms[0], "select": ms[1], "attend": ms[2]}

    def locks_last_launch_count(self) -> int:
        return int(lib().locks_last_launch_count(self.handle))


def locks_sparse_attend_noalloc(cfg: Config, q, kv: KVView, batch, page_ids, page_count, out, lse=None, stream=None):
    """Sparse attention without a context or workspace, for callers that cannot allocate device memory
    (see include/locks.h).  Raises LocksError with the library's message if the problem exceeds the
    built-in scratch."""
    s = kv.struct()
    _check(lib().locks_sparse_attend_noalloc(C.byref(cfg), _ptr(q), C.byref(s), batch, _ptr(page_ids), _ptr(page_count),
                                             _ptr(out), _ptr(lse), _stream(stream)), "locks_sparse_attend_noalloc")
