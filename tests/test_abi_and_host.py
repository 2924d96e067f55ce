"""CPU tests: the C-ABI library loads and exports every declared symbol; host-side logic."""
import ctypes
import os
import re
import socket

import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    import __graft_entry__ as ge
    ge.build()
    from paper_2607_24555_b200 import binding
    header = open(os.path.join(ROOT, "include", "locks.h")).read()
    declared = set(re.findall(r"\b(locks_[a-z_]+)\s*\(", header))
    declared -= {"locks_create()"}
    assert {"locks_build_summaries", "locks_select", "locks_sparse_attend", "locks_decode_step"} <= declared
    lib = ctypes.CDLL(binding.library_path())
    for name in sorted(declared):
        assert hasattr(lib, name), name
    assert set(binding.SYMBOLS) == declared


def test_size_helpers_and_validation_need_no_gpu():
    import paper_2607_24555_b200 as locks
    from paper_2607_24555_b200.binding import make_config
    assert locks.locks_summary_bytes(make_config(32, 8, 8, "i4", "bf16", 8, 2048, 2048)) == 832
    assert locks.locks_summary_bytes(make_config(32, 8, 4, "i4", "bf16", 8, 2048, 2048)) == 496
    assert locks.locks_summary_bytes(make_config(32, 8, 2, "i4", "bf16", 8, 2048, 2048)) == 336
    assert locks.locks_summary_bytes(make_config(4, 1, 8, "f32", "f32", 1, 256, 256)) == 5120
    assert locks.locks_workspace_bytes(make_config(32, 2, 8, "i4", "bf16", 1, 65536, 2048)) > 0
    assert locks.locks_workspace_bytes(make_config(34, 2, 8, "i4", "bf16", 1, 64, 256)) == 0    # G = 17
    assert locks.locks_workspace_bytes(make_config(8, 2, 8, "i4", "bf16", 1, 64, 256, d=64)) == 0
    # page sizes of the paper's App. D ablation: 978 / 1298 payload bytes at r = 8 int4, padded to 16
    assert locks.locks_summary_bytes(make_config(32, 8, 8, "i4", "bf16", 8, 2048, 2048, B=32)) == 992
    assert locks.locks_summary_bytes(make_config(32, 8, 8, "i4", "bf16", 8, 2048, 2048, B=64)) == 1312
    assert locks.locks_summary_bytes(make_config(4, 1, 8, "f32", "f32", 1, 256, 256, B=32)) == 4 * (128 + 8 * 128 + 32 * 8)
    assert locks.locks_workspace_bytes(make_config(8, 2, 8, "i4", "bf16", 1, 64, 256, B=48)) == 0
    # the per-head arm ranks and attends one page table per query head: its workspace is the larger one
    grouped = locks.locks_workspace_bytes(make_config(32, 2, 8, "i4", "bf16", 1, 65536, 2048))
    per_head = locks.locks_workspace_bytes(make_config(32, 2, 8, "i4", "bf16", 1, 65536, 2048, combine=locks.COMBINE_PER_HEAD))
    assert per_head > grouped
    assert locks.locks_workspace_bytes(make_config(32, 2, 8, "i4", "bf16", 1, 65536, 2048, combine=4)) == 0
    assert locks.locks_strerror(-6).startswith("page or block")
    assert locks.locks_strerror(0) == "ok"


def test_oracle_and_cuda_path_share_no_code():
    """Neither side imports the other; the generators import neither."""
    src = lambda p: open(os.path.join(ROOT, p)).read()
    assert "oracle" not in src("paper_2607_24555_b200/binding.py").replace("no CPU or PyTorch fallback", "")
    assert "paper_2607_24555_b200" not in src("oracle/__init__.py")
    assert "locks.h" not in src("oracle/locks_oracle.c") and "csrc" not in src("oracle/locks_oracle.c")
    g = src("locks_synth/__init__.py")
    assert "import oracle" not in g and "import paper_2607_24555_b200" not in g
    for f in os.listdir(os.path.join(ROOT, "paper_2607_24555_b200", "csrc")):
        assert "oracle" not in src(os.path.join("paper_2607_24555_b200", "csrc", f))


def test_shard_requests_partitions_the_batch():
    from paper_2607_24555_b200.dist import shard_requests
    for n in (1, 7, 8, 64):
        for world in (1, 2, 3, 8):
            parts = [shard_requests(n, r, world) for r in range(world)]
            assert sorted(sum(parts, [])) == list(range(n))
            assert max(map(len, parts)) - min(map(len, parts)) <= 1


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    import torch.distributed as dist
    from paper_2607_24555_b200.dist import max_over_ranks, sum_over_ranks, shard_requests, barrier
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    mine = shard_requests(9, rank, world)
    barrier()
    t = max_over_ranks(10.0 + rank)            # the step time the benchmark reports
    total = sum_over_ranks(float(len(mine)))   # units all ranks processed
    q.put((rank, mine, t, total))
    dist.destroy_process_group()


def test_two_rank_gloo_timing_reduction():
    """world_size 2 on CPU: requests are sharded with no data-path collective, the reported time is
    the max over ranks and the work the sum."""
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(60)
    assert res[0][1] == [0, 1, 2, 3, 4] and res[1][1] == [5, 6, 7, 8]
    assert res[0][2] == res[1][2] == 11.0
    assert res[0][3] == res[1][3] == 9.0
