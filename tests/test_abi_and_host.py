"""Host-side checks that need no GPU: the C-ABI library loads and exports every function include/cass.h declares,
host-only size queries and argument checks work, and the benchmark's replica reduction (world size 2, gloo)."""
import ctypes
import os
import re
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "cass.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cass_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    sys.path.insert(0, ROOT)
    import __graft_entry__
    __graft_entry__.build()
    import paper_2605_26558_b200 as cass
    names = _declared_functions()
    assert len(names) >= 25 and "cass_draft_step" in names and "cass_verify" in names and "cass_accept" in names
    lib = ctypes.CDLL(cass.binding.LIB_PATH)
    missing = [n for n in names if not hasattr(lib, n)]
    assert not missing, missing
    assert "sm_100a" in cass.cass_version()


def test_host_only_queries_and_argument_checks():
    import paper_2605_26558_b200 as cass
    fmt = cass.default_format()
    bound, ws = cass.cass_encoded_weight_bytes(fmt, 4096, 4096)
    assert bound > 4096 * 4096 * 5 // 8 and ws > 0
    bad = cass.default_format(w_t=9)
    with pytest.raises(cass.CassError) as e:
        cass.cass_encoded_weight_bytes(bad, 64, 64)
    assert e.value.code == cass.ERR_INVALID_ARG
    desc = cass.ModelDesc(2, 256, 4, 2, 64, 688, 1024, 256, 1, 4, 1.0e4, 1.0e-5)
    assert cass.cass_session_bytes(desc, fmt) > 0
    desc2 = cass.ModelDesc(2, 256, 4, 2, 64, 688, 1024, 256, 2, 4, 1.0e4, 1.0e-5)      # two sequences: twice the KV storage
    desc8 = cass.ModelDesc(2, 256, 4, 2, 64, 688, 1024, 256, 8, 4, 1.0e4, 1.0e-5)
    b1, b2, b8 = (cass.cass_session_bytes(d, fmt) for d in (desc, desc2, desc8))
    assert b1 < b2 < b8
    kv_seq = 2 * 2 * 256 * 2 * 64 * 2                    # layers x (K, V) x positions x heads x dim x bf16: the dense caches alone
    assert b2 - b1 >= kv_seq and b8 - b2 >= 6 * kv_seq
    assert [cass.cass_session_rows(d) for d in (desc, desc2, desc8)] == [16, 16, 64]
    desc3 = cass.ModelDesc(2, 256, 4, 2, 64, 688, 1024, 256, 3, 4, 1.0e4, 1.0e-5)      # 3 sequences: not a supported count
    with pytest.raises(cass.CassError) as e:
        cass.cass_session_bytes(desc3, fmt)
    assert e.value.code == cass.ERR_UNSUPPORTED
    wide = cass.ModelDesc(2, 256, 4, 2, 64, 688, 1024, 256, 8, 8, 1.0e4, 1.0e-5)       # 8 x 9 rows exceed one call
    with pytest.raises(cass.CassError) as e:
        cass.cass_session_bytes(wide, fmt)
    assert e.value.code == cass.ERR_INVALID_ARG
    assert cass.cass_calib_norms_count(desc) == 2 * 4 * 688 + 256


def _replica_worker(rank, world, port, q):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    out = bench.combine_replicas(10.0 + rank, 20.0 - rank, 100 + rank, 50 + 2 * rank, world, "cpu")
    dist.destroy_process_group()
    q.put((rank, out))


def test_replica_reduction_world_size_2():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_replica_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for r in range(2):                    # slowest rank's time, all ranks' tokens
        assert res[r] == (11.0, 20.0, 201.0, 102.0)


def test_launch_count_formula():
    sys.path.insert(0, ROOT)
    import bench
    # 10 launches per draft layer (4 projections, RoPE + KV append, attention, merge, 2 norms, SwiGLU) and per verification layer
    assert bench.launches_per_step(32, 4) == 4 * (2 + 32 * 10 + 3) + (2 + 32 * 10 + 3) + 1
    # the count depends neither on the cache length nor on the KV format
    assert bench.launches_per_step(32, 4, max_seq=4096) == bench.launches_per_step(32, 4)
    assert bench.launches_per_step(32, 4, kv_mode=2) == bench.launches_per_step(32, 4)
    # verification from the two parts: two reconstruction launches per matrix
    assert bench.launches_per_step(2, 1, from_parts=True) - bench.launches_per_step(2, 1) == 2 * (2 * 4 + 1)
