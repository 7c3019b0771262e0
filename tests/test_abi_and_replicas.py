"""CPU checks: the shared library exports every entry point the header declares, host-side argument
errors are caught without a GPU, and the replica bookkeeping works over gloo with two processes."""
import ctypes
import os
import re

import pytest
import torch
import torch.multiprocessing as mp

import gen
import paper_2607_12121_b200 as fd
from paper_2607_12121_b200 import replicas

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "flashdiff.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(fd_[a-z_0-9]+)\s*\(", text)
    return sorted(set(n for n in names if n not in ("fd_ctx",)))


def test_every_declared_entry_point_is_exported():
    declared = _declared_functions()
    assert {"fd_create", "fd_partition_regions", "fd_region_activity", "fd_regional_step", "fd_destroy"} <= set(declared)
    lib = ctypes.CDLL(fd.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    assert set(fd.EXPORTS) == set(declared)


def test_workspace_bytes_and_config_checks_need_no_gpu():
    for name in ("tiny", "audio", "image", "mmdit", "video"):
        n = fd.fd_workspace_bytes(fd.make_config(gen.workload(name)))
        assert n > 0 and n % 256 == 0
    assert fd.fd_workspace_bytes(fd.make_config(gen.workload("audio").replace(H=1500))) == 0     # H != heads * dim
    assert fd.fd_workspace_bytes(fd.make_config(gen.workload("audio"), max_batch=0)) == 0
    cfg = fd.make_config(gen.workload("audio"))
    handle = ctypes.c_void_p()
    # null weights / workspace are refused before any CUDA call
    st = fd.lib.fd_create(ctypes.byref(cfg), None, None, 0, ctypes.byref(handle))
    assert st == fd.FD_ERR_INVALID_ARG and not handle.value
    assert b"weights" in fd.lib.fd_last_error(None)
    w = fd.FdWeights(**{k: 16 for k, _ in fd.FdWeights._fields_})
    st = fd.lib.fd_create(ctypes.byref(cfg), ctypes.byref(w), None, 0, ctypes.byref(handle))
    assert st == fd.FD_ERR_WORKSPACE
    assert fd.lib.fd_destroy(None) == fd.FD_ERR_INVALID_ARG
    assert fd.lib.fd_launch_count(None) == 0


def _replica_worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    rep = replicas.from_env()
    replicas.init(rep, "gloo")
    replicas.barrier(rep)
    slow = replicas.max_over_ranks(rep, 10.0 + 5.0 * rank)
    units = replicas.sum_over_ranks(rep, 100.0 * (rank + 1))
    # request placement: both ranks derive the same assignment without talking to each other
    costs = [900, 300, 300, 500, 100, 700]
    where, load = replicas.place_requests(rep, costs)
    mine = float(sum(c for c, g in zip(costs, where) if g == rank))
    placed = replicas.sum_over_ranks(rep, mine)
    out[rank] = (slow, units, replicas.replica_seed(rep, 1000), rep.is_lead, where.tolist(), load.tolist(), placed)
    replicas.barrier(rep)
    replicas.shutdown(rep)


def test_replicas_over_gloo_world_size_two():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_replica_worker, args=(world, 29653, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 15.0                 # the slowest replica sets the job time
    assert res[0][1] == res[1][1] == 300.0                # units of all replicas
    assert res[0][2] != res[1][2]                         # each replica draws its own requests
    assert res[0][3] and not res[1][3]
    assert res[0][4] == res[1][4] == [0, 1, 1, 1, 0, 0]    # 900 | 300 300 500 | then 100, 700 to the lighter side
    assert res[0][5] == res[1][5] == [1700.0, 1100.0]
    assert res[0][6] == 2800.0                            # every request is served exactly once
    assert replicas.job_throughput(300.0, 15.0) == pytest.approx(20000.0)


def test_single_replica_needs_no_process_group():
    rep = replicas.Replica(0, 1, 0)
    replicas.init(rep, "gloo")
    assert replicas.max_over_ranks(rep, 3.5) == 3.5 and replicas.sum_over_ranks(rep, 2.0) == 2.0
    assert not torch.distributed.is_initialized()
