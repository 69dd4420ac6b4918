"""Host-side checks that need no GPU: the shared library exports every declared entry point and
refuses to work without a device; the benchmark's multi-rank timing helper (replicas, max over
ranks) works over gloo with two ranks; the search-sequence generators drive valid configurations."""
import os
import re
import subprocess
import sys

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    import paper_2302_01382_b200 as q
    lib = q.load_library()
    header = open(os.path.join(ROOT, "include", "qcfg.h")).read()
    declared = sorted(set(re.findall(r"\b(qcfg_[a-z0-9_]+)\s*\(", header)))
    assert len(declared) >= 20
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in include/qcfg.h but not exported"
    assert sorted(q.EXPORTS) == declared


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device failure path")
def test_no_device_fails_loudly():
    import paper_2302_01382_b200 as q
    with pytest.raises(q.QcfgError):
        q.Context(0)


def test_layer_struct_matches_header_layout():
    import ctypes as C
    import paper_2302_01382_b200 as q
    # 8 (pointer) + 2*8 + 14*4 = 80 bytes, no padding surprises
    assert C.sizeof(q.LayerStruct) == 80
    assert q.LayerStruct.n_out.offset == 8 and q.LayerStruct.src.offset == 24
    assert q.LayerStruct.residual_from.offset == 76


WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch, torch.distributed as dist
import bench
rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
t = bench.max_over_ranks(10.0 + 5.0 * rank, world)
assert t == 15.0, t
r, lr, w = bench.dist_env()
assert (r, w) == (rank, world)
dist.barrier()
dist.destroy_process_group()
print("ok", rank)
"""


def test_max_over_ranks_with_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29617", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r), LOCAL_RANK=str(r)),
                              stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True) for r in range(2)]
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for r, (p, o) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, o
        assert f"ok {r}" in o


def test_reference_arm_other_ranks_do_no_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1"],
                         env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""
