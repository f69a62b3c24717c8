"""CPU-side checks of the product: the library loads and exports what include/dmtd.h declares,
and the replica timing protocol works across two processes (gloo)."""
import os
import subprocess
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    import __graft_entry__
    __graft_entry__.build()
    import paper_2510_11958_b200 as pkg
    names = pkg.declared_symbols()
    assert {"dmtd_create", "dmtd_prefill", "dmtd_decode_cycle", "dmtd_decode_forced",
            "dmtd_step_layers"} <= set(names)
    dll = pkg.load_library()
    for n in names:
        assert hasattr(dll, n), n


def test_no_cpu_fallback():
    """Without a CUDA device the binding refuses to construct a context."""
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    import paper_2510_11958_b200 as pkg
    from synthetic import SHAPES, make_weights
    shape = SHAPES["tiny"]
    with pytest.raises(pkg.DmtdError):
        pkg.Dmtd(shape, make_weights(shape), L_d=2, tau=3)


def test_product_does_not_import_oracle():
    pkg_dir = os.path.join(ROOT, "paper_2510_11958_b200")
    for dirpath, _, files in os.walk(pkg_dir):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h", ".cpp")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), os.path.join(dirpath, f)


_WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import torch.distributed as dist
from paper_2510_11958_b200 import replicas
rank, world = replicas.init_from_env("gloo")
replicas.barrier()
t, u = replicas.aggregate(10.0 + 5.0 * rank, 100.0 * (rank + 1))
replicas.barrier()
assert world == 2 and t == 15.0 and u == 300.0, (t, u)
if rank == 0:
    print("OK", t, u)
dist.destroy_process_group()
"""


def test_replica_aggregation_two_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER.format(root=ROOT))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    r = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                        "--master-addr", "127.0.0.1", "--master-port", "29731", str(script)],
                       capture_output=True, text=True, timeout=240, env=env)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "OK 15.0 300.0" in r.stdout


def test_bench_gpus_flag_starts_its_own_replicas():
    """`python bench.py --gpus 2` with no launcher around it starts two ranks itself; the dry run
    exercises the rendezvous, the barriers and the max/sum aggregation on gloo, without a GPU."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run-replicas"],
                       capture_output=True, text=True, timeout=240, env=env)
    assert r.returncode == 0, r.stdout + r.stderr
    import json
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert lines == [{"dry_run": True, "n_gpus": 2, "ms_max": 11.0, "units": 200.0}]
