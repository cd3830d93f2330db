"""Host-side checks that need no GPU: the built library exports every function the public header declares
(and the binding knows each of them), and the multi-replica reduction of bench.py under a two-process
`gloo` group."""
import ctypes
import os
import re
import socket
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "confspec.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b(cs_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


@pytest.fixture(scope="module")
def library_path():
    from paper_2602_18447_b200 import build
    return build.build()          # compiles with nvcc when the sources are newer; needs no GPU


def test_library_exports_every_declared_function(library_path):
    from paper_2602_18447_b200 import binding
    declared = _declared_functions()
    assert "cs_verify_steps" in declared and "cs_escalate_mask" in declared and len(declared) >= 20
    lib = ctypes.CDLL(library_path)
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in confspec.h but not exported"
    assert sorted(binding.EXPORTED) == declared, set(binding.EXPORTED) ^ set(declared)


def test_binding_declares_signatures_and_pure_host_calls_work(library_path):
    from paper_2602_18447_b200 import binding
    lib = binding.load_library(library_path)
    assert lib.cs_version() >= 100
    assert lib.cs_strerror(binding.CS_EINVAL).decode() == "invalid argument"
    assert lib.cs_strerror(binding.CS_ETIMEOUT)
    # argument errors are reported before anything touches a device
    assert lib.cs_kv_pool_bytes(None, 4, 16) == 0
    assert lib.cs_model_free(None) == binding.CS_OK and lib.cs_kv_free(None) == binding.CS_OK
    assert lib.cs_escalate_mask(None, -1, 0.5, None, None, None, None) == binding.CS_EINVAL
    assert lib.cs_verify_steps(None, None, None, 1, None, 0, None, None, 1, 0.5, None, None, None, None) == \
        binding.CS_EINVAL
    out = ctypes.c_void_p()
    assert lib.cs_model_load(None, None, 0, ctypes.byref(out)) == binding.CS_EINVAL and not out.value
    # more than 128 query heads per kv head leaves no room for a token in a 128-row query tile: refused, not looped on
    desc = binding.cs_model_desc(1, 256, 256, 1, 64, 688, 4096, 1.0e4, 1e-6)
    assert lib.cs_model_load(ctypes.byref(desc), None, 0, ctypes.byref(out)) == binding.CS_EINVAL and not out.value
    assert lib.cs_model_set_lm_head_rows(None, None, 1, None, None) == binding.CS_EINVAL


def test_missing_library_fails_loudly(tmp_path):
    from paper_2602_18447_b200 import binding
    with pytest.raises(FileNotFoundError):
        binding.load_library(str(tmp_path / "libconfspec.so"))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _replica(rank: int, world: int, port: int, q) -> None:
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    from workloads import get_config, make_batch
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        cfg = get_config("cfg1_tiny")
        batch = make_batch(cfg, seed=bench.replica_seed(cfg, rank))
        ms = 10.0 + 5.0 * rank                       # the slower rank decides
        agg = bench.aggregate_over_ranks(ms, 2 * ms, batch.n_steps, batch.n_tokens)
        q.put((rank, agg, int(batch.step_tokens[:8].sum())))
    finally:
        dist.destroy_process_group()


def test_two_replicas_reduce_times_by_max_and_units_by_sum():
    import torch.multiprocessing as mp
    from workloads import get_config, make_batch
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_replica, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    cfg = get_config("cfg1_tiny")
    one = make_batch(cfg)
    for rank, agg, _ in got:
        assert agg == (15.0, 30.0, 2.0 * one.n_steps, 2.0 * one.n_tokens)
    assert got[0][2] != got[1][2]                   # the replicas verify different batches


def test_single_process_aggregation_is_the_identity():
    import bench
    assert bench.aggregate_over_ranks(3.0, 4.0, 16, 1163) == (3.0, 4.0, 16.0, 1163.0)


def test_gpus_flag_without_a_launcher_starts_the_replicas():
    """`python bench.py --gpus 2` started bare must bring up two processes itself. Exercised on the CPU through the
    oracle-timing arm, whose rank 0 prints the line while the other rank exits without work."""
    import json
    import subprocess
    import bench
    cmd = bench.replica_command(2, ["--gpus", "2"], 29999)
    assert "--nproc-per-node=2" in cmd and "127.0.0.1" in cmd and cmd[-2:] == ["--gpus", "2"]
    env = dict(os.environ)
    for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK"):
        env.pop(k, None)
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--workload", "cfg1_tiny", "--steps", "1", "--warmup", "0"],
                         capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                      # one line from rank 0, none from rank 1
    out = json.loads(lines[0])
    assert out["impl"] == "reference" and out["n_gpus"] == 2 and out["value"] > 0
