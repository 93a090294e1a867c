"""CPU-side checks: the C-ABI library builds, loads and exports what include/pd.h declares;
host-side logic of the benchmark's multi-rank aggregation runs under gloo with two ranks."""
import ctypes
import os
import re
import subprocess
import sys

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def header_functions():
    names = set()
    for f in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if f.endswith(".h"):
            text = open(os.path.join(ROOT, "include", f)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(pd_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2609_35158_b200 import build as pd_build

    lib_path = pd_build.build_library()
    lib = ctypes.CDLL(lib_path)
    declared = header_functions()
    assert {"pd_create", "pd_destroy", "pd_kv_append", "pd_decode_attn", "pd_decode_step_host"} <= set(declared)
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in pd.h but not exported"
    import paper_2609_35158_b200 as pd

    assert sorted(pd.EXPORTS) == declared
    for name in declared:
        assert callable(getattr(pd, name)), f"binding lacks {name}"
    assert pd.pd_version() >= 100
    assert pd.pd_status_string(pd.PD_ERR_UNSUPPORTED) == "unsupported geometry"


def test_create_rejects_bad_geometry_before_touching_the_device():
    import paper_2609_35158_b200 as pd

    for args, code in (((8, 3, 64, 16, 4, 4, 16), pd.PD_ERR_INVALID_ARG),
                       ((8, 2, 96, 16, 4, 4, 16), pd.PD_ERR_UNSUPPORTED),
                       ((8, 2, 64, 8, 4, 4, 16), pd.PD_ERR_UNSUPPORTED),
                       ((32, 2, 64, 16, 4, 4, 16), pd.PD_ERR_UNSUPPORTED),
                       ((8, 2, 64, 16, 0, 4, 16), pd.PD_ERR_INVALID_ARG),
                       ((8, 2, 64, 16, 5000, 4, 16), pd.PD_ERR_INVALID_ARG),
                       ((8, 2, 64, 16, 4, 4, 1 << 40), pd.PD_ERR_UNSUPPORTED)):
        with pytest.raises(pd.PdError) as e:
            pd.pd_create(*args)
        assert e.value.code == code
    if not torch.cuda.is_available():  # no device: a clean error code, not a crash
        with pytest.raises(pd.PdError) as e:
            pd.pd_create(8, 2, 64, 16, 4, 4, 16)
        assert e.value.code == pd.PD_ERR_CUDA


def test_pool_calls_reject_bad_arguments_without_a_device():
    import paper_2609_35158_b200 as pd

    for args in ((0, 0, 0), (-1, 1 << 20, 0)):
        with pytest.raises(pd.PdError) as e:
            pd.pd_pool_create(*args)
        assert e.value.code == pd.PD_ERR_INVALID_ARG
    assert pd.pd_pool_base(None) == 0 and pd.pd_pool_capacity(None) == 0 and pd.pd_pool_resident_bytes(None) == 0
    pd.pd_pool_destroy(None)
    if not torch.cuda.is_available():
        with pytest.raises(pd.PdError) as e:
            pd.pd_pool_create(0, 1 << 20)
        assert e.value.code == pd.PD_ERR_CUDA


def test_product_path_does_not_import_the_oracle():
    for rel in ("paper_2609_35158_b200/__init__.py", "paper_2609_35158_b200/build.py"):
        src = open(os.path.join(ROOT, rel)).read()
        assert "oracle" not in src
    for f in os.listdir(os.path.join(ROOT, "paper_2609_35158_b200", "csrc")):
        assert "oracle" not in open(os.path.join(ROOT, "paper_2609_35158_b200", "csrc", f)).read()
    assert "paper_2609_35158_b200" not in open(os.path.join(ROOT, "oracle", "__init__.py")).read()


WORKER = r"""
import os, sys
sys.path.insert(0, {root!r})
import numpy as np, torch, torch.distributed as dist
import bench, workloads as wl
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=rank, world_size=world)
lens = wl.context_lengths(1)
mine = wl.shard_sequences(lens, world)[rank]
local_tokens = float(lens[mine].sum())
ms, tokens = bench.aggregate_over_ranks(10.0 + 5.0 * rank, local_tokens, world)
assert ms == 15.0, ms                      # max over ranks
assert tokens == float(lens.sum()), tokens # every sequence on exactly one rank
gathered = [None] * world
dist.all_gather_object(gathered, mine.tolist())
assert sorted(sum(gathered, [])) == list(range(len(lens)))
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def test_two_rank_sharding_and_aggregation_under_gloo(tmp_path):
    import socket

    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT, port=port))
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    for p in procs:
        out, _ = p.communicate(timeout=180)
        assert p.returncode == 0, out


def test_error_metric_helper():
    from pd_testlib import error_metrics

    ref = np.zeros((2, 3, 4)); ref[..., 0] = 1.0
    got = torch.tensor(ref, dtype=torch.bfloat16)
    assert error_metrics(got, ref) == (0.0, 0.0)
    got[0, 0, 1] = 0.5
    m, r = error_metrics(got, ref)
    assert m == 0.5 and abs(r - 0.5) < 1e-12


def test_reference_arm_prints_the_contract_line():
    """bench.py --impl reference times the oracle on the host cores and prints one JSON line with the keys the
    driver reads (runs on the smallest configuration here)."""
    import json

    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "0",
                          "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    r = json.loads(lines[0])
    assert r["impl"] == "reference" and r["n_gpus"] == 1 and r["steps"] == 2 and r["warmup"] == 1
    assert r["unit"] == "GB/s" and r["higher_is_better"] is True and r["value"] > 0 and r["gpu_launches"] == 0
    assert r["cpu_baseline"]["kind"] == "oracle" and r["cpu_baseline"]["value"] == r["value"] and r["cpu_baseline"]["cores"] >= 1
    assert r["e2e"] == {"value": r["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert "workload" in r["config"] and r["data"] == "synthetic"


def test_gpus_flag_spawns_that_many_ranks():
    """`bench.py --gpus 2` with no launcher starts two ranks itself (here with the host stand-in step over gloo):
    rank 0 prints one line that carries n_gpus = 2, the max over ranks of the time and the sum of the units."""
    import json

    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "stub", "--gpus", "2", "--steps", "5",
                          "--warmup", "1"], capture_output=True, text=True, timeout=300, cwd=ROOT, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, res.stdout
    r = json.loads(lines[0])
    assert r["n_gpus"] == 2 and r["steps"] == 5 and r["units"] == 300.0 and r["scaling"] == "weak"
    assert r["ms_per_step"] >= 2.0          # rank 1 sleeps 2 ms per step: the slower rank sets the time
    assert r["seeds"] == [4, 1004]          # every replica draws its own batch
    # a launcher that disagrees with --gpus is an error, not a silent 1-GPU run
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "stub", "--gpus", "2"],
                         capture_output=True, text=True, timeout=60, cwd=ROOT, env=dict(env, WORLD_SIZE="1", RANK="0"))
    assert res.returncode != 0 and "WORLD_SIZE" in res.stderr


def test_hooked_steps_are_at_least_three():
    import bench

    for K in (1, 2, 3, 5, 11, 12, 20, 47, 48, 200):
        picks = bench.hooked_steps(K)
        assert len(picks) == len(set(picks)) and all(0 <= i < K for i in picks)
        assert len(picks) >= min(3, K), (K, picks)
    assert len(bench.hooked_steps(20)) == 5 and len(bench.hooked_steps(200)) == 12


def test_header_is_plain_c99_and_cxx():
    """The public headers must be usable from C and from C++ without any CUDA header."""
    for name in ("pd.h", "pd_debug.h"):
        hdr = os.path.join(ROOT, "include", name)
        for cmd in (["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only", "-x", "c", hdr],
                    ["g++", "-std=c++17", "-Wall", "-Werror", "-fsyntax-only", "-x", "c++", hdr]):
            res = subprocess.run(cmd, capture_output=True, text=True)
            assert res.returncode == 0, res.stderr


def test_shipped_build_reads_no_environment_variable_after_create():
    """Tuning knobs exist only in a -DPD_ENABLE_TUNING build: the one getenv of the sources sits under that macro."""
    csrc = os.path.join(ROOT, "paper_2609_35158_b200", "csrc")
    hits = []
    for f in sorted(os.listdir(csrc)):
        lines = open(os.path.join(csrc, f)).read().splitlines()
        hits += [(f, i) for i, line in enumerate(lines) if "getenv" in line]
    assert len(hits) == 1 and hits[0][0] == "pd_api.cu"
    lines = open(os.path.join(csrc, "pd_api.cu")).read().splitlines()
    before = lines[:hits[0][1]]
    assert max(i for i, l in enumerate(before) if l.startswith("#ifdef PD_ENABLE_TUNING")) > \
        max([i for i, l in enumerate(before) if l.startswith("#endif")] + [-1])
    from paper_2609_35158_b200 import build as pd_build

    assert not any("PD_ENABLE_TUNING" in flag for flag in pd_build.NVCC_FLAGS)
