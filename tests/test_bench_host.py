"""Host-side logic of bench.py that runs with more than one rank, exercised on CPU with the gloo backend
(two processes on 127.0.0.1): the max-over-ranks reduction of the timings, the whole-job throughput of
independent replicas, and the reference arm, which only rank 0 runs."""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch.distributed as dist
import bench
rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo", rank=rank, world_size=world)
times = [10.0 + 5.0 * rank, 3.0 - rank]          # rank 1 is slower on the first, faster on the second
got = bench.max_over_ranks(times, world, "cpu")
value = bench.whole_job_gbs(1e9, 4, got[0] * 1e-3, world)
dist.barrier()
print(json.dumps({{"rank": rank, "max": got, "value": value}}))
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _spawn(code_or_argv, world, extra_env=None):
    port = _free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), **(extra_env or {}))
        argv = [sys.executable, "-c", code_or_argv] if isinstance(code_or_argv, str) else [sys.executable, *code_or_argv]
        procs.append(subprocess.Popen(argv, env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, cwd=ROOT))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=300)
        assert p.returncode == 0, err[-2000:]
        outs.append(out)
    return outs


def test_timings_are_reduced_to_the_maximum_over_two_gloo_ranks():
    outs = _spawn(WORKER.format(root=ROOT), 2)
    res = [json.loads(o.strip().splitlines()[-1]) for o in outs]
    for r in res:
        assert r["max"] == [15.0, 3.0]                       # slowest rank per entry, same on every rank
        # two replicas of 1 GB per step, 4 steps each, all done within 15 ms
        assert r["value"] == pytest.approx(2 * 1e9 * 4 / 15e-3 / 1e9)


def test_single_process_reduction_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5], 1) == [1.5, 2.5]
    assert bench.whole_job_gbs(2e9, 10, 2.0, 1) == pytest.approx(10.0)


def test_reference_arm_runs_on_rank_zero_only():
    outs = _spawn(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "2", "--warmup", "1", "--config", "tiny"], 2)
    line = json.loads(outs[0].strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
    assert outs[1].strip() == ""                             # the other rank exits 0 without work


def test_the_roofline_names_the_binding_bound_of_each_workload():
    """bench.attention_roofline on the workload shapes: multi-head 60-node trees are bound by HBM, the grouped-query
    ones (7 or 8 query heads per kv head, 60 nodes) by the tensor cores, and the fraction is the floor over the time."""
    sys.path.insert(0, ROOT)
    import bench
    from paper_2509_15235_b200 import synth
    hbm, tflops, mhz, _ = bench.measured_peaks()
    for name, want in (("llava7b", "hbm"), ("llava13b_b4", "hbm"), ("qwen3b_S8192_N16_B4", "hbm"),
                       ("qwen7b", "tensor"), ("qwen3b_S8192_N60_B4", "tensor"), ("qwen3b_S32768_N128_B8", "tensor")):
        cfg = synth.get_config(name)
        kv_len = synth.make_tree_inputs(cfg)["kv_len"]
        r = bench.attention_roofline(cfg, kv_len, 20.0, 148)
        assert r["bound"] == want, (name, r)
        assert abs(r["frac"] - r["floor_us"][want] / 20.0) < 1e-9
        assert r["floor_us"][want] == max(r["floor_us"].values())
        kv_bytes = cfg.kv_bytes_per_layer(kv_len)
        assert abs(r["kv_gbs"] - kv_bytes / 20e-6 / 1e9) < 1e-6
        assert abs(r["floor_us"]["hbm"] - kv_bytes / (hbm * 1e9) * 1e6) < 1e-9
        tokens = sum(int(s) + cfg.N for s in kv_len) * cfg.Hkv
        assert abs(r["floor_us"]["tensor"] - tokens * 4 * cfg.D * cfg.G * cfg.N / (tflops * 1e12) * 1e6) < 1e-9
