"""The N > 1 plumbing of the benchmark, on CPU with the gloo backend (world size 2): every rank
works on its own problems (no collective on the data path) and the slowest rank sets the time."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys
    sys.path.insert(0, %r)
    import numpy as np
    import torch.distributed as dist
    import bench
    import fgr_inputs as gi
    rank, local_rank, world = bench.dist_env()
    dist.init_process_group("gloo")
    # per-rank step times 3 ms and 5 ms: the job's step time is the maximum
    ms = bench.max_over_ranks(3.0 + 2.0 * rank, world)
    assert ms == 5.0, ms
    seeds = bench.rank_seeds(rank, 4)
    gathered = [None] * world
    dist.all_gather_object(gathered, seeds)
    flat = [s for g in gathered for s in g]
    assert len(set(flat)) == len(flat) == 4 * world          # no two ranks share a problem
    # each rank's problem differs from the other rank's, same shape: weak scaling, whole-job value
    p = gi.make_config("c5", seed=seeds[0], batch=1, M=8, N=16, K=8)
    sums = [None] * world
    dist.all_gather_object(sums, float(gi.bf16_bits_to_f32(p.X).sum()))
    assert sums[0] != sums[1]
    unit, value = bench.unit_and_value("c5", p, ms * 1e-3, n_problems=world)
    assert unit == "TFLOP/s" and abs(value - world * p.flop / 5e-3 / 1e12) < 1e-12
    dist.barrier()
    dist.destroy_process_group()
    print("rank %%d ok" %% rank)
""") % ROOT


def test_two_ranks_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.STDOUT, text=True))
    outs = [p.communicate(timeout=180)[0] for p in procs]
    for rank, (p, out) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, out
        assert "rank %d ok" % rank in out


def test_reference_arm_runs_only_on_rank_zero():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--config", "c1"], env=env, capture_output=True, text=True,
                       timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_reference_arm_prints_the_contract_line():
    import json
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2",
                        "--warmup", "1", "--config", "c1"], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["steps"] == 2 and line["unit"] == "TFLOP/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["value"] == line["value"]
    assert line["config"]["workload"] == "c1" and line["vs_baseline"] is None


def test_gpus_flag_starts_the_ranks_itself():
    """`python bench.py --gpus 2` with no launcher around it starts two ranks (torch.distributed.run on
    127.0.0.1), they meet (gloo here: no GPU), and rank 0 alone prints a line that says n_gpus = 2."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--backend", "gloo", "--plumbing-only"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1 and lines[0]["n_gpus"] == 2 and lines[0]["plumbing_only"] is True
    assert lines[0]["max_over_ranks_check"] == 2.0           # ranks report 1 ms and 2 ms: the slowest one counts


def test_both_arms_name_the_workload_with_the_same_keys():
    """The reference arm's `config` carries the same shape keys, with the same values, as ours (built here
    from the same helper without a GPU), for the default workload - the largest named one."""
    import json
    sys.path.insert(0, ROOT)
    import bench
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                       capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    want = bench.shape_keys(bench.HEADLINE, bench.make_cfg(bench.HEADLINE, materialize=False))
    assert want["workload"] == "c3" and {k: line["config"][k] for k in want} == want


def test_bench_extra_workloads_are_well_formed():
    """The extra bench legs resolve to problems of the documented shapes (no data is generated here)."""
    sys.path.insert(0, ROOT)
    import bench
    import fgr_inputs as gi
    f2 = bench.make_cfg("f2", materialize=False)
    assert (f2.dtype, f2.M, f2.N, f2.K, f2.write_y) == (gi.DTYPE_F32, 4096, 4096, 4096, 1)
    v2 = bench.make_cfg("v2", materialize=False)
    assert (v2.batch, v2.M, v2.N, v2.K, v2.conv_taps, v2.w_shared) == (8, 2048, 4096, 2048, 4, 1)
    assert v2.flop == 2.0 * 8 * 2048 * 4096 * 2048
    v3 = bench.make_cfg("v3", materialize=False)
    assert (v3.batch, v3.M, v3.N, v3.K, v3.conv_rows, v3.conv_taps, v3.conv_width) == (16, 63 * 66 + 64, 1024, 576, 3, 3, 66)
    g2 = bench.make_cfg("g2", materialize=False)
    assert (g2.M, g2.N, g2.K) == (2, 16384, 8192)
    for name in ("c2", "c3", "c4", "c5", "f2", "v2", "g2"):
        assert name in bench.TRAFFIC
    assert set(bench.NSHARD_CONFIGS) == {"c4n"} and "r_max_long" in bench.REDUCE_CONFIGS
