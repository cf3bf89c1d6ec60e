"""The N > 1 plumbing of bench.py on two CPU ranks (gloo): the path shards by token rows with no
data-path collective, so what N ranks share is the launch contract -- per-rank seeds, barrier,
max-over-ranks timing, whole-job aggregation, one JSON line from rank 0."""
import json
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _torchrun(args, nproc=2, port=29571):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={nproc}",
           "--master-addr", "127.0.0.1", "--master-port", str(port)] + args
    env = dict(os.environ, OMP_NUM_THREADS="2")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)


def test_harness_on_two_gloo_ranks(tmp_path):
    script = tmp_path / "ranks.py"
    script.write_text(textwrap.dedent(f"""
        import json, os, sys, time
        sys.path.insert(0, {ROOT!r})
        import bench
        h = bench.Harness(backend="gloo")
        assert h.world == 2 and h.rank in (0, 1)
        seed = h.rank_seed(100)
        h.barrier()
        ms = 10.0 if h.rank == 0 else 30.0            # rank 1 is the slow one
        worst = h.max_over_ranks(ms)
        rate = h.whole_job_rate(units_per_rank_step=6.0, steps=5, ms=worst)
        h.barrier()
        if h.rank == 0:
            print(json.dumps({{"worst": worst, "rate": rate}}))
        with open(os.path.join({str(tmp_path)!r}, f"seed{{h.rank}}"), "w") as f:
            f.write(str(seed))
        h.close()
    """))
    res = _torchrun([str(script)])
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["worst"] == 30.0                        # the max over ranks, not rank 0's own time
    assert abs(out["rate"] - 6.0 * 5 * 2 / 0.030) < 1e-6  # both ranks' units over that time
    seeds = sorted(int(open(tmp_path / f"seed{r}").read()) for r in (0, 1))
    assert seeds == [100, 1100]                        # every rank its own batch


def test_reference_arm_under_torchrun_prints_one_line_from_rank_0():
    res = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                     "--workload", "cfg0_single_layer"], port=29572)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0
