"""The multi-process side of bench.py on CPU: two gloo ranks.

The path does not shard on one GPU, so N GPUs run N independent replicas; what the ranks share is a barrier, the
maximum of their timed regions and the sum of the views they processed.  That plumbing (paper_1806_03925_b200/
replicas.py) and the reference arm's rank handling are exercised here with world_size 2.
"""
import json
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _torchrun(script_args, n=2, timeout=300):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port())] + script_args
    env = dict(os.environ, PYTHONPATH=ROOT, OMP_NUM_THREADS="1")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_two_gloo_ranks_agree_on_the_slowest_time_and_the_whole_job_rate(tmp_path):
    script = tmp_path / "ranks.py"
    script.write_text(textwrap.dedent("""
        import json, sys
        from paper_1806_03925_b200.replicas import Replicas
        r = Replicas.from_env()
        r.init("gloo")
        assert r.world == 2 and r.seed == r.rank
        r.barrier()
        ms = r.max_over_ranks(10.0 + 5.0 * r.rank)          # rank 1 is the slow one
        rate = r.whole_job_rate(1000.0, ms)
        r.barrier()
        open(sys.argv[1] + "/rank%d.json" % r.rank, "w").write(json.dumps({"rank": r.rank, "ms": ms, "rate": rate}))
        r.close()
    """))
    out = _torchrun([str(script), str(tmp_path)])
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(open(tmp_path / ("rank%d.json" % k)).read()) for k in range(2)]
    assert sorted(d["rank"] for d in lines) == [0, 1]
    for d in lines:
        assert d["ms"] == 15.0                               # the maximum over the ranks, on every rank
        assert abs(d["rate"] - 2 * 1000.0 / 15e-3) < 1e-6    # both replicas' units over the slowest time


def test_reference_arm_under_two_ranks_prints_one_line():
    out = _torchrun([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                     "--workload", "tiny"])
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                   # rank 0 alone runs the oracle and reports
    d = lines[0]
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    from paper_1806_03925_b200.replicas import Replicas
    r = Replicas(0, 1, 0)
    r.init("gloo")
    r.barrier()
    assert r.max_over_ranks(3.5) == 3.5 and r.whole_job_rate(10.0, 2.0) == 5000.0
    r.close()
