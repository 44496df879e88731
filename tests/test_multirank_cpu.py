"""The more-than-one-rank path on CPU: two gloo processes, each with its own shard, no exchange on
the data path, the job time taken as the maximum over ranks (CPU only)."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _launch(world, script, args=()):
    port = _free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, WORLD_SIZE=str(world), RANK=str(rank), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), OMP_NUM_THREADS="2")
        procs.append(subprocess.Popen([sys.executable, script, *args], env=env, cwd=ROOT, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=300)
        assert p.returncode == 0, err[-2000:]
        outs.append(out)
    return outs


def test_two_ranks_shard_without_exchange():
    outs = _launch(2, os.path.join(ROOT, "tests", "multirank_worker.py"))
    recs = sorted((json.loads(o.strip().splitlines()[-1]) for o in outs), key=lambda r: r["rank"])
    assert [r["rank"] for r in recs] == [0, 1] and all(r["world"] == 2 and r["joined"] for r in recs)
    # every rank sees the slowest rank's time, and the rate counts both ranks' work over that time
    assert all(r["job_ms"] == 15.0 for r in recs)
    assert all(abs(r["value"] - 2 * r["macs"] / 15e-3) < 1e-6 * r["value"] for r in recs)
    # the ranks hold different data (own seeds) and agree on who holds what
    assert recs[0]["digests"] == recs[1]["digests"] and len(set(recs[0]["digests"])) == 2
    assert recs[0]["checksum"] != recs[1]["checksum"]


def test_single_process_needs_no_group():
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "tests", "multirank_worker.py")], env=env, cwd=ROOT,
                         capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    rec = json.loads(out.stdout.strip().splitlines()[-1])
    assert rec["world"] == 1 and not rec["joined"] and rec["job_ms"] == 10.0


def test_reference_arm_runs_on_rank_zero_only():
    # under a two-rank launch every rank but the first leaves at once, without output
    env = dict(os.environ, WORLD_SIZE="2", RANK="1", LOCAL_RANK="1", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(_free_port()))
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "0"], env=env, cwd=ROOT, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0 and out.stdout.strip() == ""
