"""The N>1 path of the benchmark on CPU: two gloo ranks, barrier and max-over-ranks timing."""
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["REPO_ROOT"])
from paper_2609_04098_b200.replicas import Replicas
r = Replicas(backend="gloo")
r.barrier()
ms = 10.0 + 5.0 * r.rank                      # rank 1 is slower
slowest = r.max_over_ranks(ms)
value = r.aggregate(units_per_rank=3.0e12, ms=ms)
r.barrier()
print(json.dumps({"rank": r.rank, "world": r.world, "slowest": slowest, "value": value}))
r.close()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_rank_gloo_barrier_and_max_timing():
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2",
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), REPO_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err
        outs.append(out.strip().splitlines()[-1])
    import json
    res = sorted((json.loads(o) for o in outs), key=lambda d: d["rank"])
    assert [d["rank"] for d in res] == [0, 1] and all(d["world"] == 2 for d in res)
    # both ranks agree on the slowest time and on the aggregate: 2 x 3e12 units in 15 ms
    assert all(abs(d["slowest"] - 15.0) < 1e-9 for d in res)
    assert all(abs(d["value"] - 2 * 3.0e12 / 15e-3) / d["value"] < 1e-12 for d in res)


def test_single_rank_needs_no_process_group(monkeypatch):
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        monkeypatch.delenv(k, raising=False)
    sys.path.insert(0, ROOT)
    from paper_2609_04098_b200.replicas import Replicas
    r = Replicas()
    assert r.world == 1 and r.max_over_ranks(7.5) == 7.5 and r.aggregate(2.0, 1000.0) == 2.0
    r.barrier()
    r.close()


def test_spawn_replicas_starts_one_process_per_rank(tmp_path):
    # what `bench.py --gpus N` does when nobody exported RANK / WORLD_SIZE: N children, rank 0's line is the output
    sys.path.insert(0, ROOT)
    from paper_2609_04098_b200.replicas import spawn_replicas
    script = tmp_path / "worker.py"
    script.write_text(WORKER + "\nopen(os.environ['OUT_DIR'] + '/rank%d' % r.rank, 'w').write(str(r.world))\n")
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    rc = spawn_replicas(2, [sys.executable, str(script)], extra_env={"REPO_ROOT": ROOT, "OUT_DIR": str(tmp_path)},
                        timeout=120)
    assert rc == 0
    assert (tmp_path / "rank0").read_text() == "2" and (tmp_path / "rank1").read_text() == "2"
    assert spawn_replicas(2, [sys.executable, "-c", "import os, sys; sys.exit(3 if os.environ['RANK'] == '1' else 0)"]) == 3
