"""The multi-GPU protocol of the benchmark (independent replicas, barrier + max over ranks) on two CPU ranks over gloo."""
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, sys.argv[1])
from paper_1802_08435_b200 import replicas
rank, world, local = replicas.rank_env()
pg = replicas.init("gloo")
assert pg is not None and pg.get_world_size() == 2
replicas.barrier(pg)
mine = 10.0 + 5.0 * rank                       # rank 1 is the slow one
slowest = replicas.max_over_ranks(mine, pg)
replicas.barrier(pg)
print(json.dumps({"rank": rank, "world": world, "local": local, "seed": replicas.rank_seed(100, rank), "slowest": slowest,
                  "value": replicas.aggregate_throughput(world, 24000, slowest * 1e-3)}))
pg.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_replicas_over_gloo(tmp_path):
    import json
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        try:
            o, e = p.communicate(timeout=120)
        except subprocess.TimeoutExpired:
            p.kill()
            raise
        assert p.returncode == 0, e[-2000:]
        outs.append(json.loads(o.strip().splitlines()[-1]))
    outs.sort(key=lambda r: r["rank"])
    assert [r["rank"] for r in outs] == [0, 1] and all(r["world"] == 2 for r in outs)
    assert outs[0]["seed"] != outs[1]["seed"]                          # replicas draw different streams
    assert outs[0]["slowest"] == outs[1]["slowest"] == 15.0            # every rank reports the slowest rank's time
    assert outs[0]["value"] == pytest.approx(2 * 24000 / 15e-3)        # whole-job samples per second


def test_single_process_needs_no_group(monkeypatch):
    from paper_1802_08435_b200 import replicas
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        monkeypatch.delenv(k, raising=False)
    assert replicas.rank_env() == (0, 1, 0)
    assert replicas.init("gloo") is None
    assert replicas.max_over_ranks(3.5, None) == 3.5
    assert replicas.aggregate_throughput(1, 24000, 0.2) == 120000.0


def test_launch_local_starts_the_ranks_and_reports_failures(tmp_path, monkeypatch):
    """`--gpus N` without a launcher: the benchmark starts its own N ranks.  Two CPU ranks over gloo through that helper;
    a rank that fails makes the launch fail; a world size other than the one asked for is refused."""
    from paper_1802_08435_b200 import replicas
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT"):
        monkeypatch.delenv(k, raising=False)
    assert replicas.needs_launch(2) and not replicas.needs_launch(1)
    script = tmp_path / "worker.py"
    script.write_text(WORKER + "\nreplicas.check_world(2)\nopen(sys.argv[2] + '.%d' % rank, 'w').write(str(slowest))\n")
    mark = str(tmp_path / "done")
    assert replicas.launch_local(2, [sys.executable, str(script), ROOT, mark], timeout_s=120) == 0
    assert open(mark + ".0").read() == open(mark + ".1").read() == "15.0"
    bad = tmp_path / "bad.py"
    bad.write_text("import os, sys\nsys.exit(3 if os.environ['RANK'] == '1' else 0)\n")
    assert replicas.launch_local(2, [sys.executable, str(bad)], timeout_s=60) == 3
    monkeypatch.setenv("WORLD_SIZE", "2")
    assert not replicas.needs_launch(4)
    with pytest.raises(SystemExit):
        replicas.check_world(4)
