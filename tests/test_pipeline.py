"""The one-way device pipeline of subscale generation (Section 5.3, closing paragraph): host protocol on CPU ranks over gloo,
with the CPU oracle standing in for a device's generator.  The pipelined run must reproduce the oracle's one-process
generation bit for bit; a message that never comes ends in an error, not in an endless wait."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

from paper_1802_08435_b200 import pipeline as pl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_schedule_arithmetic_every_sample_arrives_once_and_in_time():
    for (B, L, F, chunk, lag, world) in ((8, 40, 6, 4, 12, 4), (16, 50, 8, 8, 16, 2), (4, 9, 2, 4, 8, 4), (6, 30, 5, 5, 10, 3)):
        K = pl.n_chunks(B, L, chunk, lag)
        for rank in range(1, world):
            have = {}
            for k in range(K + rank - 1):                     # the messages rank - 1 sends
                for (r, p, n) in pl.outgoing_segments(rank - 1, world, B, L, chunk, lag, k):
                    for q in range(p, p + n):
                        assert (r, q) not in have             # never twice
                        have[(r, q)] = k
            lo, _ = pl.rows_of(rank, world, B)
            assert all((z, q) in have for z in range(lo) for q in range(L))       # everything upstream arrives
            for k in range(K):
                for (r_lo, n_rows, p_lo, n) in pl.own_calls(rank, world, B, L, chunk, lag, k):
                    for b in range(n_rows):
                        p = p_lo - b * lag
                        for z in range(lo):
                            for q in range(p, min(L, p + n + F)):
                                assert have[(z, q)] <= k - 1, (rank, k, z, q)     # before the chunk that needs it
        # the calls of all ranks together are the single-device schedule: every position of every row exactly once, in order
        pos = {r: 0 for r in range(B)}
        for k in range(K):
            for rank in range(world):
                for (r_lo, n_rows, p_lo, n) in pl.own_calls(rank, world, B, L, chunk, lag, k):
                    for b in range(n_rows):
                        assert pos[r_lo + b] == p_lo - b * lag
                        pos[r_lo + b] += n
        assert all(v == L for v in pos.values())


WORKER = r"""
import json, os, sys
import numpy as np, torch, torch.distributed as dist
sys.path.insert(0, sys.argv[1])
from oracle import subscale_net as sn, wrnn_oracle as orc
from paper_1802_08435_b200 import pipeline as pl, synth
mode = sys.argv[2]
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
H, B, L, D, hop, F, chunk, lag, seed = 16, 4, 26, 3, 7, 6, 4, 12, 11
w = synth.make_weights(H, cond_dim=D, seed_w=21, seed_b=22)
om = orc.OracleModel(w, "f32")
net = sn.SubscaleNet(synth.make_subscale_net(B, cond_dim=D, conv_ch=6, res_ch=8, dilations=(1, 2)))
assert net.reach <= F
frames = synth.make_cond(B, (B * L) // hop + 2, D)
hist = torch.zeros((B, L), dtype=torch.int16)
state = {r: (np.zeros((1, H), np.float32), np.array([128], np.uint8), np.array([0], np.uint8)) for r in range(B)}

def generate(r_lo, n_rows, p_lo, n):
    # the oracle as this rank's device: row by row, conditioning from the rank's own copy of the history
    for b in range(n_rows):
        r, p = r_lo + b, p_lo - b * lag
        cond = np.zeros((L, D), np.float32)
        idx = (B * np.arange(p, p + n) + r) // hop
        cond[p:p + n] = frames[r][idx] + net.conditioning(hist.numpy(), r)[p:p + n]
        h, c, f = state[r]
        res = om.run(cond[None], n, 1, seed, hop=1, step0=p, stream0=r, h=h, c_prev=c, f_prev=f)
        hist[r, p:p + n] = torch.from_numpy(res.out[0])
        state[r] = (res.h, res.c_prev, res.f_prev)

pipe = pl.SubscalePipeline(dist, rank, world, B, L, F, chunk, lag, timeout_s=4.0 if mode == "lost" else 60.0)
out = {"rank": rank}
try:
    if mode == "lost" and rank == 0:
        # a sender that stops after its first messages: the failure is made on the host, nothing hangs
        for k in range(3):
            pipe.step(k, hist, generate)
    else:
        pipe.run(hist, generate)
    out["ok"] = True
except pl.PipelineError as e:
    out["ok"] = False
    out["error"] = str(e)
out["sent"], out["received"] = pipe.sent, pipe.received
if rank == world - 1 and out["ok"]:
    ref, _, _ = sn.subscale_net_run(om, net, frames, L, hop, seed)
    out["identical"] = bool(np.array_equal(hist.numpy(), ref))
print(json.dumps(out), flush=True)
if mode != "lost":
    dist.destroy_process_group()
os._exit(0)
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _launch(tmp_path, world, mode):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = _free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT, mode], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        try:
            o, e = p.communicate(timeout=240)
        except subprocess.TimeoutExpired:
            p.kill()
            raise
        assert p.returncode == 0, e[-2000:]
        outs.append(json.loads(o.strip().splitlines()[-1]))
    return sorted(outs, key=lambda r: r["rank"])


@pytest.mark.parametrize("world", [2, 4])
def test_pipeline_over_gloo_reproduces_the_one_process_generation(tmp_path, world):
    outs = _launch(tmp_path, world, "run")
    assert all(o["ok"] for o in outs), outs
    assert outs[-1]["identical"] is True
    K = pl.n_chunks(4, 26, 4, 12)
    for o in outs:                                   # strictly one way: rank r sends K + r messages downstream, the last none
        assert o["sent"] == (K + o["rank"] if o["rank"] < world - 1 else 0)
        assert o["received"] == (K + o["rank"] - 1 if o["rank"] > 0 else 0)


def test_a_message_that_never_comes_ends_in_an_error(tmp_path):
    outs = _launch(tmp_path, 2, "lost")
    assert outs[1]["ok"] is False and "no message for chunk 3" in outs[1]["error"], outs
