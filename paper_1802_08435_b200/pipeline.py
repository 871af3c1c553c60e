"""Subscale generation spread over several devices, the samples handed on one way and online (the paper's closing remark of
Section 5.3: with B sub-tensors on a rack of devices "the generated bits are sent one-way and online from each device to the
next").  Host-side protocol only; what generates a rank's rows is a callback (on a GPU: `binding.wrnn_subscale_net_rows`).

Rank r of N owns the B / N consecutive sub-tensors r B / N .. (r + 1) B / N - 1.  Global time advances one chunk at a time
as in the staggered schedule of one device: at chunk k, row z is at position k * chunk - z * lag.  A row needs the rows
before it up to F positions ahead of its own; lag >= F + chunk puts every earlier row a whole chunk further ahead than that,
which is the slack the links use: after chunk k a rank sends its successor ONE message with what its own rows generated in
chunk k and what it received itself before chunk k (so a row owned j ranks back arrives j - 1 chunks late, and is j B / N
lags ahead).  Links are strictly next-neighbour and one way; every message starts with (chunk index, number of samples) so
that a lost or reordered message is noticed; a receive waits at most `timeout_s` and then raises -- it never waits forever.
The receiver copies the samples into its own history before it uses them.
"""
from __future__ import annotations

import datetime
from typing import Callable, List, Tuple

import numpy as np

Segment = Tuple[int, int, int]     # (row, first position, number of positions)


class PipelineError(RuntimeError):
    pass


def rows_of(rank: int, world: int, B: int) -> Tuple[int, int]:
    if B % world:
        raise ValueError("the number of sub-tensors must be a multiple of the number of devices")
    per = B // world
    return rank * per, (rank + 1) * per


def n_chunks(B: int, L: int, chunk: int, lag: int) -> int:
    """Global chunks until the last row is done."""
    return -(-((B - 1) * lag + L) // chunk)


def generated_in_chunk(k: int, row: int, L: int, chunk: int, lag: int) -> Segment:
    """What row `row` generates during global chunk k: (row, first position, count); count 0 outside its lifetime."""
    p = k * chunk - row * lag
    if p < 0 or p >= L:
        return (row, max(p, 0), 0)
    return (row, p, min(chunk, L - p))


def outgoing_segments(rank: int, world: int, B: int, L: int, chunk: int, lag: int, k: int) -> List[Segment]:
    """The message rank -> rank + 1 after global chunk k: the rank's own rows' samples of chunk k, and, for the rows owned j
    ranks back, what they generated in chunk k - j (it reached this rank before chunk k - j + 1 ... and is passed on now)."""
    segs: List[Segment] = []
    per = B // world
    for owner in range(rank + 1):
        kk = k - (rank - owner)
        if kk < 0:
            continue
        for row in range(owner * per, (owner + 1) * per):
            seg = generated_in_chunk(kk, row, L, chunk, lag)
            if seg[2] > 0:
                segs.append(seg)
    return segs


def own_calls(rank: int, world: int, B: int, L: int, chunk: int, lag: int, k: int) -> List[Tuple[int, int, int, int]]:
    """The stepping calls (first row, rows, position of the first row, steps) of this rank's rows in global chunk k: rows that
    run a whole chunk go together, a row that ends inside the chunk goes alone (all rows of a call take the same steps)."""
    lo, hi = rows_of(rank, world, B)
    live = [generated_in_chunk(k, r, L, chunk, lag) for r in range(lo, hi)]
    live = [s for s in live if s[2] > 0]
    calls = []
    full = [s for s in live if s[2] == chunk]
    for s in live:
        if s[2] != chunk:
            calls.append((s[0], 1, s[1], s[2]))
    if full:
        calls.append((full[0][0], len(full), full[0][1], chunk))
    return calls


class SubscalePipeline:
    """One rank of the pipeline.  `dist` is torch.distributed (initialised by the launcher) or None for a single rank;
    `device` the torch device of the message tensors (cpu for gloo, the rank's GPU for nccl)."""

    def __init__(self, dist, rank: int, world: int, B: int, L: int, F: int, chunk: int, lag: int, device="cpu", timeout_s: float = 30.0):
        if lag < F + chunk or lag % chunk:
            raise ValueError("lag must be a multiple of chunk and at least F + chunk")
        self.dist, self.rank, self.world = dist, rank, world
        self.B, self.L, self.F, self.chunk, self.lag = B, L, F, chunk, lag
        self.device, self.timeout_s = device, timeout_s
        self.lo, self.hi = rows_of(rank, world, B)
        self.sent = self.received = 0

    # ---- messages: int32 [2 + n]: (chunk index, n, samples widened to int32)
    def _pack(self, hist, k: int, segs: List[Segment]):
        import torch
        parts = [hist[r, p:p + n].to(torch.int32) for (r, p, n) in segs]
        body = torch.cat(parts) if parts else torch.zeros(0, dtype=torch.int32, device=hist.device)
        head = torch.tensor([k, int(body.numel())], dtype=torch.int32, device=hist.device)
        return torch.cat([head, body]).to(self.device)

    def _unpack(self, msg, hist, k: int, segs: List[Segment]):
        import torch
        n = sum(s[2] for s in segs)
        if int(msg[0]) != k or int(msg[1]) != n:
            raise PipelineError("rank %d expected message (chunk %d, %d samples), got (chunk %d, %d samples)" % (self.rank, k, n, int(msg[0]), int(msg[1])))
        o = 2
        for (r, p, c) in segs:
            hist[r, p:p + c] = msg[o:o + c].to(hist.device).to(torch.int16)      # the consumer's own copy
            o += c

    def _recv(self, k: int, hist):
        import torch
        segs = outgoing_segments(self.rank - 1, self.world, self.B, self.L, self.chunk, self.lag, k)
        msg = torch.zeros(2 + sum(s[2] for s in segs), dtype=torch.int32, device=self.device)
        work = self.dist.irecv(msg, src=self.rank - 1)
        try:
            done = work.wait(datetime.timedelta(seconds=self.timeout_s))
        except RuntimeError as e:
            raise PipelineError("rank %d: no message for chunk %d from rank %d within %.1f s (%s)" % (self.rank, k, self.rank - 1, self.timeout_s, str(e)[:80]))
        if done is False:
            raise PipelineError("rank %d: no message for chunk %d from rank %d within %.1f s" % (self.rank, k, self.rank - 1, self.timeout_s))
        self._unpack(msg, hist, k, segs)
        self.received += 1

    def n_iterations(self) -> int:
        """Iterations of `step` this rank runs: the global chunks, plus one per rank upstream to pass their last samples on."""
        return n_chunks(self.B, self.L, self.chunk, self.lag) + self.rank

    def step(self, k: int, hist, generate: Callable[[int, int, int, int], None]) -> None:
        """Iteration k: take in what the predecessor knew after chunk k - 1, generate this rank's rows of chunk k, pass on."""
        if self.rank > 0 and k >= 1:
            self._recv(k - 1, hist)
        if k < n_chunks(self.B, self.L, self.chunk, self.lag):
            for (r_lo, n_rows, p_lo, n) in own_calls(self.rank, self.world, self.B, self.L, self.chunk, self.lag, k):
                generate(r_lo, n_rows, p_lo, n)
        if self.rank < self.world - 1:
            msg = self._pack(hist, k, outgoing_segments(self.rank, self.world, self.B, self.L, self.chunk, self.lag, k))
            self.dist.send(msg, dst=self.rank + 1)
            self.sent += 1

    def run(self, hist, generate: Callable[[int, int, int, int], None]) -> None:
        """hist: this rank's int16 [B][L] history (torch tensor, zeroed); generate(r_lo, n_rows, p_lo, n) advances the given rows of
        it in place.  On return the rows up to this rank's last are complete; the last rank holds the whole signal."""
        for k in range(self.n_iterations()):
            self.step(k, hist, generate)


def main() -> None:
    """python -m paper_1802_08435_b200.pipeline [--rows 16 --positions 6000]: the Subscale WaveRNN 16x of the benchmark
    (dense H = 896 bf16, ten-layer conditioning network, F = 128, chunk 128) with its sub-tensors spread over the ranks the
    launcher started (one process per GPU, NCCL point-to-point between neighbours); a single process runs all rows itself.
    Prints one JSON line on the last rank (which holds the whole signal)."""
    import argparse
    import json
    import time

    import torch

    from paper_1802_08435_b200 import binding as B, replicas, synth

    ap = argparse.ArgumentParser()
    ap.add_argument("--rows", type=int, default=16)
    ap.add_argument("--positions", type=int, default=6000)
    ap.add_argument("--chunk", type=int, default=128)
    args = ap.parse_args()
    rank, world, local = replicas.rank_env()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = replicas.init("nccl", dev)
    Bsub, L, F, chunk = args.rows, args.positions, 128, args.chunk
    lag = -(-(F + chunk) // chunk) * chunk
    w = synth.make_weights(896)
    frames = torch.from_numpy(synth.make_cond(Bsub, (Bsub * L) // synth.HOP + 2)).to(dev)
    lo, hi = rows_of(rank, world, Bsub)
    model = B.wrnn_create(w, "bf16", max_batch=hi - lo)
    net = B.wrnn_subscale_net_create(synth.make_subscale_net(Bsub))
    hist = torch.zeros((Bsub, L), dtype=torch.int16, device=dev)
    h = torch.zeros((Bsub, 896), dtype=torch.float32, device=dev)
    cp = torch.full((Bsub,), 128, dtype=torch.uint8, device=dev)
    fp = torch.zeros((Bsub,), dtype=torch.uint8, device=dev)
    pipe = SubscalePipeline(dist, rank, world, Bsub, L, F, chunk, lag, device=dev, timeout_s=60.0)

    def gen(r_lo, n_rows, p_lo, n):
        B.wrnn_subscale_net_rows(model, net, frames, lag, hist, h, cp, fp, r_lo, n_rows, p_lo, n, synth.SEED_SAMPLING)
        if world > 1:
            torch.cuda.current_stream().synchronize()       # the samples must be there before they are packed and sent

    replicas.barrier(dist)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    pipe.run(hist, gen)
    torch.cuda.synchronize()
    dt = replicas.max_over_ranks(time.perf_counter() - t0, dist, dev)
    assert B.wrnn_poll_status(model) == 0, B.wrnn_last_error(model)
    if rank == world - 1:
        print(json.dumps({"metric": "audio samples/sec", "value": Bsub * L / dt, "n_gpus": world, "rows_per_gpu": hi - lo, "seconds": dt,
                          "workload": "subscale%d_net_896_bf16_%d over %d device(s), one-way pipeline" % (Bsub, L, world)}), flush=True)
    B.wrnn_subscale_net_destroy(net)
    B.wrnn_destroy(model)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
