"""GPU parity of the masked dilated conditioning network of the Subscale WaveRNN (Sections 4.1, 5.3; the shape the paper
states: ten layers, kernels of size 3, 384 / 768 channels, five dilation stages) and of subscale generation through it,
against the CPU oracle: the conditioning vectors element by element on a random history, the staggered schedule against
the row-after-row order, and every draw of every row against the oracle forced on the device's own samples."""
import numpy as np
import pytest

from oracle import subscale_net as sn
from oracle import wrnn_oracle as orc
from paper_1802_08435_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu

SEED = synth.SEED_SAMPLING


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_1802_08435_b200 import binding as B
    assert torch.cuda.is_available()
    return torch, B


@pytest.mark.parametrize("B_rows,L,dil", [(16, 300, synth.NET_DILATIONS), (8, 130, synth.NET_DILATIONS), (5, 61, (1, 3, 2))])
def test_conditioning_vectors_against_the_oracle(env, B_rows, L, dil):
    """Every sub-tensor's conditioning vectors at every position, on a random history: positions near the row end see
    zeros beyond it, several position tiles per row and a ragged last tile."""
    torch, Bn = env
    dev = "cuda:0"
    w = synth.make_subscale_net(B_rows, dilations=dil)
    net_o = sn.SubscaleNet(w)
    rng = np.random.default_rng(7)
    hist = rng.integers(-32768, 32767, size=(B_rows, L)).astype(np.int16)
    frames = synth.make_cond(B_rows, (B_rows * L) // synth.HOP + 2, synth.COND_DIM)
    net = Bn.wrnn_subscale_net_create(w)
    try:
        h_d, f_d = torch.from_numpy(hist).to(dev), torch.from_numpy(frames).to(dev)
        worst = 0.0
        for row in range(B_rows):
            v = torch.zeros((L, synth.COND_DIM), dtype=torch.float32, device=dev)
            Bn.wrnn_subscale_net_conditioning(net, h_d, f_d, row, v)
            torch.cuda.synchronize()
            assert Bn.wrnn_subscale_net_status(net) == 0
            idx = (B_rows * np.arange(L) + row) // synth.HOP
            ref = frames[row][idx] + net_o.conditioning(hist, row)
            worst = max(worst, pu.rel_err(v.cpu().numpy(), ref))
        print("\n[parity] conditioning network B=%d L=%d layers=%d: worst relative error %.2e" % (B_rows, L, len(dil), worst))
        assert worst < 1e-4
    finally:
        Bn.wrnn_subscale_net_destroy(net)


@pytest.mark.parametrize("H,dtype,B_rows,L,chunk,kernel", [(64, "bf16", 5, 96, 32, "generic"), (896, "bf16", 16, 384, 128, "auto")])
def test_generation_through_the_network(env, H, dtype, B_rows, L, chunk, kernel):
    torch, Bn = env
    dev = "cuda:0"
    w = synth.make_weights(H, cond_dim=synth.COND_DIM, seed_w=31, seed_b=32)
    nw = synth.make_subscale_net(B_rows, dilations=synth.NET_DILATIONS if H > 100 else (1, 2, 4))
    net_o = sn.SubscaleNet(nw)
    F = 128 if H > 100 else 16
    frames = synth.make_cond(B_rows, (B_rows * L) // synth.HOP + 2, synth.COND_DIM)
    om = orc.OracleModel(w, dtype)
    m = Bn.wrnn_create(w, dtype, max_batch=B_rows, kernel=Bn.WRNN_KERNEL_GENERIC if kernel == "generic" else Bn.WRNN_KERNEL_AUTO)
    net = Bn.wrnn_subscale_net_create(nw)
    try:
        f_d = torch.from_numpy(frames).to(dev)

        def run(ch, lag):
            out = torch.zeros((B_rows * L,), dtype=torch.int16, device=dev)
            Bn.wrnn_sample_subscale_net(m, net, f_d, F, ch, lag, B_rows * L, SEED, out)
            torch.cuda.synchronize()
            assert Bn.wrnn_poll_status(m) == 0, Bn.wrnn_last_error(m)
            assert Bn.wrnn_subscale_net_status(net) == 0
            return out.cpu().numpy()

        lag = ((F + chunk + chunk - 1) // chunk) * chunk
        stag = run(chunk, lag)
        if kernel == "generic":      # one kernel family: neither the schedule nor the chunk can change a bit
            seq = run(chunk, ((L + F + chunk) // chunk + 1) * chunk)
            assert np.array_equal(stag, seq)
            assert np.array_equal(run(chunk // 2, 2 * lag), stag)
        got = orc.fold(stag, B_rows)
        want, _, mg = sn.subscale_net_run(om, net_o, frames, L, synth.HOP, SEED, forced=got, teacher=True)
        gc, gf = pu._split(got)
        wc, wf = pu._split(want)
        nd_c, bad_c = pu.check_indices(gc, wc, mg[:, :, 0])
        nd_f, bad_f = pu.check_indices(gf, wf, mg[:, :, 1])
        print("\n[parity] subscale generation through the %d-layer network, H=%d %s: %d rows x %d positions, oracle forced on the device's "
              "samples: idx_diff=%d (near-boundary draws %d, bad %d)" % (net_o.n_layers, H, kernel, B_rows, L, nd_c + nd_f,
                                                                          int((mg < pu.MARGIN).sum()), bad_c + bad_f))
        assert bad_c + bad_f == 0
    finally:
        Bn.wrnn_subscale_net_destroy(net)
        Bn.wrnn_destroy(m)


class _LocalLinks:
    """In-process stand-in for the next-neighbour links of the pipeline (one GPU here): messages queue per destination."""

    def __init__(self):
        self.q = {}

    def send(self, msg, dst):
        self.q.setdefault(dst, []).append(msg.clone())

    def irecv(self, buf, src):
        links, dst = self, src + 1

        class _Work:
            def wait(self, timeout=None):
                if not links.q.get(dst):
                    return False
                buf.copy_(links.q[dst].pop(0))
                return True
        return _Work()


def test_pipeline_ranks_on_one_gpu(env):
    """The device side of the one-way pipeline (Section 5.3): two ranks' worth of sub-tensors generated through
    wrnn_subscale_net_rows on their own history and carry buffers, the samples handed on by the pipeline's messages (ranks
    run turn by turn on the one GPU here); every draw of the last rank's history against the oracle forced on it."""
    torch, Bn = env
    from paper_1802_08435_b200 import pipeline as pl
    dev = "cuda:0"
    H, B_rows, L, chunk, F, world = 896, 16, 384, 128, 128, 2
    lag = F + chunk
    w = synth.make_weights(H, cond_dim=synth.COND_DIM, seed_w=31, seed_b=32)
    nw = synth.make_subscale_net(B_rows)
    frames = synth.make_cond(B_rows, (B_rows * L) // synth.HOP + 2, synth.COND_DIM)
    om, net_o = orc.OracleModel(w, "bf16"), sn.SubscaleNet(nw)
    m = Bn.wrnn_create(w, "bf16", max_batch=B_rows // world)
    net = Bn.wrnn_subscale_net_create(nw)
    try:
        f_d = torch.from_numpy(frames).to(dev)
        links = _LocalLinks()
        ranks = []
        for r in range(world):
            hist = torch.zeros((B_rows, L), dtype=torch.int16, device=dev)
            h = torch.zeros((B_rows, H), dtype=torch.float32, device=dev)
            cp = torch.full((B_rows,), 128, dtype=torch.uint8, device=dev)
            fp = torch.zeros((B_rows,), dtype=torch.uint8, device=dev)
            pipe = pl.SubscalePipeline(links, r, world, B_rows, L, F, chunk, lag, device=dev, timeout_s=1.0)

            def gen(r_lo, n_rows, p_lo, n, hist=hist, h=h, cp=cp, fp=fp):
                Bn.wrnn_subscale_net_rows(m, net, f_d, lag, hist, h, cp, fp, r_lo, n_rows, p_lo, n, SEED)
                torch.cuda.synchronize()
                assert Bn.wrnn_poll_status(m) == 0, Bn.wrnn_last_error(m)
            ranks.append((pipe, hist, gen))
        for k in range(max(p.n_iterations() for p, _, _ in ranks)):
            for pipe, hist, gen in ranks:
                if k < pipe.n_iterations():
                    pipe.step(k, hist, gen)
        got = ranks[-1][1].cpu().numpy()
        assert np.array_equal(ranks[0][1].cpu().numpy()[:B_rows // 2], got[:B_rows // 2])        # what rank 0 made is what rank 1 holds
        want, _, mg = sn.subscale_net_run(om, net_o, frames, L, synth.HOP, SEED, forced=got, teacher=True)
        gc, gf = pu._split(got)
        wc, wf = pu._split(want)
        nd_c, bad_c = pu.check_indices(gc, wc, mg[:, :, 0])
        nd_f, bad_f = pu.check_indices(gf, wf, mg[:, :, 1])
        print("\n[parity] two pipeline ranks x 8 sub-tensors: idx_diff=%d (near-boundary draws %d, bad %d); messages %s" % (
            nd_c + nd_f, int((mg < pu.MARGIN).sum()), bad_c + bad_f, [(p.sent, p.received) for p, _, _ in ranks]))
        assert bad_c + bad_f == 0
    finally:
        Bn.wrnn_subscale_net_destroy(net)
        Bn.wrnn_destroy(m)
