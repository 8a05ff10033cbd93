"""Workers spread over several ranks: the split round (lqsgd_round_*) and its orchestration.

* On one GPU, two contexts stand for two ranks and are driven one after the other, the test
  playing the collectives (no kernel waits on another): the result must equal, bit for bit, one
  context simulating all the workers.
* On CPU, two gloo processes run paper_2506_17974_b200.distributed.distributed_round with a
  stand-in compressor built from the oracle, which checks the sequence of collectives."""
import os

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import lqsgd_oracle as orc
from paper_2506_17974_b200 import distributed as D
from paper_2506_17974_b200 import workloads as wl

DEV = "cuda:0"


@pytest.mark.gpu
@pytest.mark.parametrize("bits,average", [(4, "codes"), (3, "codes"), (4, "values")])
def test_two_emulated_ranks_equal_one_process_bitwise(bits, average):
    from paper_2506_17974_b200 import binding as B
    w = wl.Workload("dist", ((96, 200), (64, 27), (130, 36), (20, 1), (512, 1152)), rank=4, bits=bits, workers=4,
                    steps=3, dist="student_t3", scale="fan_in", seed=5)
    ref = B.LQSGD(w.layers, w.rank, bits, workers=4, seed=5, average=average)
    ranks = [B.LQSGD(w.layers, w.rank, bits, workers=2, seed=5, world_workers=4, average=average) for _ in range(2)]
    nl = len(w.layers)
    for t in range(3):
        g = wl.draw_gradients(w, t, device=DEV)
        gh_ref = [torch.empty(s, device=DEV) for s in w.layers]
        ref.step(g, gh_ref)
        gh = [[torch.empty(s, device=DEV) for s in w.layers] for _ in range(2)]
        local = [g[0:2], g[2:4]]
        for k in range(2):
            ranks[k].round_begin(local[k], gh[k])
        for which, sid, tid in ((0, B.XCHG_SCALES_P, B.XCHG_STREAMS_P), (1, B.XCHG_SCALES_Q, B.XCHG_STREAMS_Q)):
            views = [ranks[k].exchange_view(sid) for k in range(2)]
            mx = torch.maximum(views[0], views[1])                  # all-reduce MAX
            for v in views:
                v.copy_(mx)
            for k in range(2):
                ranks[k].round_pack(which)
            gathered = torch.cat([ranks[k].exchange_view(tid) for k in range(2)])   # all-gather
            for k in range(2):
                ranks[k].round_reduce(which, gathered, 2)
        for k in range(2):
            ranks[k].round_end()
        torch.cuda.synchronize()
        for l in range(nl):
            if ref.is_matrix(l):
                for k in range(2):
                    assert torch.equal(gh[k][l], gh_ref[l]), (t, l, k)
                    assert torch.equal(ranks[k].get_state(B.STATE_P_BAR, l), ref.get_state(B.STATE_P_BAR, l))
                    assert torch.equal(ranks[k].get_state(B.STATE_Q, l), ref.get_state(B.STATE_Q, l))
                    for wk in range(2):
                        assert torch.equal(ranks[k].get_state(B.STATE_E, l, wk), ref.get_state(B.STATE_E, l, 2 * k + wk))
                        assert torch.equal(ranks[k].get_state(B.STATE_CODES_Q, l, wk), ref.get_state(B.STATE_CODES_Q, l, 2 * k + wk))
            else:
                total = gh[0][l] + gh[1][l]                          # all-reduce SUM of the shares
                assert torch.allclose(total, gh_ref[l], rtol=1e-6, atol=1e-9)
        for k in range(2):
            assert torch.equal(ranks[k].payload(1), ref.payload(2 * k + 1))
    with pytest.raises(B.LqsgdError):
        ranks[0].round_pack(0)                                       # out of order
    with pytest.raises(B.LqsgdError):
        ranks[0].step(local[0], gh[0])                               # a context of a larger world cannot run the fused step


class OracleRank:
    """CPU stand-in with the library's round interface, one layer set, built from the oracle."""

    def __init__(self, layers, rank, bits, alpha, workers, world_workers, Q0):
        self.layers, self.rank, self.bits, self.alpha, self.W, self.Wt = layers, rank, bits, alpha, workers, world_workers
        self.mats = [l for l, s in enumerate(layers) if s[0] > 1 and s[1] > 1]
        self.Q = {l: Q0[l].copy() for l in self.mats}
        self.E = {l: np.zeros((workers,) + tuple(layers[l])) for l in self.mats}
        self.views = {}

    def is_matrix(self, l):
        return l in self.mats

    def round_begin(self, grads, ghat, weights=None, lr=0.0):
        self.ghat = ghat
        self.M, self.P = {}, {}
        for l in self.mats:
            self.M[l] = [orc.error_feedback(grads[w][l].numpy(), self.E[l][w]) for w in range(self.W)]
            self.P[l] = [orc.orthonormalize(orc.power_step_p(m, self.Q[l]))[0] for m in self.M[l]]
        for l, s in enumerate(self.layers):
            if l not in self.mats:
                ghat[l].copy_(torch.from_numpy(np.sum([grads[w][l].numpy() for w in range(self.W)], axis=0) / self.Wt))
        self.views[D.XCHG_SCALES_P] = torch.tensor([float(orc.factor_scale(self.P[l])) for l in self.mats])
        self.cur = self.P

    def exchange_view(self, which):
        return self.views[which]

    def round_pack(self, which):
        scales = self.views[D.XCHG_SCALES_Q if which else D.XCHG_SCALES_P]
        streams = []
        for w in range(self.W):
            for i, l in enumerate(self.mats):
                codes = orc.log_quantize(self.cur[l][w], np.float32(scales[i].item()), self.bits, self.alpha)
                streams.append(orc.pack_codes(codes, self.bits))
        self.views[D.XCHG_STREAMS_Q if which else D.XCHG_STREAMS_P] = torch.from_numpy(np.concatenate(streams))

    def round_reduce(self, which, gathered, n_ranks):
        scales = self.views[D.XCHG_SCALES_Q if which else D.XCHG_SCALES_P]
        per_worker = gathered.numpy().reshape(n_ranks * self.W, -1)
        off, mean = 0, {}
        for i, l in enumerate(self.mats):
            n, m = self.layers[l]
            rows = m if which else n
            count = rows * min(self.rank, n, m)
            nb = (count * self.bits + 7) // 8
            codes = [orc.unpack_codes(per_worker[w, off:off + nb], count, self.bits).reshape(rows, -1)
                     for w in range(n_ranks * self.W)]
            mean[l] = orc.average_dequantize(codes, np.float32(scales[i].item()), self.bits, self.alpha)
            off += nb
        if which == 0:
            self.P_bar = mean
            self.Qw = {l: [orc.power_step_q(m, mean[l]) for m in self.M[l]] for l in self.mats}
            self.views[D.XCHG_SCALES_Q] = torch.tensor([float(orc.factor_scale(self.Qw[l])) for l in self.mats])
            self.cur = self.Qw
        else:
            self.Q = mean

    def round_end(self):
        for l in self.mats:
            G_hat = orc.reconstruct(self.P_bar[l], self.Q[l])
            self.ghat[l].copy_(torch.from_numpy(G_hat).float())
            for w in range(self.W):
                self.E[l][w] = orc.error_update(self.M[l][w], G_hat)


def _gloo_rank(rank, world, port, layers, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = wl.Workload("dist_cpu", tuple(layers), rank=2, bits=4, workers=4, steps=2, dist="normal", scale="fan_in", seed=3)
    rng = np.random.default_rng(0)
    Q0 = {l: rng.standard_normal((s[1], min(2, s[0], s[1]))) for l, s in enumerate(layers) if s[0] > 1 and s[1] > 1}
    comp = OracleRank(layers, 2, 4, 127.0, 2, 4, Q0)
    outs = []
    for t in range(2):
        g = wl.draw_gradients(w, t, device="cpu")[2 * rank:2 * rank + 2]
        ghat = [torch.empty(s) for s in layers]
        D.distributed_round(comp, g, ghat)
        outs.append([x.numpy().copy() for x in ghat])
    np.save(os.path.join(out_dir, f"rank{rank}.npy"), np.concatenate([x.reshape(-1) for o in outs for x in o]))
    dist.destroy_process_group()


def test_distributed_round_over_gloo_matches_single_process_oracle(tmp_path):
    layers = [(24, 40), (12, 1), (16, 36)]
    port = 29500 + os.getpid() % 2000
    mp.spawn(_gloo_rank, args=(2, port, layers, str(tmp_path)), nprocs=2, join=True)
    # reference: one oracle with all 4 workers
    w = wl.Workload("dist_cpu", tuple(layers), rank=2, bits=4, workers=4, steps=2, dist="normal", scale="fan_in", seed=3)
    rng = np.random.default_rng(0)
    Q0 = {l: rng.standard_normal((s[1], min(2, s[0], s[1]))) for l, s in enumerate(layers) if s[0] > 1 and s[1] > 1}
    o = orc.Oracle(layers, 2, 4, 4, 127.0, 4, Q0)
    want = []
    for t in range(2):
        g = [[x.numpy() for x in per] for per in wl.draw_gradients(w, t, device="cpu")]
        out = o.step(g)
        want += [(out[l]["G_hat"] if "G_hat" in out[l] else out[l]["mean"]).reshape(-1) for l in range(len(layers))]
    want = np.concatenate(want)
    for r in range(2):
        got = np.load(tmp_path / f"rank{r}.npy")
        assert np.max(np.abs(got - want)) <= 1e-6 * np.max(np.abs(want))
