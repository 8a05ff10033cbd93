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
@pytest.mark.parametrize("bits,average,column_scales", [(4, "codes", False), (3, "codes", False), (4, "values", False),
                                                        (32, "codes", False), (5, "codes", True)])
def test_two_emulated_ranks_equal_one_process_bitwise(bits, average, column_scales):
    """Two contexts stand for two ranks, the test plays the five collectives of a round.  Also with the quantiser
    bypassed (the fp32 factors are gathered) and with one scale per factor column (r scales per matrix agreed)."""
    from paper_2506_17974_b200 import binding as B
    w = wl.Workload("dist", ((96, 200), (64, 27), (130, 36), (20, 1), (512, 1152), (1, 77)), rank=4, bits=bits, workers=4,
                    steps=3, dist="student_t3", scale="fan_in", seed=5)
    kw = dict(seed=5, average=average, column_scales=column_scales)
    ref = B.LQSGD(w.layers, w.rank, bits, workers=4, **kw)
    ranks = [B.LQSGD(w.layers, w.rank, bits, workers=2, world_workers=4, **kw) for _ in range(2)]
    nl = len(w.layers)
    wts_ref = [torch.ones(s, device=DEV) for s in w.layers]
    wts = [[torch.ones(s, device=DEV) for s in w.layers] for _ in range(2)]
    for t in range(3):
        g = wl.draw_gradients(w, t, device=DEV)
        gh_ref = [torch.empty(s, device=DEV) for s in w.layers]
        ref.step_update(g, gh_ref, wts_ref, 0.25)
        gh = [[torch.empty(s, device=DEV) for s in w.layers] for _ in range(2)]
        local = [g[0:2], g[2:4]]
        for k in range(2):
            ranks[k].round_begin(local[k], gh[k], wts[k], 0.25)
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
        vecs = [ranks[k].exchange_view(B.XCHG_VECTORS) for k in range(2)]
        assert vecs[0].numel() == 20 + 77
        total = vecs[0] + vecs[1]                                    # all-reduce SUM: every 1-D tensor at once
        for v in vecs:
            v.copy_(total)
        for k in range(2):
            ranks[k].round_end()
        torch.cuda.synchronize()
        for l in range(nl):
            for k in range(2):
                if ref.is_matrix(l):
                    assert torch.equal(gh[k][l], gh_ref[l]), (t, l, k)
                    assert torch.equal(wts[k][l], wts_ref[l]), (t, l, k)
                    assert torch.equal(ranks[k].get_state(B.STATE_P_BAR, l), ref.get_state(B.STATE_P_BAR, l))
                    assert torch.equal(ranks[k].get_state(B.STATE_Q, l), ref.get_state(B.STATE_Q, l))
                    assert torch.equal(ranks[k].get_state(B.STATE_SCALES, l), ref.get_state(B.STATE_SCALES, l))
                    for wk in range(2):
                        assert torch.equal(ranks[k].get_state(B.STATE_E, l, wk), ref.get_state(B.STATE_E, l, 2 * k + wk))
                        if bits != 32:
                            assert torch.equal(ranks[k].get_state(B.STATE_CODES_Q, l, wk), ref.get_state(B.STATE_CODES_Q, l, 2 * k + wk))
                else:                                                # the mean, and the model update of the 1-D tensor
                    assert torch.allclose(gh[k][l], gh_ref[l], rtol=1e-6, atol=1e-9)
                    assert torch.allclose(wts[k][l], wts_ref[l], rtol=1e-6, atol=1e-9)
        for k in range(2):
            assert torch.equal(ranks[k].payload(1), ref.payload(2 * k + 1))
    with pytest.raises(B.LqsgdError):
        ranks[0].round_pack(0)                                       # out of order
    with pytest.raises(B.LqsgdError):
        ranks[0].step(local[0], gh[0])                               # a context of a larger world cannot run the fused step


@pytest.mark.gpu
@pytest.mark.parametrize("overlapped", [False, True])
def test_one_rank_nccl_round_equals_the_fused_step(overlapped):
    """The orchestration on the real thing - the CUDA library and NCCL collectives on CUDA streams - with a
    process group of one rank (all this run has): the split round, whole or cut in two halves on two streams,
    gives bit for bit what lqsgd_step gives."""
    from paper_2506_17974_b200 import binding as B
    if not dist.is_initialized():
        dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{29400 + os.getpid() % 500}", rank=0, world_size=1,
                                device_id=torch.device(DEV))
        import atexit
        atexit.register(lambda: dist.is_initialized() and dist.destroy_process_group())   # shared by both cases of this test
    w = wl.Workload("nccl1", ((96, 200), (64, 27), (130, 36), (20, 1), (256, 1152), (1, 77)), rank=4, bits=4, workers=3,
                    steps=3, dist="student_t3", scale="fan_in", seed=8)
    ref = B.LQSGD(w.layers, w.rank, w.bits, workers=3, seed=8)
    if overlapped:
        idx = D.split_layers(w.layers)
        comps = [B.LQSGD([w.layers[i] for i in part], w.rank, w.bits, workers=3, seed=8, world_workers=3) for part in idx]
        for comp, part in zip(comps, idx):                       # Q_0 is drawn per layer index: take the reference's
            for k, i in enumerate(part):
                if ref.is_matrix(i):
                    comp.set_state(B.STATE_Q, k, 0, ref.get_state(B.STATE_Q, i))
        streams = [torch.cuda.Stream(device=DEV) for _ in range(2)]
    else:
        comp = B.LQSGD(w.layers, w.rank, w.bits, workers=3, seed=8, world_workers=3)
    for t in range(3):
        g = wl.draw_gradients(w, t, device=DEV)
        gh_ref = [torch.empty(s, device=DEV) for s in w.layers]
        gh = [torch.empty(s, device=DEV) for s in w.layers]
        ref.step(g, gh_ref)
        torch.cuda.synchronize()
        if overlapped:
            D.distributed_round_overlapped([(comps[h], [[per[i] for i in idx[h]] for per in g], [gh[i] for i in idx[h]])
                                            for h in range(2)], streams=streams)
        else:
            D.distributed_round(comp, g, gh)
        torch.cuda.synchronize()
        for l in range(len(w.layers)):
            if ref.is_matrix(l):
                assert torch.equal(gh[l], gh_ref[l]), (t, l)
            else:
                assert torch.allclose(gh[l], gh_ref[l], rtol=1e-6, atol=1e-9)
    if not overlapped:
        assert torch.equal(comp.payload(2), ref.payload(2))
        assert torch.equal(comp.get_state(B.STATE_E, 4, 1), ref.get_state(B.STATE_E, 4, 1))


class OracleRank:
    """CPU stand-in with the library's round interface, one layer set, built from the oracle."""

    def __init__(self, layers, rank, bits, alpha, workers, world_workers, Q0):
        self.layers, self.rank, self.bits, self.alpha, self.W, self.Wt = layers, rank, bits, alpha, workers, world_workers
        self.mats = [l for l, s in enumerate(layers) if s[0] > 1 and s[1] > 1]
        self.Q = {l: Q0[l].copy() for l in self.mats}
        self.E = {l: np.zeros((workers,) + tuple(layers[l])) for l in self.mats}
        self.views = {}
        self.vecs = [l for l, s in enumerate(layers) if l not in self.mats]

    def is_matrix(self, l):
        return l in self.mats

    def round_begin(self, grads, ghat, weights=None, lr=0.0):
        self.ghat = ghat
        self.M, self.P = {}, {}
        for l in self.mats:
            self.M[l] = [orc.error_feedback(grads[w][l].numpy(), self.E[l][w]) for w in range(self.W)]
            self.P[l] = [orc.orthonormalize(orc.power_step_p(m, self.Q[l]))[0] for m in self.M[l]]
        shares = [np.sum([grads[w][l].numpy() for w in range(self.W)], axis=0).reshape(-1) / self.Wt for l in self.vecs]
        self.views[D.XCHG_VECTORS] = torch.from_numpy(np.concatenate(shares)) if shares else torch.zeros(0)
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
        off = 0
        for l in self.vecs:                      # the flat buffer was summed over the ranks meanwhile
            k = self.layers[l][0] * self.layers[l][1]
            self.ghat[l].copy_(self.views[D.XCHG_VECTORS][off:off + k].reshape(self.layers[l]).float())
            off += k
        for l in self.mats:
            G_hat = orc.reconstruct(self.P_bar[l], self.Q[l])
            self.ghat[l].copy_(torch.from_numpy(G_hat).float())
            for w in range(self.W):
                self.E[l][w] = orc.error_update(self.M[l][w], G_hat)


def _gloo_rank(rank, world, port, layers, out_dir, overlapped):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    W = 2 * world                                                  # two workers per rank
    w = wl.Workload("dist_cpu", tuple(layers), rank=2, bits=4, workers=W, steps=2, dist="normal", scale="fan_in", seed=3)
    rng = np.random.default_rng(0)
    Q0 = {l: rng.standard_normal((s[1], min(2, s[0], s[1]))) for l, s in enumerate(layers) if s[0] > 1 and s[1] > 1}
    if overlapped:                                                  # the layer table cut in two, one compressor per half
        idx = D.split_layers(layers)
        comps = [OracleRank([layers[i] for i in part], 2, 4, 127.0, 2, W, {k: Q0[i] for k, i in enumerate(part) if i in Q0})
                 for part in idx]
    else:
        comp = OracleRank(layers, 2, 4, 127.0, 2, W, Q0)
    outs = []
    for t in range(2):
        g = wl.draw_gradients(w, t, device="cpu")[2 * rank:2 * rank + 2]
        ghat = [torch.empty(s) for s in layers]
        if overlapped:
            D.distributed_round_overlapped([(comps[h], [[per[i] for i in idx[h]] for per in g], [ghat[i] for i in idx[h]])
                                            for h in range(2)])
        else:
            D.distributed_round(comp, g, ghat)
        outs.append([x.numpy().copy() for x in ghat])
    np.save(os.path.join(out_dir, f"rank{rank}.npy"), np.concatenate([x.reshape(-1) for o in outs for x in o]))
    dist.destroy_process_group()


@pytest.mark.parametrize("world,overlapped", [(2, False), (3, False), (2, True)])
def test_distributed_round_over_gloo_matches_single_process_oracle(tmp_path, world, overlapped):
    """gloo processes run the orchestration with a CPU stand-in built from the oracle: two and three ranks with
    different gradient streams per worker, and the variant with the layer table cut in two halves whose
    exchanges interleave.  Every rank must end up with what ONE oracle holding all the workers computes."""
    layers = [(24, 40), (12, 1), (16, 36), (1, 9), (20, 28)]
    port = 29500 + (os.getpid() * 7 + world * 3 + int(overlapped)) % 2000
    mp.spawn(_gloo_rank, args=(world, port, layers, str(tmp_path), overlapped), nprocs=world, join=True)
    W = 2 * world
    w = wl.Workload("dist_cpu", tuple(layers), rank=2, bits=4, workers=W, steps=2, dist="normal", scale="fan_in", seed=3)
    rng = np.random.default_rng(0)
    Q0 = {l: rng.standard_normal((s[1], min(2, s[0], s[1]))) for l, s in enumerate(layers) if s[0] > 1 and s[1] > 1}
    o = orc.Oracle(layers, 2, 4, 4, 127.0, W, Q0)
    want = []
    for t in range(2):
        g = [[x.numpy() for x in per] for per in wl.draw_gradients(w, t, device="cpu")]
        out = o.step(g)
        want += [(out[l]["G_hat"] if "G_hat" in out[l] else out[l]["mean"]).reshape(-1) for l in range(len(layers))]
    want = np.concatenate(want)
    for r in range(world):
        got = np.load(tmp_path / f"rank{r}.npy")
        assert np.max(np.abs(got - want)) <= 1e-6 * np.max(np.abs(want))


def test_split_layers_balances_the_two_halves():
    layers = wl.resnet18_layers(10)
    a, b = D.split_layers(layers)
    assert sorted(a + b) == list(range(len(layers))) and not set(a) & set(b)
    size = lambda idx: sum(layers[i][0] * layers[i][1] for i in idx if wl.is_matrix(layers[i]))
    assert abs(size(a) - size(b)) <= 0.05 * (size(a) + size(b))
    assert all(i in a for i, s in enumerate(layers) if not wl.is_matrix(s))       # the 1-D tensors ride with the first half
