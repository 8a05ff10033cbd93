"""lqsgd_step_stats against the oracle: the count of factor entries within one fp32 step of a decision
threshold (an integer decision, taken on both sides on the same fp32 number |x|/s, on the device's own
factors: exact), the pivot ratio of the factor given to Orthonormalize (1e-4), scales, status, code counts
and payload bytes."""
import numpy as np
import pytest
import torch

from oracle import lqsgd_oracle as orc
from paper_2506_17974_b200 import binding as B
from paper_2506_17974_b200 import workloads as wl
import parity as par

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

RAGGED = ((96, 200), (130, 36), (64, 27), (20, 1), (300, 512), (33, 17), (700, 64))


def _check_layer(comp, l, st):
    n, m = comp.layers[l]
    W = comp.W
    r = min(comp.rank, n, m)
    assert st["rank_eff"] == r
    assert st["status"] == comp.status()[l]
    sc = par.host(comp.get_state(B.STATE_SCALES, l))
    if comp.column_scales:
        s_p, s_q = sc[0], sc[1]
        assert np.float32(st["scale_p"]) == np.float32(sc[0].max()) and np.float32(st["scale_q"]) == np.float32(sc[1].max())
    else:
        s_p, s_q = np.float32(sc[0]), np.float32(sc[1])
        assert np.float32(st["scale_p"]) == s_p and np.float32(st["scale_q"]) == s_q
    P = [par.host(comp.get_state(B.STATE_P, l, w)) for w in range(W)]
    Qw = [par.host(comp.get_state(B.STATE_Q_W, l, w)) for w in range(W)]
    raw = [par.host(comp.get_state(B.STATE_P_RAW, l, w)) for w in range(W)]
    if comp.bits_p == 32:
        assert st["codes_p"] == 0 and st["near_p"] == 0
    else:
        assert st["codes_p"] == W * n * r
        assert st["near_p"] == sum(orc.near_threshold_count(P[w], s_p, comp.bits_p, comp.alpha) for w in range(W)), l
    if comp.bits_q == 32:
        assert st["codes_q"] == 0 and st["near_q"] == 0
    else:
        assert st["codes_q"] == W * m * r
        assert st["near_q"] == sum(orc.near_threshold_count(Qw[w], s_q, comp.bits_q, comp.alpha) for w in range(W)), l
    want = min(orc.pivot_ratio(raw[w]) for w in range(W))
    assert st["pivot_ratio"] == pytest.approx(want, rel=1e-4, abs=1e-7), (l, st["pivot_ratio"], want)
    return st["near_p"] + st["near_q"]


@pytest.mark.parametrize("rank,bits,W,kw", [
    (3, 4, 3, {}), (8, 8, 2, {}), (1, 2, 1, {}), (16, 8, 2, {}), (40, 5, 2, {}),
    (4, 3, 2, dict(column_scales=True)), (4, 6, 2, dict(one_launch=True)), (5, 32, 2, {}),
    (6, 4, 2, dict(bits_q=8)), (8, 4, 2, dict(register_path=True)),
])
def test_step_stats_match_the_oracle_on_ragged_layers(rank, bits, W, kw):
    w = wl.Workload("stats", RAGGED, rank=rank, bits=bits, workers=W, steps=2, dist="student_t3", scale="fan_in",
                    seed=70 + rank)
    kw = dict(kw)
    comp = B.LQSGD(w.layers, w.rank, w.bits, kw.pop("bits_q", None), alpha=w.alpha, workers=W, seed=w.seed, **kw)
    first = comp.step_stats(0)                                   # before any round: zeros, no fault
    assert first["near_p"] == 0 and first["near_q"] == 0 and first["pivot_ratio"] == 0.0
    for t in range(2):
        g = wl.draw_gradients(w, t, device=DEV)
        comp.step(g, [torch.empty(s, device=DEV) for s in w.layers])
    torch.cuda.synchronize()
    total = 0
    for l, shape in enumerate(w.layers):
        st = comp.step_stats(l)
        if comp.is_matrix(l):
            _check_layer(comp, l, st)
        else:
            assert st["rank_eff"] == 0 and st["codes_p"] == 0 and st["near_p"] == 0 and st["pivot_ratio"] == 0.0
        total += st["payload_bytes"]
    assert total == comp.payload_nbytes
    assert comp.step_stats(1) == comp.step_stats(1)              # asking twice changes nothing


def test_step_stats_find_entries_on_thresholds_on_the_resnet_set():
    """Enough codes (7 M at 8 bits) that some factor entries do sit on a threshold: the device's count is the
    oracle's, layer by layer, and the fraction is of the order the 254 fp32 numbers around 127 thresholds give."""
    w = wl.config3(workers=4, rank=8, bits=8)
    comp = B.LQSGD(w.layers, w.rank, w.bits, None, alpha=w.alpha, workers=w.workers, seed=w.seed)
    g = wl.draw_gradients(w, 0, device=DEV)
    comp.step(g, [torch.empty(s, device=DEV) for s in w.layers])
    torch.cuda.synchronize()
    near = codes = 0
    for l in range(len(w.layers)):
        if comp.is_matrix(l):
            st = comp.step_stats(l)
            near += _check_layer(comp, l, st)
            codes += st["codes_p"] + st["codes_q"]
    assert near > 0
    assert near / codes < 1e-4
    print("entries within one fp32 step of a threshold:", near, "of", codes, f"({near / codes:.2e})")


def test_step_stats_zero_gradient_and_bad_arguments():
    layers = ((64, 48), (48, 1))
    comp = B.LQSGD(layers, 3, 4, None, workers=2)
    g = [[torch.zeros(s, device=DEV) for s in layers] for _ in range(2)]
    comp.step(g, [torch.empty(s, device=DEV) for s in layers])
    torch.cuda.synchronize()
    st = comp.step_stats(0)
    assert st["near_p"] == 0 and st["near_q"] == 0 and st["pivot_ratio"] == 0.0
    assert st["status"] & B.STATUS_DEPENDENT_COLUMN
    for bad in (-1, 2):
        with pytest.raises(B.LqsgdError) as e:
            comp.step_stats(bad)
        assert e.value.code == B.ERR_OUT_OF_RANGE
