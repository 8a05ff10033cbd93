"""Pins of the oracle's low-rank round (Algorithm 1 body, Eq. 3, Eq. 6-8, Section IV-C) against
LAPACK QR, the truncated SVD, planted low-rank recovery, error-feedback identities and the
closed-form communication cost - plus planted-mistake checks showing the pins bite."""
import numpy as np
import pytest

from oracle import lqsgd_oracle as orc
from paper_2506_17974_b200 import workloads as wl


# ------------------------------------------------------------------ orthonormalisation
def check_orthonormalize():
    rng = np.random.default_rng(0)
    for n, r in [(5, 1), (17, 3), (256, 2), (300, 7), (64, 16)]:
        A = rng.standard_normal((n, r)) * rng.uniform(0.1, 10, size=r)
        Qm, dep = orc.orthonormalize(A)
        assert not dep.any()
        assert np.max(np.abs(Qm.T @ Qm - np.eye(r))) < 1e-10
        R = Qm.T @ A
        assert np.max(np.abs(np.tril(R, -1))) < 1e-10 * np.max(np.abs(R))     # upper triangular
        assert np.all(np.diag(R) > 0)                                          # positive diagonal
        assert np.allclose(Qm @ R, A, atol=1e-12 * np.max(np.abs(A)))
        Ql, Rl = np.linalg.qr(A)                                               # LAPACK Householder
        Ql = Ql * np.sign(np.diag(Rl))[None, :]
        assert np.max(np.abs(Qm - Ql)) < 1e-10


def test_orthonormalize_against_lapack_qr():
    check_orthonormalize()


def test_orthonormalize_dependent_and_zero_columns():
    rng = np.random.default_rng(1)
    a = rng.standard_normal(40)
    A = np.stack([a, 2 * a, rng.standard_normal(40)], axis=1)
    Qm, dep = orc.orthonormalize(A)
    assert dep.tolist() == [False, True, False]
    assert np.all(Qm[:, 1] == 0)
    assert abs(Qm[:, 0] @ Qm[:, 2]) < 1e-12 and abs(Qm[:, 2] @ Qm[:, 2] - 1) < 1e-12
    Z, dep = orc.orthonormalize(np.zeros((6, 2)))
    assert dep.all() and np.all(Z == 0)


# ------------------------------------------------------------------ planted low rank (Eq. 3)
def check_planted_rank_recovery():
    rng = np.random.default_rng(2)
    for n, m, r, W in [(30, 50, 3, 1), (64, 27, 4, 1), (12, 40, 2, 3)]:
        # integer factors: the product is exactly representable in fp32, so G is exactly rank r
        A = rng.integers(-4, 5, (n, r)).astype(np.float64)
        B = rng.integers(-4, 5, (m, r)).astype(np.float64)
        G = (A @ B.T)
        G32 = np.stack([G.astype(np.float32)] * W)
        Q0 = rng.standard_normal((m, r))
        res = orc.layer_round(G32, np.zeros_like(G32, dtype=np.float64), Q0, 32, 32, 127.0)
        ref = G32[0].astype(np.float64)
        assert np.linalg.norm(res["G_hat"] - ref) <= 1e-10 * np.linalg.norm(ref)
        assert np.max(np.abs(res["E_new"])) <= 1e-10 * np.max(np.abs(ref))


def test_planted_rank_r_is_recovered_exactly_without_quantiser():
    check_planted_rank_recovery()


def check_power_iteration_converges_to_truncated_svd():
    rng = np.random.default_rng(3)
    n, m, r = 24, 18, 3
    U, _ = np.linalg.qr(rng.standard_normal((n, n)))
    V, _ = np.linalg.qr(rng.standard_normal((m, m)))
    sv = np.array([10, 7, 5, 1.0, 0.7, 0.5] + [0.1] * 12)
    G = (U[:, :18] * sv) @ V.T
    G32 = G.astype(np.float32)[None]
    Q = rng.standard_normal((m, r))
    E0 = np.zeros((1, n, m))
    for _ in range(60):                      # fixed G, no error feedback, warm-started Q
        res = orc.layer_round(G32, E0, Q, 32, 32, 127.0)
        Q = res["Q_bar"]
    G64 = G32[0].astype(np.float64)
    Uf, sf, Vf = np.linalg.svd(G64)
    best = (Uf[:, :r] * sf[:r]) @ Vf[:r]
    assert np.linalg.norm(res["G_hat"] - best) <= 1e-8 * np.linalg.norm(best)   # Eckart-Young optimum


def test_power_iteration_converges_to_best_rank_r():
    check_power_iteration_converges_to_truncated_svd()


# ------------------------------------------------------------------ error feedback (Eq. 6-8)
def check_error_feedback_telescopes():
    rng = np.random.default_rng(4)
    layers = [(20, 36), (7, 1), (9, 12)]
    W, r = 3, 2
    Q0 = {0: rng.standard_normal((36, r)), 2: rng.standard_normal((12, r))}
    o = orc.Oracle(layers, r, 4, 4, 127.0, W, Q0)
    sum_G = {0: np.zeros((W, 20, 36)), 2: np.zeros((W, 9, 12))}
    sum_hat = {0: np.zeros((20, 36)), 2: np.zeros((9, 12))}
    for t in range(6):
        grads = [[rng.standard_normal(s).astype(np.float32) * 0.1 for s in layers] for _ in range(W)]
        E_prev = {li: o.E[li].copy() for li in o.E}
        Q_prev = {li: o.Q[li].copy() for li in o.Q}
        out = o.step(grads)
        for li in (0, 2):
            Gl = np.stack([grads[w][li] for w in range(W)]).astype(np.float64)
            # E_t + G_hat_t = G_t + E_{t-1}, element-wise, per worker
            assert np.max(np.abs(out[li]["E_new"] + out[li]["G_hat"][None] - Gl - E_prev[li])) < 1e-14
            # the products are taken on M = G + E with the warm-started Q
            assert np.allclose(out[li]["P_raw"][1], (Gl[1] + E_prev[li][1]) @ Q_prev[li], atol=1e-13)
            assert np.allclose(out[li]["Qw"][2], (Gl[2] + E_prev[li][2]).T @ out[li]["P_bar"], atol=1e-13)
            assert np.array_equal(o.Q[li], out[li]["Q_bar"])            # warm start for t+1
            sum_G[li] += Gl
            sum_hat[li] += out[li]["G_hat"]
        v = np.stack([grads[w][1] for w in range(W)]).reshape(W, -1).astype(np.float64)
        assert np.allclose(out[1]["mean"], v.sum(0) / W, atol=1e-15)    # Eq. 1 for the 1-D tensor
    for li in (0, 2):                        # sum_t G_hat_t + E_T = sum_t G_t  (E_0 = 0)
        assert np.max(np.abs(sum_hat[li][None] + o.E[li] - sum_G[li])) < 1e-12


def test_error_feedback_identities_and_state_machine():
    check_error_feedback_telescopes()


def check_round_uses_dequantised_average():
    """P_bar must be the dequantised worker mean (on the level grid for W=1), and Q must be
    computed from it, not from the orthonormal P."""
    rng = np.random.default_rng(6)
    n, m, r = 16, 24, 2
    G = rng.standard_normal((1, n, m)).astype(np.float32)
    res = orc.layer_round(G, np.zeros((1, n, m)), rng.standard_normal((m, r)), 4, 4, 127.0)
    s = float(res["xp"]["scale"])
    lv = orc.level_values(4, 127.0) * s
    d = np.min(np.abs(np.abs(res["P_bar"])[..., None] - lv), axis=-1)
    assert np.max(d) < 1e-12
    assert np.allclose(res["Qw"][0], G[0].astype(np.float64).T @ res["P_bar"], atol=1e-12)
    assert np.allclose(res["G_hat"], res["P_bar"] @ res["Q_bar"].T, atol=1e-13)
    assert s == np.max(np.abs(res["P"].astype(np.float32)))


def test_round_structure():
    check_round_uses_dequantised_average()


# ------------------------------------------------------------------ planted mistakes
MISTAKES = {
    "drop_error_feedback": ("error_feedback", lambda G, E: np.asarray(G, dtype=np.float64)),
    "error_sign": ("error_update", lambda M, Gh: Gh - np.asarray(M, dtype=np.float64)),
    "p_uses_abs_q": ("power_step_p", lambda M, Q: np.asarray(M, np.float64) @ np.abs(Q)),
    "q_without_transpose_effect": ("power_step_q", lambda M, P: np.asarray(M, np.float64).T @ np.abs(P)),
    "recon_scaled": ("reconstruct", lambda P, Q: 0.5 * np.asarray(P) @ np.asarray(Q).T),
    "no_orthonormalise": ("orthonormalize", lambda P: (np.array(P, dtype=np.float64),
                                                        np.zeros(np.shape(P)[1], dtype=bool))),
}


@pytest.mark.parametrize("name", sorted(MISTAKES))
def test_planted_mistake_is_caught(name, monkeypatch):
    attr, bad = MISTAKES[name]
    monkeypatch.setattr(orc, attr, bad)
    failed = 0
    for chk in (check_orthonormalize, check_planted_rank_recovery,
                check_power_iteration_converges_to_truncated_svd,
                check_error_feedback_telescopes, check_round_uses_dequantised_average):
        try:
            chk()
        except AssertionError:
            failed += 1
    assert failed >= 1, f"no pin noticed the mistake {name}"


# ------------------------------------------------------------------ communication cost (Section IV-C)
def test_payload_closed_forms(golden_dir):
    rows = [l.split() for l in open(f"{golden_dir}/payload_bytes.txt") if l.strip() and not l.startswith("#")]
    cfgs = {"config1": wl.config1(), "config2": wl.config2(), "config3": wl.config3()}
    for a, b in wl.CONFIG4_SIZES:
        cfgs[f"config4_{a}x{b}"] = wl.config4(a, b)
    cfgs["config5_r1_b2"] = wl.config5(1, 2)
    cfgs["config5_r16_b8"] = wl.config5(16, 8)
    seen = 0
    for name, want in rows:
        c = cfgs[name]
        assert orc.payload_bytes(c.layers, c.rank, c.bits, c.bits) == int(want), name
        seen += 1
    assert seen == len(cfgs)
    # r(n+m)b bits and the 32/b ratio against fp32 factors
    assert orc.factor_bits(256, 576, 2, 4) == 2 * (256 + 576) * 4
    for b in (2, 4, 8):
        assert 32 * 2 * (256 + 576) / orc.factor_bits(256, 576, 2, b) == 32 / b
    assert orc.factor_bits(10, 512, 16, 4) == 10 * (10 + 512) * 4          # r_eff = min(r, n, m)


def _payload_layout_case(golden_dir):
    want = {}
    for line in open(f"{golden_dir}/payload_layout.txt"):
        if line.strip() and not line.startswith("#"):
            name, *hexes = line.split()
            want[name] = np.frombuffer(bytes.fromhex("".join(hexes)), dtype=np.uint8)
    layers = ((2, 3), (3, 2), (2, 1))
    scales = [(np.float32(1.0), np.float32(2.0)), (np.float32(0.5), np.float32(4.0))]
    codes_p = [np.array([[5], [3]], np.uint8), np.array([[7], [0], [6]], np.uint8)]
    codes_q = [np.array([[1], [2], [4]], np.uint8), np.array([[6], [1]], np.uint8)]
    return want, layers, scales, codes_p, codes_q


def check_payload_layout(golden_dir):
    want, layers, scales, codes_p, codes_q = _payload_layout_case(golden_dir)
    got = orc.assemble_payload(layers, 1, 3, 3, scales, codes_p, codes_q, [np.array([1.5, -2.0], np.float32)])
    assert got.dtype == np.uint8 and got.tobytes() == want["default"].tobytes(), got.tobytes().hex()
    assert got.size == orc.payload_bytes(layers, 1, 3, 3) == 30
    got = orc.assemble_payload(layers, 1, 3, 3, scales, codes_p, codes_q, [np.array([4, 7], np.uint8)],
                               vector_scales=[np.float32(3.0)])
    assert got.tobytes() == want["quantized_vectors"].tobytes(), got.tobytes().hex()
    assert got.size == orc.payload_bytes(layers, 1, 3, 3, quantize_vectors=True) == 27


def test_payload_layout_byte_for_byte(golden_dir):
    """assemble_payload against a byte string written out by hand from the documented order
    (scales, 1-D tensors, P streams, Q streams; Section IV-C bit streams), both layouts."""
    check_payload_layout(golden_dir)


@pytest.mark.parametrize("mistake", ["p_q_swapped", "scales_last", "per_layer_interleaved", "big_endian_codes"])
def test_payload_layout_pin_catches_a_wrong_order(mistake, golden_dir, monkeypatch):
    """Plausible layout mistakes planted in the oracle must fail the byte-for-byte pin."""
    good = orc.assemble_payload
    pack = orc.pack_codes

    def bad(layers, rank, bits_p, bits_q, scales, codes_p, codes_q, vectors, vector_scales=None):
        if mistake == "p_q_swapped":
            return good(layers, rank, bits_q, bits_p, scales, codes_q, codes_p, vectors, vector_scales)
        if mistake == "scales_last":
            out = good(layers, rank, bits_p, bits_q, scales, codes_p, codes_q, vectors, vector_scales)
            k = 8 * len(scales)
            return np.concatenate([out[k:], out[:k]])
        if mistake == "per_layer_interleaved":
            head = good(layers, rank, bits_p, bits_q, scales, [], [], vectors, vector_scales)
            return np.concatenate([head] + [x for cp, cq in zip(codes_p, codes_q)
                                            for x in (pack(cp, bits_p), pack(cq, bits_q))])
        return good(layers, rank, bits_p, bits_q, scales, codes_p, codes_q, vectors, vector_scales)

    def msb_first(codes, bits):                       # element 0 in the HIGHEST bits of the first byte
        flat = np.asarray(codes, np.uint8).reshape(-1)
        out = np.zeros((flat.size * bits + 7) // 8, np.uint8)
        for i, c in enumerate(flat):
            for j in range(bits):
                pos = i * bits + j
                out[pos >> 3] |= ((int(c) >> (bits - 1 - j)) & 1) << (7 - (pos & 7))
        return out

    if mistake == "big_endian_codes":
        monkeypatch.setattr(orc, "pack_codes", msb_first)
    monkeypatch.setattr(orc, "assemble_payload", bad)
    with pytest.raises(AssertionError):
        check_payload_layout(golden_dir)


def test_resnet18_shape_list_reproduces_published_epoch_sizes():
    """Tables I-III: MB sent per epoch by uncompressed SGD and by rank-1 PowerSGD.  With 5
    workers and batch 128, CIFAR has 50000/640 = 78 iterations per epoch and MNIST 60000/640 = 93."""
    MiB = 2.0 ** 20

    def sizes(layers, iters):
        full = 4 * sum(n * m for n, m in layers) * iters / MiB
        r1 = 4 * (sum(n + m for n, m in layers if wl.is_matrix((n, m)))
                  + wl.vector_elements(layers)) * iters / MiB
        return full, r1

    c10 = wl.resnet18_layers(10)
    assert sum(n * m for n, m in c10) == 11_173_962
    assert len([s for s in c10 if wl.is_matrix(s)]) == 21 and wl.vector_elements(c10) == 9610
    full, r1 = sizes(c10, 78)
    assert round(full) == 3325 and round(r1) == 14                       # Table I
    full, r1 = sizes(wl.resnet18_layers(100), 78)
    assert round(full) == 3339 and round(r1) == 14                       # Table II
    full, r1 = sizes(wl.resnet18_layers(10, in_channels=1), 93)
    assert round(full) == 3964 and round(r1) == 16                       # Table III


def test_quantised_vectors_variant():
    """1-D tensors through the factor exchange: payload closed form, one-worker round trip of the
    levels, and agreement with exchange_factor on the reshaped tensor."""
    layers = ((6, 5), (1, 9), (7, 1))
    assert orc.payload_bytes(layers, 2, 4, 4, quantize_vectors=True) == (2 * 6 * 4 + 7) // 8 + (2 * 5 * 4 + 7) // 8 + 8 \
        + (4 + (9 * 4 + 7) // 8) + (4 + (7 * 4 + 7) // 8)
    assert orc.payload_bytes(layers, 2, 32, 32, quantize_vectors=True) == orc.payload_bytes(layers, 2, 32, 32)
    rng = np.random.default_rng(3)
    Q0 = {0: rng.standard_normal((5, 2))}
    o = orc.Oracle(layers, 2, 4, 4, 127.0, 1, Q0, quantize_vectors=True)
    lev = orc.level_values(4, 127.0)
    v = np.float32(2.0) * np.array([lev[7], -lev[3], lev[0], lev[5], -lev[7], lev[1], lev[2], -lev[6], lev[4]], np.float32)
    g = [[rng.standard_normal((6, 5)).astype(np.float32), v.reshape(1, 9), rng.standard_normal((7, 1)).astype(np.float32)]]
    out = o.step(g)
    assert out[1]["scale"] == np.float32(2.0)
    assert np.allclose(out[1]["mean"], v.astype(np.float64), rtol=1e-6, atol=0)       # every level round-trips
    assert list(out[1]["codes"][0] & 7) == [7, 3, 0, 5, 7, 1, 2, 6, 4]
    x = orc.exchange_factor([g[0][2].reshape(-1, 1)], 4, 127.0)
    assert np.array_equal(out[2]["mean"], x["mean"].reshape(-1))
    pay = orc.assemble_payload(layers, 2, 4, 4, [(out[0]["xp"]["scale"], out[0]["xq"]["scale"])],
                               [out[0]["xp"]["codes"][0]], [out[0]["xq"]["codes"][0]],
                               [out[1]["codes"][0], out[2]["codes"][0]], vector_scales=[out[1]["scale"], out[2]["scale"]])
    assert pay.size == orc.payload_bytes(layers, 2, 4, 4, quantize_vectors=True)
    assert np.array_equal(pay[8:16].view("<f4"), np.array([out[1]["scale"], out[2]["scale"]], dtype="<f4"))


def test_several_power_iterations_option():
    """power_iters = T repeats the power step on the same M: with the quantiser bypassed and one
    worker it is T steps of subspace iteration written out by hand (library QR), it leaves a
    rank-r matrix fixed, and more iterations bring P_bar Q_bar^T closer to the truncated SVD."""
    rng = np.random.default_rng(8)
    n, m, r = 30, 22, 3
    G = rng.standard_normal((1, n, m)).astype(np.float32)
    E = np.zeros((1, n, m))
    Q0 = rng.standard_normal((m, r))
    res = orc.layer_round(G, E, Q0, 32, 32, 127.0, power_iters=3)
    M, Q = G[0].astype(np.float64), Q0
    for _ in range(3):
        P, R = np.linalg.qr(M @ Q)
        P = P * np.sign(np.diag(R))
        Q = M.T @ P
    assert np.allclose(res["P_bar"], P, atol=1e-10) and np.allclose(res["Q_bar"], Q, atol=1e-10)
    assert np.allclose(res["G_hat"], P @ Q.T, atol=1e-10)
    U, sv, Vt = np.linalg.svd(M)
    best = (U[:, :r] * sv[:r]) @ Vt[:r]
    err = [np.linalg.norm(orc.layer_round(G, E, Q0, 32, 32, 127.0, power_iters=T)["G_hat"] - best) for T in (1, 4, 16)]
    assert err[0] > err[1] > err[2]
    A, Bm = rng.integers(-3, 4, (n, r)).astype(np.float32), rng.integers(-3, 4, (m, r)).astype(np.float32)
    low = (A @ Bm.T)[None]
    for T in (1, 2, 5):
        assert np.allclose(orc.layer_round(low, E, Q0, 32, 32, 127.0, power_iters=T)["G_hat"], low[0], atol=1e-9)
    # one iteration is Algorithm 1 as it stands
    one = orc.layer_round(G, E, Q0, 4, 4, 127.0)
    assert np.array_equal(one["G_hat"], orc.layer_round(G, E, Q0, 4, 4, 127.0, power_iters=1)["G_hat"])


def test_pivot_ratio_is_the_diagonal_of_the_qr_factor():
    """pivot_ratio against LAPACK: min |R_jj| / max |R_jj| of numpy's QR; a hand case; a dependent column."""
    A = np.zeros((4, 2))
    A[0, 0], A[1, 1], A[0, 1] = 3.0, 1.0, 5.0          # R = [[3, 5], [0, 1]]
    assert orc.pivot_ratio(A) == pytest.approx(1.0 / 3.0, rel=1e-14)
    rng = np.random.default_rng(11)
    for n, r in [(50, 1), (40, 5), (300, 16)]:
        X = rng.standard_normal((n, r)) * np.logspace(0, -3, r)
        d = np.abs(np.diag(np.linalg.qr(X)[1]))
        assert orc.pivot_ratio(X) == pytest.approx(d.min() / d.max(), rel=1e-10)
    X = rng.standard_normal((30, 3))
    X[:, 2] = X[:, 0] - 2 * X[:, 1]
    assert orc.pivot_ratio(X) == 0.0
    assert orc.pivot_ratio(np.zeros((6, 2))) == 0.0
