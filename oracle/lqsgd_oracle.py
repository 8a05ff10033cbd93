"""CPU oracle for one LQ-SGD compression round.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 restatement of Algorithm 1 (iteration body, error feedback to
error update) and of the quantiser of Eq. 4 / Eq. 5 of "Trustworthy Efficient
Communication for Distributed Learning using LQ-SGD Algorithm".  It exists to
check the CUDA library; the library never calls it, and it imports nothing
from the library (numpy only).  Only tests, the smoke check and the CPU-baseline
leg of the benchmark may execute it.

Notation is the paper's Section IV: G in R^{n x m}, P in R^{n x r},
Q in R^{m x r}, E the error buffer, M = G' = G + E, W workers.

Every function states the passage it follows.  Where the paper is silent the
reading taken is stated next to the code:

* bits b = 1 sign bit + (b-1) magnitude bits, L = 2^(b-1) magnitude levels,
  placed uniformly in the companded domain with both end points, |q|_k = k/(L-1);
* nearest level in the companded domain, ties (exact half) away from zero;
* one scale s per factor and layer, s = max over workers of max |x|, and the
  division x/s is an fp32 division (the precision the library stores s and x
  in), so that the integer decision is taken on the same number on both sides;
* the worker average is the mean of the signed level indices (Alg. 1 applies
  All-Reduce to the quantised factor, then dequantises once);
* Orthonormalize = the thin-QR Q factor with positive-diagonal R, computed by
  modified Gram-Schmidt; a column whose residual norm^2 is <= 1e-10 of its
  original norm^2 (a relative residual of 1e-5: the factor is fp32 data, so
  anything smaller is rounding noise of the product, not a direction), or that
  is exactly zero, becomes a zero column.

Pins (tests/test_oracle_*.py): hand-worked level/threshold tables, brute-force
nearest-level matching, closed-form inverse pair, LAPACK QR, truncated SVD,
planted-rank recovery, error-feedback telescoping, payload closed forms, and the payload
layout against a byte string written out by hand (tests/golden/payload_layout.txt).
The value of alpha and the readings above have no printed worked example in
the paper: against the authors' own code they are "parity unpinned".
"""
from __future__ import annotations

import numpy as np

RANK_EPS = 1e-10     # relative residual norm^2 below which a column counts as dependent


# ----------------------------------------------------------------------------
# Eq. 4 / Eq. 5: the compander pair
# ----------------------------------------------------------------------------
def compand(x, alpha):
    """Eq. 4: q(x) = sign(x) * log(1 + alpha|x|) / log(1 + alpha)."""
    x = np.asarray(x, dtype=np.float64)
    return np.sign(x) * np.log1p(alpha * np.abs(x)) / np.log1p(alpha)


def expand(q, alpha):
    """Eq. 5: x = sign(q) * ((1 + alpha)^|q| - 1) / alpha."""
    q = np.asarray(q, dtype=np.float64)
    return np.sign(q) * np.expm1(np.abs(q) * np.log1p(alpha)) / alpha


def magnitude_levels(bits):
    """Number of magnitude levels L for a b-bit code with one sign bit."""
    if not 2 <= bits <= 8:
        raise ValueError("bits must be in 2..8")
    return 1 << (bits - 1)


def level_values(bits, alpha):
    """x-domain magnitudes of the L levels: expand(k / (L-1)), k = 0..L-1."""
    L = magnitude_levels(bits)
    return expand(np.arange(L, dtype=np.float64) / (L - 1), alpha)


# ----------------------------------------------------------------------------
# LogQuantize / LogDequantize (the quantise and dequantise steps of Alg. 1; Section IV-A)
# ----------------------------------------------------------------------------
def factor_scale(factors, per_column=False):
    """s = max over workers and entries of |x| (fp32 values, exact).  per_column (a variant):
    one scale per column of the factor, s_j = max over workers and rows of |x[:, j]|."""
    if per_column:
        cols = np.asarray(factors[0]).shape[1]
        s = np.zeros(cols, dtype=np.float32)
        for f in factors:
            f32 = np.asarray(f, dtype=np.float32)
            if f32.size:
                s = np.maximum(s, np.max(np.abs(f32), axis=0))
        return s.astype(np.float32)
    s = np.float32(0.0)
    for f in factors:
        f32 = np.asarray(f, dtype=np.float32)
        if f32.size:
            s = max(s, np.float32(np.max(np.abs(f32))))
    return np.float32(s)


def log_quantize(x, s, bits, alpha, return_margin=False):
    """b-bit code of every entry of x: (sign bit << (b-1)) | k.

    k = nearest level index of compand(|x|/s) on the grid k/(L-1), half away
    from zero.  x and s are taken as fp32 and |x|/s is an fp32 division.
    With return_margin also returns, in level units, the distance of the
    companded magnitude from the nearest decision threshold.
    """
    L = magnitude_levels(bits)
    x32 = np.asarray(x, dtype=np.float32)
    s32 = np.asarray(s, dtype=np.float32)                   # a scalar, or one scale per column
    neg = x32 < 0
    if s32.ndim == 0 and s32 == 0:
        v = np.zeros(x32.shape, dtype=np.float64)
    else:
        with np.errstate(divide="ignore", invalid="ignore"):
            t = (np.abs(x32) / s32).astype(np.float32)      # fp32 division
        t = np.where(np.broadcast_to(s32 == 0, x32.shape), np.float32(0), t)   # a zero scale: all codes 0
        v = (L - 1) * compand(t.astype(np.float64), alpha)  # in [0, L-1]
    k = np.floor(v + 0.5)
    k = np.clip(k, 0, L - 1).astype(np.uint8)
    codes = (neg.astype(np.uint8) << (bits - 1)) | k
    if return_margin:
        return codes, np.abs(v - (np.floor(v) + 0.5))
    return codes


def near_threshold_count(x, s, bits, alpha):
    """How many entries of x have |x|/s (an fp32 number) within one fp32 step of a decision
    threshold of Eq. 4's nearest-level rule: the two fp32 neighbours of |x|/s get different
    level indices.  These are the codes a last-place difference in |x|/s can change."""
    L = magnitude_levels(bits)
    x32 = np.asarray(x, dtype=np.float32)
    s32 = np.asarray(s, dtype=np.float32)
    with np.errstate(divide="ignore", invalid="ignore"):
        t = (np.abs(x32) / s32).astype(np.float32)
    ok = np.broadcast_to((s32 > 0) & np.isfinite(s32), x32.shape) & np.isfinite(t)
    t = np.where(ok, t, np.float32(0))
    below = np.where(t > 0, np.nextafter(t, np.float32(-np.inf)), np.float32(0)).astype(np.float32)
    above = np.nextafter(t, np.float32(np.inf)).astype(np.float32)

    def level(u):
        u = np.minimum(u.astype(np.float64), np.finfo(np.float32).max)
        return np.clip(np.floor((L - 1) * compand(u, alpha) + 0.5), 0, L - 1)

    return int(np.count_nonzero(ok & (level(below) != level(above))))


def signed_levels(codes, bits):
    """Signed level index (-1)^sign * k of each code, as int64."""
    codes = np.asarray(codes).astype(np.int64)
    k = codes & ((1 << (bits - 1)) - 1)
    neg = (codes >> (bits - 1)) & 1
    return np.where(neg == 1, -k, k)


def average_dequantize(codes_per_worker, s, bits, alpha):
    """All-Reduce (mean, Eq. 1) of the signed quantised values, then Eq. 5 once.

    q_bar = sum_w (+-k_w) / (W (L-1));  result = s * expand(q_bar).
    """
    L = magnitude_levels(bits)
    W = len(codes_per_worker)
    S = np.zeros(np.asarray(codes_per_worker[0]).shape, dtype=np.int64)
    for c in codes_per_worker:
        S += signed_levels(c, bits)
    q_bar = S.astype(np.float64) / (W * (L - 1))
    return np.asarray(s, dtype=np.float32).astype(np.float64) * expand(q_bar, alpha)


def dequantize_average(codes_per_worker, s, bits, alpha):
    """The other reading of the exchange (a parameter server that decodes what it receives,
    Section V set-up): Eq. 5 applied to every worker's quantised value, then the mean of Eq. 1
    over the dequantised values.  Not Algorithm 1's order (which averages first); offered as
    a variant.  result = (1/W) sum_w s * expand(+-k_w / (L-1))."""
    L = magnitude_levels(bits)
    W = len(codes_per_worker)
    total = np.zeros(np.asarray(codes_per_worker[0]).shape, dtype=np.float64)
    for c in codes_per_worker:                      # worker order
        q = signed_levels(c, bits).astype(np.float64) / (L - 1)
        total += np.asarray(s, dtype=np.float32).astype(np.float64) * expand(q, alpha)
    return total / W


def pack_codes(codes, bits):
    """Little-endian bit stream: element i (row-major) occupies bits [i*b, (i+1)*b)."""
    flat = np.asarray(codes, dtype=np.uint8).reshape(-1)
    nbytes = (flat.size * bits + 7) // 8
    out = np.zeros(nbytes, dtype=np.uint8)
    for j in range(bits):                       # bit j of every code
        pos = np.arange(flat.size, dtype=np.int64) * bits + j
        bit = (flat >> j) & 1
        np.bitwise_or.at(out, pos >> 3, (bit << (pos & 7)).astype(np.uint8))
    return out


def unpack_codes(stream, count, bits):
    """Inverse of pack_codes for `count` elements."""
    stream = np.asarray(stream, dtype=np.uint8)
    codes = np.zeros(count, dtype=np.uint8)
    for j in range(bits):
        pos = np.arange(count, dtype=np.int64) * bits + j
        bit = (stream[pos >> 3] >> (pos & 7)) & 1
        codes |= (bit << j).astype(np.uint8)
    return codes


# ----------------------------------------------------------------------------
# Orthonormalize (the orthonormalisation step of Alg. 1)
# ----------------------------------------------------------------------------
def orthonormalize(P):
    """Modified Gram-Schmidt, columns left to right.  Returns (P_orth, dependent_mask)."""
    A = np.array(P, dtype=np.float64, copy=True)
    r = A.shape[1]
    dependent = np.zeros(r, dtype=bool)
    for j in range(r):
        norm0 = float(A[:, j] @ A[:, j])
        for i in range(j):
            A[:, j] -= (A[:, i] @ A[:, j]) * A[:, i]
        norm1 = float(A[:, j] @ A[:, j])
        if norm0 == 0.0 or norm1 <= RANK_EPS * norm0:
            A[:, j] = 0.0
            dependent[j] = True
        else:
            A[:, j] /= np.sqrt(norm1)
    return A, dependent


def pivot_ratio(P):
    """Conditioning of the factor given to Orthonormalize: with P = P_orth R (R upper triangular,
    positive diagonal; R_jj is the norm left of column j after the earlier columns are taken
    out), min_j R_jj / max_j R_jj; 0 when a column is dropped as dependent."""
    A = np.array(P, dtype=np.float64, copy=True)
    r = A.shape[1]
    diag = np.zeros(r)
    for j in range(r):
        norm0 = float(A[:, j] @ A[:, j])
        for i in range(j):
            A[:, j] -= (A[:, i] @ A[:, j]) * A[:, i]
        norm1 = float(A[:, j] @ A[:, j])
        if norm0 == 0.0 or norm1 <= RANK_EPS * norm0:
            A[:, j] = 0.0
        else:
            diag[j] = np.sqrt(norm1)
            A[:, j] /= diag[j]
    return float(diag.min() / diag.max()) if diag.max() > 0 else 0.0


# ----------------------------------------------------------------------------
# One factor exchange: scale, quantise, All-Reduce, dequantise
# ----------------------------------------------------------------------------
def exchange_factor(factors, bits, alpha, forced_codes=None, average="codes", column_scales=False):
    """Quantise every worker's factor, average, dequantise (Alg. 1, the three steps
    after each product).  bits == 32 bypasses the quantiser (plain PowerSGD mean).

    forced_codes: optional list (per worker) of int16 arrays; entries >= 0 replace
    the code computed here (used by parity tests for near-threshold elements).
    average: "codes" (Algorithm 1: mean of the quantised values, then Eq. 5) or "values"
    (Eq. 5 per worker, then the mean).
    Returns dict(scale, codes[list], margin[list], mean) with mean in fp64.
    """
    assert average in ("codes", "values")
    W = len(factors)
    if bits == 32:
        mean = sum(np.asarray(f, dtype=np.float64) for f in factors) / W
        return dict(scale=np.float32(0), codes=None, margin=None, mean=mean)
    s = factor_scale(factors, per_column=column_scales)
    codes, margins = [], []
    for w, f in enumerate(factors):
        c, mg = log_quantize(f, s, bits, alpha, return_margin=True)
        if forced_codes is not None and forced_codes[w] is not None:
            fc = np.asarray(forced_codes[w]).reshape(c.shape)
            c = np.where(fc >= 0, fc, c).astype(np.uint8)
        codes.append(c)
        margins.append(mg)
    mean = (average_dequantize if average == "codes" else dequantize_average)(codes, s, bits, alpha)
    return dict(scale=s, codes=codes, margin=margins, mean=mean)


# ----------------------------------------------------------------------------
# The stages of one round for one layer (Algorithm 1, loop body)
# ----------------------------------------------------------------------------
def error_feedback(G, E):
    """M = G' = G + E (Eq. 8)."""
    return np.asarray(G, dtype=np.float64) + np.asarray(E, dtype=np.float64)


def power_step_p(M, Q):
    """P = M Q."""
    return np.asarray(M, dtype=np.float64) @ np.asarray(Q, dtype=np.float64)


def power_step_q(M, P_bar):
    """Q = M^T P_bar, with the dequantised, averaged P."""
    return np.asarray(M, dtype=np.float64).T @ np.asarray(P_bar, dtype=np.float64)


def reconstruct(P_bar, Q_bar):
    """G_hat = P Q^T (Eq. 6)."""
    return np.asarray(P_bar, dtype=np.float64) @ np.asarray(Q_bar, dtype=np.float64).T


def error_update(M, G_hat):
    """E = G' - G_hat (Eq. 7)."""
    return np.asarray(M, dtype=np.float64) - G_hat


def effective_rank(rank, n, m):
    return min(rank, n, m)


def layer_round(G, E, Q, bits_p, bits_q, alpha, forced_p=None, forced_q=None, average="codes", power_iters=1,
                column_scales=False):
    """One iteration of Algorithm 1 for one n x m layer and W workers.

    power_iters > 1 (an option, Algorithm 1 does one): the power step with its two exchanges is
    repeated on the same M, each time from the Q_bar just obtained; the last P_bar, Q_bar form
    G_hat.  forced_* apply to the last repetition; the returned intermediates are the last ones.

    G, E: arrays [W, n, m];  Q: [m, r] shared by all workers (warm start).
    Returns a dict with every intermediate:
      M [W,n,m], P_raw [W,n,r], P [W,n,r] (orthonormal), dependent [W,r],
      xp (exchange_factor result for P), P_bar [n,r], Qw [W,m,r], xq, Q_bar [m,r],
      G_hat [n,m], E_new [W,n,m].
    """
    G = np.asarray(G)
    W = G.shape[0]
    M = [error_feedback(G[w], E[w]) for w in range(W)]
    for it in range(power_iters):
        last = it == power_iters - 1
        P_raw = [power_step_p(M[w], Q) for w in range(W)]
        orth = [orthonormalize(P_raw[w]) for w in range(W)]
        P = [o[0] for o in orth]
        xp = exchange_factor(P, bits_p, alpha, forced_p if last else None, average, column_scales)
        P_bar = xp["mean"]
        Qw = [power_step_q(M[w], P_bar) for w in range(W)]
        xq = exchange_factor(Qw, bits_q, alpha, forced_q if last else None, average, column_scales)
        Q_bar = xq["mean"]
        Q = Q_bar
    G_hat = reconstruct(P_bar, Q_bar)
    E_new = [error_update(M[w], G_hat) for w in range(W)]
    return dict(M=np.stack(M), P_raw=np.stack(P_raw), P=np.stack(P),
                dependent=np.stack([o[1] for o in orth]), xp=xp, P_bar=P_bar,
                Qw=np.stack(Qw), xq=xq, Q_bar=Q_bar, G_hat=G_hat, E_new=np.stack(E_new))


def vector_mean(V):
    """Eq. 1 for a tensor that bypasses compression: mean over workers, V is [W, len]."""
    return np.mean(np.asarray(V, dtype=np.float64), axis=0)


# ----------------------------------------------------------------------------
# Communication cost (Section IV-C) and the payload the library documents
# ----------------------------------------------------------------------------
def factor_bits(n, m, rank, bits):
    """r (n + m) b bits per layer and iteration."""
    r = effective_rank(rank, n, m)
    return r * (n + m) * bits


def payload_bytes(layers, rank, bits_p, bits_q, quantize_vectors=False, column_scales=False):
    """Bytes one worker sends per round: for each matrix the two code streams, each
    padded to a whole byte, plus the two fp32 scales; fp32 for every 1-D tensor, or, with
    quantize_vectors (the variant that log-quantises them too, b_p bits), one fp32 scale and
    a code stream padded to a whole byte."""
    total = 0
    for n, m in layers:
        if n > 1 and m > 1:
            r = effective_rank(rank, n, m)
            total += (r * n * bits_p + 7) // 8 + (r * m * bits_q + 7) // 8 + (8 * r if column_scales else 8)
        elif quantize_vectors and bits_p != 32:
            total += 4 + (n * m * bits_p + 7) // 8
        else:
            total += 4 * n * m
    return total


def assemble_payload(layers, rank, bits_p, bits_q, scales, codes_p, codes_q, vectors, vector_scales=None):
    """One worker's payload in the library's documented order:
    [s_P, s_Q of every matrix][every 1-D tensor, fp32][P codes of every matrix][Q codes ...].
    scales: list of (s_P, s_Q); codes_*: per matrix uint8 code arrays; vectors: per 1-D tensor.
    With vector_scales (the variant that quantises the 1-D tensors): `vectors` holds their uint8
    codes, and the order is [matrix scales][one scale per 1-D tensor][their code streams][P][Q]."""
    # a matrix's scales: s_P then s_Q, each one value or (column-scale variant) r values
    parts = [np.concatenate([np.atleast_1d(np.asarray(v, dtype="<f4")) for pair in scales for v in pair]).view(np.uint8)
             if scales else np.zeros(0, np.uint8)]
    if vector_scales is not None:
        parts += [np.asarray(list(vector_scales), dtype="<f4").view(np.uint8)]
        parts += [pack_codes(c, bits_p) for c in vectors]
    else:
        parts += [np.asarray(v, dtype="<f4").reshape(-1).view(np.uint8) for v in vectors]
    parts += [pack_codes(c, bits_p) for c in codes_p]
    parts += [pack_codes(c, bits_q) for c in codes_q]
    return np.concatenate(parts) if parts else np.zeros(0, np.uint8)


# ----------------------------------------------------------------------------
# Multi-layer, multi-step driver with the persistent state (E per worker, shared Q)
# ----------------------------------------------------------------------------
class Oracle:
    """State machine of Algorithm 1 over a list of layers: E_0 = 0, Q_0 supplied by the
    caller (drawn N(0,1) outside), Q_t = dequantised averaged Q of step t-1."""

    def __init__(self, layers, rank, bits_p, bits_q, alpha, workers, Q0, average="codes", quantize_vectors=False,
                 power_iters=1, column_scales=False):
        self.layers = [tuple(s) for s in layers]
        self.column_scales = bool(column_scales)
        self.power_iters = int(power_iters)
        self.average = average
        self.quantize_vectors = bool(quantize_vectors) and bits_p != 32
        self.rank, self.bits_p, self.bits_q = rank, bits_p, bits_q
        self.alpha, self.W = float(alpha), workers
        self.E, self.Q = {}, {}
        for li, (n, m) in enumerate(self.layers):
            if n > 1 and m > 1:
                r = effective_rank(rank, n, m)
                self.E[li] = np.zeros((workers, n, m), dtype=np.float64)
                q0 = np.asarray(Q0[li], dtype=np.float64)
                assert q0.shape == (m, r), (q0.shape, (m, r))
                self.Q[li] = q0.copy()

    def step(self, grads, forced=None):
        """grads[w][layer] -> list over layers of layer_round dicts (or dict(mean=...) for 1-D)."""
        out = []
        for li, (n, m) in enumerate(self.layers):
            Gl = np.stack([np.asarray(grads[w][li], dtype=np.float32).reshape(n, m)
                           for w in range(self.W)])
            if li in self.E:
                f = (forced or {}).get(li, (None, None))
                res = layer_round(Gl, self.E[li], self.Q[li], self.bits_p, self.bits_q,
                                  self.alpha, f[0], f[1], self.average, self.power_iters, self.column_scales)
                self.E[li] = res["E_new"]
                self.Q[li] = res["Q_bar"]
            elif self.quantize_vectors:
                # variant: a 1-D tensor goes through the same exchange as a factor (one scale, b_p bits)
                x = exchange_factor([Gl[w].reshape(-1, 1) for w in range(self.W)], self.bits_p, self.alpha,
                                    average=self.average)
                res = dict(mean=x["mean"].reshape(-1), scale=x["scale"], codes=[c.reshape(-1) for c in x["codes"]])
            else:
                res = dict(mean=vector_mean(Gl.reshape(self.W, -1)))
            out.append(res)
        return out
