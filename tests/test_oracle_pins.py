"""Pins for the CPU oracle: each test checks an oracle function against something
the paper or plain mathematics fixes, computed here without going through the
oracle's own formula (brute-force loops, finite differences, closed forms,
library routines on the un-compressed object, numbers printed in the paper).
"""

import math

import numpy as np
import pytest

from conftest import read_golden
from oracle import cobs_oracle as O
from paper_2607_09052_b200 import synth


def rng(seed):
    return np.random.default_rng(seed)


def brute_log_mass(qs, kblock):
    """ln sum_t exp(q' . k_t) by python loops (Eq. bg-defs)."""
    tot = 0.0
    for t in range(kblock.shape[0]):
        dot = 0.0
        for j in range(kblock.shape[1]):
            dot += qs[j] * kblock[t, j]
        tot += math.exp(dot)
    return math.log(tot)


# --- P1: exact masses by brute force; constant-key block --------------------

def test_exact_masses_match_brute_force():
    r = rng(1)
    G, D, L, NB = 2, 4, 4, 4
    q = r.normal(size=(G, D))
    K = r.normal(size=(NB * L, D))
    got = O.exact_log_masses(q, K, L, NB)
    for g in range(G):
        for b in range(NB):
            ref = brute_log_mass(q[g] / math.sqrt(D), K[b * L:(b + 1) * L])
            assert abs(got[g, b] - ref) < 1e-12


def test_constant_key_block_estimate_is_exact_and_second_order_vanishes():
    r = rng(2)
    D, L = 8, 16
    q = r.normal(size=(3, D))
    k0 = r.normal(size=D)
    K = np.tile(k0, (L, 1))
    mean, xi, lam = O.build_summaries(K, L, rank=4)
    assert np.all(xi == 0.0) and np.all(lam == 0.0)
    e = O.log_mass_estimates(q, mean, xi, L)
    for g in range(3):
        assert abs(e[g, 0] - (math.log(L) + (q[g] / math.sqrt(D)) @ k0)) < 1e-12
        assert abs(e[g, 0] - brute_log_mass(q[g] / math.sqrt(D), K)) < 1e-12


# --- P2: first and second derivative of the exact log-mass at q = 0 -----------

def test_estimate_matches_curvature_of_exact_log_mass():
    r = rng(3)
    D, L = 6, 12
    K = r.normal(size=(L, D)) + r.normal(size=D)
    q = r.normal(size=(1, D))
    qs = q[0] / math.sqrt(D)
    f = lambda t: brute_log_mass(t * qs, K)
    h = 1e-3
    d1 = (f(h) - f(-h)) / (2 * h)
    d2 = (f(h) - 2 * f(0.0) + f(-h)) / (h * h)
    # full-rank factors so the quadratic form is the whole covariance
    mean, xi, _ = O.build_summaries(K, L, rank=D)
    e = O.log_mass_estimates(q, mean, xi, L)[0, 0]
    first = e - math.log(L) - 0.5 * sum((xi[0, i] @ qs) ** 2 for i in range(D))
    second = 2.0 * (e - math.log(L) - first)
    assert abs(f(0.0) - math.log(L)) < 1e-12
    assert abs(first - d1) < 1e-6 * max(1.0, abs(d1))
    assert abs(second - d2) < 2e-5 * max(1.0, abs(d2))
    # the 1/L normalisation, not 1/(L-1): the two differ by 9 % here
    assert abs(second * L / (L - 1) - d2) > 1e-2 * abs(d2)


# --- P3: Gaussian keys: second-order cumulant matches the log-MGF -------------

def test_gaussian_keys_log_mgf():
    r = rng(4)
    D, L = 8, 200_000
    A = r.normal(size=(D, D)) / math.sqrt(D)
    C = A @ A.T * 0.5
    mu = r.normal(size=D) * 0.3
    K = r.multivariate_normal(mu, C, size=L)
    q = r.normal(size=(1, D))
    qs = q[0] / math.sqrt(D)
    closed = qs @ mu + 0.5 * qs @ C @ qs          # ln E exp(q.X) for X ~ N(mu, C)
    exact = O.exact_log_masses(q, K, L, 1)[0, 0] - math.log(L)
    # L is huge here, so take the factors by the D x D covariance route (same factors, see the Gram pin)
    mean, xi, _ = O.scaled_eigenvectors_covariance(K, rank=D)
    est = O.log_mass_estimates(q, mean[None], xi[None], L)[0, 0] - math.log(L)
    assert abs(exact - closed) < 0.02
    assert abs(est - closed) < 0.01
    assert abs(est - exact) < 0.01


# --- P4: full rank recovers the covariance; truncation error bound ------------

def test_full_rank_recovers_quadratic_form_and_truncation_bound():
    r = rng(5)
    D, L = 24, 10            # D > L: covariance rank <= L - 1
    K = r.normal(size=(L, D))
    q = r.normal(size=D)
    kc = K - K.mean(axis=0)
    sigma = np.zeros((D, D))
    for t in range(L):
        sigma += np.outer(kc[t], kc[t]) / L
    full = q @ sigma @ q
    _, xi, lam = O.scaled_eigenvectors_gram(K, rank=L - 1)
    assert abs(sum((xi[i] @ q) ** 2 for i in range(L - 1)) - full) < 1e-11 * full
    evals = np.sort(np.linalg.eigvalsh(sigma))[::-1]
    assert np.allclose(lam, evals[:L - 1], rtol=1e-10, atol=1e-12)
    # rank L (one beyond the covariance rank): the extra factor is exactly zero
    _, xi_l, lam_l = O.scaled_eigenvectors_gram(K, rank=L)
    assert np.all(xi_l[L - 1] == 0.0) and lam_l[L - 1] == 0.0
    for rnk in (1, 2, 4):
        _, xr, _ = O.scaled_eigenvectors_gram(K, rank=rnk)
        part = sum((xr[i] @ q) ** 2 for i in range(rnk))
        assert -1e-12 <= full - part <= evals[rnk] * (q @ q) + 1e-12


# --- P5: Gram trick equals the covariance route --------------------------------

@pytest.mark.parametrize("subspace", [False, True])
def test_gram_route_equals_covariance_route(subspace):
    r = rng(6)
    D, L, rnk = 16, 8, 4
    K = r.normal(size=(L, D)) * r.uniform(0.2, 2.0, size=D)
    u_q = np.linalg.qr(r.normal(size=(D, 6)))[0] if subspace else None
    m1, x1, l1 = O.scaled_eigenvectors_gram(K, rnk, u_q)
    m2, x2, l2 = O.scaled_eigenvectors_covariance(K, rnk, u_q)
    assert np.allclose(m1, m2, atol=1e-14)
    assert np.allclose(l1, l2, rtol=1e-10)
    for i in range(rnk):
        assert np.allclose(np.outer(x1[i], x1[i]), np.outer(x2[i], x2[i]), atol=1e-10)
        assert abs(x1[i] @ x1[i] - l1[i]) < 1e-10            # |xi_i|^2 = lambda_i
        assert x1[i, np.argmax(np.abs(x1[i]))] > 0            # sign rule
        for j in range(i):
            assert abs(x1[i] @ x1[j]) < 1e-10
    # and both equal the sign-fixed sqrt(lambda) u from a library eigendecomposition
    assert np.allclose(x1, x2, atol=1e-9)


# --- P6: subspace projection is exact for queries inside the subspace ---------

def test_subspace_exact_inside_subspace_and_identity_basis():
    r = rng(7)
    D, L, s = 12, 32, 5
    K = r.normal(size=(L, D))
    u_q = np.linalg.qr(r.normal(size=(D, s)))[0]
    q_in = (u_q @ r.normal(size=s)) * math.sqrt(D)        # scaled query lies in span(U_Q)
    _, sigma = O.block_mean_and_covariance(K)
    _, xi_ss, _ = O.scaled_eigenvectors_gram(K, rank=s, u_q=u_q)   # full rank inside the subspace
    qs = q_in / math.sqrt(D)
    assert abs(sum((xi_ss[i] @ (u_q.T @ qs)) ** 2 for i in range(s)) - qs @ sigma @ qs) < 1e-11
    # U_Q = I reproduces the full-space descriptor
    m_a, x_a, _ = O.scaled_eigenvectors_gram(K, 3, None)
    m_b, x_b, _ = O.scaled_eigenvectors_gram(K, 3, np.eye(D))
    assert np.array_equal(m_a, m_b) and np.allclose(x_a, x_b, atol=1e-13)
    q = r.normal(size=(2, D))
    e_a = O.log_mass_estimates(q, m_a[None], x_a[None], L)
    e_b = O.log_mass_estimates(q, m_b[None], x_b[None], L, u_q=np.eye(D))
    assert np.allclose(e_a, e_b, atol=1e-12)


# --- P7: all blocks selected reproduces dense softmax attention ----------------

def brute_dense_attention(qs, K, V):
    w = [math.exp(sum(qs[j] * K[t, j] for j in range(K.shape[1]))) for t in range(K.shape[0])]
    z = sum(w)
    return np.array([sum(w[t] * V[t, d] for t in range(K.shape[0])) / z for d in range(V.shape[1])]), math.log(z)


@pytest.mark.parametrize("seq_len", [64, 61])
def test_all_blocks_selected_equals_dense(seq_len):
    r = rng(8)
    D, L, G, W = 4, 8, 2, 16
    K = r.normal(size=(seq_len, D)); V = r.normal(size=(seq_len, D)); q = r.normal(size=(G, D))
    n_sum = seq_len // L
    mean, xi, _ = O.build_summaries(K, L, 2, n_blocks=n_sum)
    st = O.store_summaries(mean, xi, "fp32")
    res = O.decode_step(q, K, V, seq_len, st, L, topk=1000, window=W)
    n_cand = O.window_start(seq_len, W, L) // L
    assert list(res["sel"]) == list(range(n_cand))
    for g in range(G):
        o, lse = brute_dense_attention(q[g] / math.sqrt(D), K, V)
        assert np.allclose(res["out"][g], o, atol=1e-12)
        assert abs(res["lse"][g] - lse) < 1e-12
    o_d, lse_d = O.dense_attention(q, K, V, seq_len)
    assert np.allclose(o_d, res["out"], atol=1e-12)


# --- P8: exact single-head error identity --------------------------------------

def test_error_identity_for_dropped_blocks():
    r = rng(9)
    D, L, NB = 5, 4, 6
    T = NB * L
    K = r.normal(size=(T, D)); V = r.normal(size=(T, D)); q = r.normal(size=(1, D))
    qs = q[0] / math.sqrt(D)
    m = np.array([sum(math.exp(qs @ K[t]) for t in range(b * L, (b + 1) * L)) for b in range(NB)])
    P = m / m.sum()
    cent = np.array([sum(math.exp(qs @ K[t]) * V[t] for t in range(b * L, (b + 1) * L)) / m[b] for b in range(NB)])
    o_star = (P[:, None] * cent).sum(axis=0)
    S = [1, 4]                      # kept blocks; window of zero tokens via seq_len == ws
    toks = np.concatenate([np.arange(b * L, (b + 1) * L) for b in S])
    o_hat, _ = O.attend(q, K, V, toks)
    tau = sum(P[b] for b in range(NB) if b not in S)
    rhs = sum(P[b] * (cent[b] - o_star) for b in range(NB) if b not in S) / (1 - tau)
    assert np.allclose(o_star - o_hat[0], rhs, atol=1e-13)
    assert np.allclose(O.dense_attention(q, K, V, T)[0][0], o_star, atol=1e-13)


# --- P9: group-score invariants --------------------------------------------------

def test_group_score_invariants():
    r = rng(10)
    G, NB = 4, 37
    e = r.normal(size=(G, NB)) * 3
    s = O.group_scores(e)
    assert abs(s.sum() - G) < 1e-12
    # brute force of the boxed GQA score with masses m = exp(e)
    for b in range(NB):
        ref = sum(math.exp(e[g, b]) / sum(math.exp(e[g, c]) for c in range(NB)) for g in range(G))
        assert abs(s[b] - ref) < 1e-12
    # per-head constant shifts (e.g. the ln L term) change nothing
    assert np.allclose(O.group_scores(e + r.normal(size=(G, 1))), s, atol=1e-12)
    # G = 1: ranking by score is ranking by log-mass
    e1 = e[:1]
    assert list(np.argsort(-O.group_scores(e1), kind="stable")) == list(np.argsort(-e1[0], kind="stable"))


def test_gqa_estimated_score_is_eq_gqa_secondorder():
    """Literal evaluation of the second-order GQA score with the D x D covariance."""
    r = rng(11)
    G, D, L, NB = 3, 6, 8, 5
    K = r.normal(size=(NB * L, D)); q = r.normal(size=(G, D))
    mean, xi, _ = O.build_summaries(K, L, rank=D)       # full rank: sum of factors = covariance
    s = O.group_scores(O.log_mass_estimates(q, mean, xi, L))
    qs = q / math.sqrt(D)
    t = np.zeros((G, NB))
    for g in range(G):
        for b in range(NB):
            kb, sig = O.block_mean_and_covariance(K[b * L:(b + 1) * L])
            t[g, b] = math.exp(qs[g] @ kb + 0.5 * qs[g] @ sig @ qs[g])
    ref = (t / t.sum(axis=1, keepdims=True)).sum(axis=0)
    assert np.allclose(s, ref, atol=1e-12)


# --- P10 / P11: numbers the paper prints ---------------------------------------

def test_descriptor_bytes_match_quantisation_table():
    for rank, dim, bf16_b, fp4_b in read_golden("quant_table.txt"):
        assert O.factor_bytes(int(rank), int(dim), "bf16") == int(bf16_b)
        assert O.factor_bytes(int(rank), int(dim), "fp4") == int(fp4_b)
    # "340 rather than 512 floats" at r = 4: s = 85 against D = 128
    assert 4 * 85 == 340 and 4 * 128 == 512


def test_summary_traffic_matches_bandwidth_table():
    n_blocks, hkv, D, L, k, W = 32768 // 32, 4, 128, 32, 16, 256
    for name, rank, sub, fmt, summ, win, fine in read_golden("traffic_table.txt"):
        if name == "dense":
            assert 32768 * hkv * D * 2 * 2 / 1024 == float(fine)
            continue
        got = O.summary_key_kib(n_blocks, hkv, D, int(rank), float(sub), fmt if fmt != "none" else "bf16")
        assert round(got) == int(summ), (name, got)
        assert W * hkv * D * 2 * 2 / 1024 == float(win)
        assert k * L * hkv * D * 2 * 2 / 1024 == float(fine)


def test_adaptive_sub_dim_rule_against_per_layer_figure():
    rows = [(int(a), int(b), int(c)) for a, b, c in read_golden("adaptive_s_per_layer.txt")]
    dark = [b for _, b, _ in rows]
    total = [b + c for _, b, c in rows]
    assert sum(dark) / 16 == 68.0 and sum(total) / 16 == 84.875
    for d, t in zip(dark, total):
        # the figure's dark bars are rounded head-averages, so allow the rounding slack
        assert abs(O.adaptive_sub_dim([d]) - t) <= 1
    assert O.adaptive_sub_dim([68.0]) == 85
    # energy rank: 90 % of a flat spectrum of 10 needs 9
    assert O.energy_rank(np.ones(10)) == 9
    assert O.energy_rank([8.0, 1.0, 0.5, 0.5]) == 2


def test_calibration_queries_give_sub_dim_85_and_basis():
    wl = synth.named_workloads()["cfg3a_32k_subspace"]
    ranks = []
    for h in range(2):
        qc = O.scale_query(synth.calibration_queries(wl, 4096, h).numpy())
        u, lam = O.query_subspace(qc, wl.sub_dim)
        ranks.append(O.energy_rank(lam))
        basis = synth.query_basis(wl)[h, :, :wl.sub_dim].numpy()
        # leading directions agree with the generator's population eigenvectors
        assert np.linalg.norm(basis[:, :8].T @ u[:, :16], axis=1).min() > 0.9
        assert np.allclose(u.T @ u, np.eye(wl.sub_dim), atol=1e-10)
    assert abs(O.adaptive_sub_dim(ranks) - 85) <= 3


# --- P12: the E2M1 grid ------------------------------------------------------------

def test_e2m1_grid_round_trip_ties_saturation():
    vals = np.concatenate([O.E2M1_MAGNITUDES, -O.E2M1_MAGNITUDES[1:]])
    # a vector whose max magnitude is 6 has scale exactly 1
    codes, scale = O.quantise_e2m1(vals[None, :])
    assert scale[0] == 1.0
    assert np.array_equal(O.dequantise_e2m1(codes, scale)[0], vals)
    ties = np.array([6.0, 0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, -0.25, -2.5])
    want = np.array([6.0, 0.0, 1.0, 1.0, 2.0, 2.0, 4.0, 4.0, -0.0, -2.0])
    codes, scale = O.quantise_e2m1(ties[None, :])
    assert np.array_equal(O.dequantise_e2m1(codes, scale)[0], want)
    assert codes[0, 8] == 8                           # small negative keeps its sign bit
    # nearest-value property on a dense grid, by brute force over the 8 magnitudes
    x = np.linspace(-6, 6, 4801)
    x[0] = -6.0; x[-1] = 6.0
    codes, scale = O.quantise_e2m1(x[None, :])
    deq = O.dequantise_e2m1(codes, scale)[0]
    for xv, dv in zip(x, deq):
        best = min(abs(abs(np.float32(xv)) - m) for m in O.E2M1_MAGNITUDES)
        assert abs(abs(np.float32(xv)) - abs(dv)) <= best + 1e-7
    # all-zero vector; fp16 scale
    codes, scale = O.quantise_e2m1(np.zeros((2, 8)))
    assert np.all(codes == 0) and np.all(scale == 0)
    xi = rng(12).normal(size=(5, 64))
    c16, s16 = O.quantise_e2m1(xi, "fp16")
    assert np.array_equal(s16, s16.astype(np.float16).astype(np.float32))
    c32, s32 = O.quantise_e2m1(xi, "fp32")
    assert np.max(np.abs(O.dequantise_e2m1(c32, s32) - xi)) <= np.max(s32) * 1.0 + 1e-6  # half the widest gap (2) * scale
    assert np.all((c32 & 7).max(axis=1) == 7)         # the largest entry maps to magnitude 6


def test_round_to_bf16_against_torch():
    import torch
    x = rng(13).normal(size=4096) * np.exp(rng(14).normal(size=4096) * 3)
    x32 = x.astype(np.float32)
    ref = torch.from_numpy(x32).to(torch.bfloat16).double().numpy()   # fp32 -> bf16 is a single RNE rounding
    assert np.array_equal(O.round_to_bf16(x32.astype(np.float64)), ref)
    assert O.round_to_bf16(1.0 + 2 ** -8) == 1.0 and O.round_to_bf16(1.0 + 3 * 2 ** -8) == 1.0 + 2 ** -6


# --- P13 / P14: planted blocks; tiny brute force of the whole step -----------------

def test_planted_blocks_found_in_tiny_config():
    wl = synth.named_workloads()["cfg1_tiny"]
    inp = synth.generate(wl)
    K, V = synth.unit_kv(inp, wl, 0, 0)
    q = synth.unit_q(inp, wl, 0, 0).numpy()
    K, V = K.numpy(), V.numpy()
    mean, xi, _ = O.build_summaries(K, wl.block_size, wl.rank)
    st = O.store_summaries(mean, xi, "fp32")
    res = O.decode_step(q, K, V, wl.seq_len, st, wl.block_size, wl.topk, wl.window)
    planted = set(inp["planted"][0, 0].tolist())
    assert planted <= set(res["sel"].tolist())
    n_cand = O.window_start(wl.seq_len, wl.window, wl.block_size) // wl.block_size
    exact = O.group_scores(O.exact_log_masses(q, K, wl.block_size, wl.seq_len // wl.block_size))
    assert planted <= set(O.select_topk(exact, n_cand, wl.topk).tolist())


def test_selection_order_ties_and_window():
    score = np.array([0.5, 0.9, 0.9, 0.1, 0.9, 0.7])
    assert list(O.select_topk(score, 6, 2)) == [1, 2]         # tie -> lower index
    assert list(O.select_topk(score, 6, 4)) == [1, 2, 4, 5]
    assert list(O.select_topk(score, 3, 5)) == [0, 1, 2]      # fewer candidates than k
    assert list(O.select_topk(score, 0, 5)) == []
    assert O.window_start(2048, 64, 64) == 1984
    assert O.window_start(2047, 64, 64) == 1920               # partial last block lies in the window
    assert O.window_start(40, 64, 64) == 0
    toks = O.token_set(np.array([0, 2]), 150, 32, 16)
    assert list(toks) == list(range(0, 16)) + list(range(32, 48)) + list(range(112, 150))


def test_skew_is_third_derivative_of_exact_log_mass_and_cuts_the_error_order():
    """Diagonal skew (Appendix, "Cheap diagonal skew").  (1) g_i is the third cumulant of the keys projected on
    u_i, i.e. the third derivative at 0 of t -> ln m_b(t u_i): checked by a central finite difference of the EXACT
    log mass.  (2) For a block whose keys vary along one direction only the diagonal is the whole third-order
    tensor: the estimate with the skew term is exact to O(t^4) where the second-order one is exact to O(t^3)
    (halving t divides the errors by ~16 and ~8 respectively), and the second-order error / t^3 tends to g / 6."""
    rng = np.random.default_rng(11)
    L, D, r = 32, 16, 3
    K = rng.standard_normal((L, D)) * np.array([2.0, 1.5, 1.2] + [0.3] * (D - 3))
    K[:, 0] = np.abs(K[:, 0]) ** 1.5                        # a skewed coordinate
    mean, xi, lam = O.scaled_eigenvectors_gram(K, r)
    c = O.block_skew(K, xi)
    for i in range(r):
        u = xi[i] / np.sqrt(lam[i])
        f = lambda t: O.exact_log_masses((t * u * np.sqrt(D))[None, :], K, L, 1)[0, 0]
        h = 0.02
        third = (f(2 * h) - 2 * f(h) + 2 * f(-h) - f(-2 * h)) / (2 * h ** 3)
        g = c[i] * lam[i] ** 1.5
        assert abs(third - g) <= 2e-3 * max(1.0, abs(g)), (i, third, g)
    assert abs(c[0]) > 1e-3                                  # the skewed direction has a skew to speak of
    # rank-one block: k_t = kbar + a_t v
    v = rng.standard_normal(D)
    v /= np.linalg.norm(v)
    a = rng.gamma(2.0, 1.0, L)
    K1 = 0.3 * rng.standard_normal(D)[None, :] + a[:, None] * v[None, :]
    mean1, xi1, lam1 = O.scaled_eigenvectors_gram(K1, 1)
    c1 = O.block_skew(K1, xi1)
    g1 = c1[0] * lam1[0] ** 1.5
    sign = np.sign(xi1[0] @ v)
    errs2, errs3 = [], []
    for t in (0.2, 0.1, 0.05):
        q = (t * sign * v * np.sqrt(D))[None, :]
        exact = O.exact_log_masses(q, K1, L, 1)[0, 0]
        e2 = O.log_mass_estimates(q, mean1[None], xi1[None], L)[0, 0]
        e3 = O.log_mass_estimates_skew(q, mean1[None], xi1[None], c1[None], L)[0, 0]
        errs2.append(exact - e2)
        errs3.append(exact - e3)
    assert 6.5 < errs2[0] / errs2[1] < 9.5 and 6.5 < errs2[1] / errs2[2] < 9.5       # O(t^3)
    assert 10.0 < errs3[0] / errs3[1] < 22.0 and 10.0 < errs3[1] / errs3[2] < 22.0   # O(t^4)
    assert all(abs(e3) < 0.01 * abs(e2) for e2, e3 in zip(errs2, errs3))
    assert abs(errs2[2] / 0.05 ** 3 - g1 / 6.0) <= 0.05 * abs(g1 / 6.0)
    # a null factor stores 0; sign of the factor does not matter for the correction
    assert O.block_skew(K1, np.zeros((1, D)))[0] == 0.0
    qq = rng.standard_normal((2, D))
    ea = O.log_mass_estimates_skew(qq, mean[None], xi[None], c[None], L)
    eb = O.log_mass_estimates_skew(qq, mean[None], -xi[None], O.block_skew(K, -xi)[None], L)
    assert np.allclose(ea, eb, rtol=0, atol=1e-12)


def test_adaptive_count_closed_form_and_brute_force():
    """The adaptive block count (an extension, not in the paper).  (1) Geometric scores 2^-1, 2^-2, ... hold
    1 - 2^-k of a total that tends to 1 in their k largest: k = ceil(log2(1 / tau)) up to the truncation of the
    series.  (2) Brute force over all subsets of small random score vectors: the count is the size of the smallest
    subset holding (1 - tau) of the total, and the selected set reaches that mass.  (3) Clamps and ties."""
    import itertools
    n = 40
    score = np.array([2.0 ** -(j + 1) for j in range(n)])
    rng = np.random.default_rng(3)
    perm = rng.permutation(n)
    shuffled = np.zeros(n)
    shuffled[perm] = score                                   # the order in memory must not matter
    for tau, want in ((0.5, 1), (0.3, 2), (0.25, 2), (0.2, 3), (0.01, 7), (1e-3, 10), (2.0 ** -20, 20)):
        assert O.adaptive_count(shuffled, n, tau, 1, n) == want, tau
        sel = O.select_adaptive(shuffled, n, tau, 1, n)
        assert sorted(sel.tolist()) == sorted(perm[:want].tolist())
    for trial in range(30):
        m = int(rng.integers(3, 11))
        s = rng.random(m) ** 3
        tau = float(rng.choice([0.05, 0.2, 0.5]))
        total = s.sum()
        best = m
        for size in range(1, m + 1):
            if any(sum(s[list(c)]) >= (1 - tau) * total for c in itertools.combinations(range(m), size)):
                best = size
                break
        k = O.adaptive_count(s, m, tau, 1, m)
        assert k == best, (trial, k, best)
        sel = O.select_adaptive(s, m, tau, 1, m)
        assert s[sel].sum() >= (1 - tau) * total and len(sel) == k
    s = np.array([5.0, 1.0, 1.0, 1.0, 1.0, 1.0])
    assert O.adaptive_count(s, 6, 0.5, 1, 6) == 1                       # 5 of 10
    assert O.adaptive_count(s, 6, 0.5, 3, 6) == 3                       # k_min
    assert O.adaptive_count(s, 6, 0.0, 1, 4) == 4                       # k_max
    assert O.adaptive_count(s, 4, 0.0, 1, 6) == 4                       # candidates only
    assert O.select_adaptive(s, 6, 0.25, 1, 6).tolist() == [0, 1, 2, 3]  # 5 + 1 + 1 + 1 = 8 >= 7.5; ties -> low index
    assert O.adaptive_count(s, 0, 0.1, 1, 6) == 0


def test_fast_scores_equal_loop_scores_and_whole_step_brute_force():
    r = rng(15)
    G, D, L, NB, rnk, W, k = 2, 4, 4, 4, 2, 4, 2
    T = NB * L
    K = r.normal(size=(T, D)); V = r.normal(size=(T, D)); q = r.normal(size=(G, D))
    mean, xi, _ = O.build_summaries(K, L, rnk)
    assert np.allclose(O.log_mass_estimates(q, mean, xi, L), O.log_mass_estimates_fast(q, mean, xi, L), atol=1e-13)
    st = O.store_summaries(mean, xi, "fp32")
    res = O.decode_step(q, K, V, T, st, L, k, W)
    # independent literal evaluation
    qs = q / math.sqrt(D)
    e = np.zeros((G, NB))
    for g in range(G):
        for b in range(NB):
            kb = K[b * L:(b + 1) * L]
            mu = kb.mean(axis=0)
            cov = (kb - mu).T @ (kb - mu) / L
            lam, u = np.linalg.eigh(cov)
            top = np.argsort(-lam)[:rnk]
            mu32 = mu.astype(np.float32).astype(np.float64)
            quad = 0.0
            for i in top:
                f = (math.sqrt(lam[i]) * u[:, i])
                f = f.astype(np.float32).astype(np.float64)
                quad += (f @ qs[g]) ** 2
            e[g, b] = math.log(L) + qs[g] @ mu32 + 0.5 * quad
    p = np.exp(e) / np.exp(e).sum(axis=1, keepdims=True)
    score = p.sum(axis=0)
    assert np.allclose(res["score"], score, atol=1e-12)
    n_cand = (T - W) // L
    order = sorted(range(n_cand), key=lambda b: (-score[b], b))[:k]
    assert sorted(order) == list(res["sel"])
    toks = sorted([t for b in order for t in range(b * L, (b + 1) * L)] + list(range(T - W, T)))
    for g in range(G):
        o, lse = brute_dense_attention(qs[g], K[toks], V[toks])
        assert np.allclose(res["out"][g], o, atol=1e-12) and abs(res["lse"][g] - lse) < 1e-12
