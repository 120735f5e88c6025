"""CPU oracle for the COBS per-decode-step path (test infrastructure, not product code).

This file is a plain, slow, double-precision restatement of what the paper's
method computes, written from the paper's equations so that a reader can check
each function against the cited passage by eye.  It is imported only by the
tests, by the smoke check and by the benchmark's CPU-baseline leg.  It shares no
code, table or constant with the CUDA library and never imports it.

Conventions
-----------
* All arithmetic is numpy float64 unless the storage format fixes a precision
  (the FP4 quantiser is defined in IEEE binary32, see ``quantise_e2m1``).
* Inputs that live in bf16 on the device are passed here as float64 arrays
  holding exactly the bf16 values.
* "q" is always the raw query; the attention scale 1/sqrt(D) is absorbed into
  it by ``scale_query`` (Background, Notation: the usual scale is folded into q).
* One call handles one KV head of one sequence: K, V are [T, D]; the G query
  heads sharing that KV head are the rows of q [G, D].

Parity pins
-----------
Every function below is pinned by tests that do not go through this file's own
formula: brute-force masses, finite-difference curvature of the exact log-mass,
the Gaussian log-MGF closed form, the D x D covariance route for the Gram trick,
dense softmax attention, the exact error identity, and the byte counts printed
in the paper's traffic and quantisation tables.  What the paper does not fix
(tie order, window alignment, normaliser domain, eigenvector sign, the FP4
scale formula and rounding rule) is a stated reading: parity unpinned by the
paper for those choices; they are tested for self-consistency only.
``block_skew`` / ``log_mass_estimates_skew`` (the paper's diagonal-skew variant) are
pinned by the third derivative of the exact log mass and by the order of the
remaining error.  ``adaptive_count`` / ``select_adaptive`` are an extension the paper does not
define; they are pinned by a closed form and by brute force over subsets.
"""

from __future__ import annotations

import numpy as np

# ---------------------------------------------------------------------------
# storage roundings
# ---------------------------------------------------------------------------


def round_to_bf16(x):
    """Round float64 values to the nearest bfloat16 (8 significant bits), ties to even.

    One rounding straight from double (no intermediate float32).  Values are
    assumed to be inside the normal bf16 range, which holds for every summary
    this project stores.
    """
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)  # x = m * 2**e, 0.5 <= |m| < 1
    return np.ldexp(np.rint(np.ldexp(m, 8)), e - 8)  # np.rint rounds half to even


def round_to_fp32(x):
    return np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)


# E2M1: 1 sign, 2 exponent, 1 mantissa bit.  Magnitudes by 3-bit code.
E2M1_MAGNITUDES = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0], dtype=np.float64)


def quantise_e2m1(xi, scale_dtype="fp32"):
    """FP4 (E2M1) quantiser with one scale per vector (Method, Quantization).

    The paper fixes the format (E2M1), the scale granularity (one scale per
    stored eigenvector) and that the mean stays bf16.  The scale formula and
    the rounding rule are this project's reading, defined in binary32 so that
    two implementations can agree bit for bit:

      a      = max_j |xi_j|
      scale  = a / 6                (binary32 division, round to nearest)
      scale  = fp16(scale)          (only when scale_dtype == "fp16")
      t_j    = xi_j / scale         (binary32 division)
      code_j = sign bit of xi_j, then the E2M1 magnitude nearest to |t_j|,
               ties to the code with an even mantissa bit, saturating at 6.
      scale == 0  ->  all codes 0.

    xi: float array [..., n]; it is first rounded to binary32 (the precision
    the factors have when they reach the quantiser).
    Returns (codes uint8 [..., n] with values 0..15, scale float32 [...]).
    """
    x = np.asarray(xi, dtype=np.float64).astype(np.float32)
    a = np.max(np.abs(x), axis=-1)
    scale = (a / np.float32(6.0)).astype(np.float32)
    if scale_dtype == "fp16":
        scale = scale.astype(np.float16).astype(np.float32)
    elif scale_dtype != "fp32":
        raise ValueError(scale_dtype)
    safe = np.where(scale > 0, scale, np.float32(1.0)).astype(np.float32)
    t = (np.abs(x) / safe[..., None]).astype(np.float32)
    # round |t| to the E2M1 grid, ties to even mantissa bit (codes 0, 2, 4, 6 are even)
    mag = np.zeros(t.shape, dtype=np.uint8)
    # thresholds are midpoints; the tie goes to the even neighbour
    mag += (t > np.float32(0.25)).astype(np.uint8)   # 0.25 ties to 0   (code 0, even)
    mag += (t >= np.float32(0.75)).astype(np.uint8)  # 0.75 ties to 1.0 (code 2, even)
    mag += (t > np.float32(1.25)).astype(np.uint8)   # 1.25 ties to 1.0 (code 2)
    mag += (t >= np.float32(1.75)).astype(np.uint8)  # 1.75 ties to 2.0 (code 4, even)
    mag += (t > np.float32(2.5)).astype(np.uint8)    # 2.5  ties to 2.0 (code 4)
    mag += (t >= np.float32(3.5)).astype(np.uint8)   # 3.5  ties to 4.0 (code 6, even)
    mag += (t > np.float32(5.0)).astype(np.uint8)    # 5.0  ties to 4.0 (code 6)
    sign = np.signbit(x).astype(np.uint8)
    codes = (sign << 3) | mag
    codes = np.where((scale > 0)[..., None], codes, np.uint8(0)).astype(np.uint8)
    return codes, scale


def dequantise_e2m1(codes, scale):
    """value(code) * scale, exact in double."""
    codes = np.asarray(codes, dtype=np.uint8)
    mag = E2M1_MAGNITUDES[codes & 7]
    val = np.where((codes & 8) != 0, -mag, mag)
    return val * np.asarray(scale, dtype=np.float64)[..., None]


# ---------------------------------------------------------------------------
# (a) per-block summaries
# ---------------------------------------------------------------------------


def block_mean_and_covariance(k_block):
    """First two cumulants of a block's empirical key distribution (Eq. cgf-cumulants).

    k_block: [L, D].  Mean over the L keys; covariance with the 1/L (not 1/(L-1))
    normalisation.
    """
    k_block = np.asarray(k_block, dtype=np.float64)
    L = k_block.shape[0]
    kbar = k_block.sum(axis=0) / L
    kc = k_block - kbar
    sigma = kc.T @ kc / L
    return kbar, sigma


# Eigenvalues below this fraction of the block's mean squared key norm are treated as zero.
NULL_EIGENVALUE_TOL = 1e-12


def canonical_sign(xi):
    """Eigenvector sign is free; fix it: the entry of largest magnitude is positive
    (first such entry on exact ties).  A reading, not something the paper states."""
    xi = np.array(xi, dtype=np.float64, copy=True)
    for i in range(xi.shape[0]):
        j = int(np.argmax(np.abs(xi[i])))
        if xi[i, j] < 0:
            xi[i] = -xi[i]
    return xi


def scaled_eigenvectors_gram(k_block, rank, u_q=None):
    """Top-r scaled eigenvectors by the Gram trick (Method, Cost: eigenvector computation).

    K~ = centred keys [L, D] (projected onto the query subspace, K~ U_Q, when
    u_q [D, s] is given).  Eigenpairs (lambda_i, w_i) of the L x L matrix
    K~ K~^T / L; stored factor xi_i = K~^T w_i / sqrt(L) = sqrt(lambda_i) u_i
    (Eq. lowrank).  Eigenvalues in descending order.  A direction whose
    eigenvalue is below NULL_EIGENVALUE_TOL times the block's mean squared key
    norm carries no variance (constant-key block, or rank beyond L - 1) and is
    returned as exact zeros.

    Returns (kbar [D], xi [rank, Ds], lam [rank]).
    """
    k_block = np.asarray(k_block, dtype=np.float64)
    L = k_block.shape[0]
    kbar = k_block.sum(axis=0) / L
    kc = k_block - kbar
    if u_q is not None:
        kc = kc @ np.asarray(u_q, dtype=np.float64)
    gram = kc @ kc.T / L
    lam, w = np.linalg.eigh(gram)  # ascending
    order = np.argsort(-lam, kind="stable")
    lam = lam[order]
    w = w[:, order]
    ds = kc.shape[1]
    xi = np.zeros((rank, ds))
    lam_out = np.zeros(rank)
    floor = NULL_EIGENVALUE_TOL * np.sum(k_block * k_block) / L
    for i in range(min(rank, L)):
        if lam[i] > floor:
            xi[i] = kc.T @ w[:, i] / np.sqrt(L)
            lam_out[i] = lam[i]
    return kbar, canonical_sign(xi), lam_out


def scaled_eigenvectors_covariance(k_block, rank, u_q=None):
    """Same factors by the direct route: eigenvectors of the D x D covariance
    (Eq. lowrank), or of B_b = U_Q^T Sigma_b U_Q (Eq. subspace).  Used only to
    check the Gram route."""
    k_block = np.asarray(k_block, dtype=np.float64)
    kbar, sigma = block_mean_and_covariance(k_block)
    if u_q is not None:
        u_q = np.asarray(u_q, dtype=np.float64)
        sigma = u_q.T @ sigma @ u_q
    lam, u = np.linalg.eigh(sigma)
    order = np.argsort(-lam, kind="stable")
    lam, u = lam[order], u[:, order]
    xi = np.zeros((rank, sigma.shape[0]))
    lam_out = np.zeros(rank)
    floor = NULL_EIGENVALUE_TOL * np.sum(k_block * k_block) / k_block.shape[0]
    for i in range(min(rank, sigma.shape[0])):
        if lam[i] > floor:
            xi[i] = np.sqrt(lam[i]) * u[:, i]
            lam_out[i] = lam[i]
    return kbar, canonical_sign(xi), lam_out


def build_summaries(K, block_size, rank, u_q=None, n_blocks=None):
    """Summaries of every full block of one KV head: mean [NB, D], xi [NB, r, Ds], lam [NB, r]."""
    K = np.asarray(K, dtype=np.float64)
    L = block_size
    nb = K.shape[0] // L if n_blocks is None else n_blocks
    D = K.shape[1]
    ds = D if u_q is None else np.asarray(u_q).shape[1]
    mean = np.zeros((nb, D))
    xi = np.zeros((nb, rank, ds))
    lam = np.zeros((nb, rank))
    for b in range(nb):
        mean[b], xi[b], lam[b] = scaled_eigenvectors_gram(K[b * L:(b + 1) * L], rank, u_q)
    return mean, xi, lam


def block_skew(k_block, xi):
    """Diagonal of the third cumulant in the stored eigenbasis (Appendix, "Cheap diagonal skew").

    For every stored factor xi_i = sqrt(lam_i) u_i of a block (full-space descriptor):
      g_i = 1/L * sum_{t in b} (u_i . (k_t - kbar))^3 .
    The correction to the block log-score is 1/6 * sum_i (u_i . q')^3 g_i.  With u_i . q' = (xi_i . q') / sqrt(lam_i)
    it equals 1/6 * sum_i c_i (xi_i . q')^3 for c_i = g_i / lam_i^(3/2), which is the scalar returned (and stored)
    per factor; a null factor (lam_i = 0) gets 0.
    k_block [L, D], xi [r, D] -> c [r].
    """
    k_block = np.asarray(k_block, dtype=np.float64)
    xi = np.asarray(xi, dtype=np.float64)
    L = k_block.shape[0]
    kbar = k_block.sum(axis=0) / L
    c = np.zeros(xi.shape[0])
    for i in range(xi.shape[0]):
        lam = float(xi[i] @ xi[i])
        if lam == 0.0:
            continue
        u = xi[i] / np.sqrt(lam)
        g = 0.0
        for t in range(L):
            g += float(u @ (k_block[t] - kbar)) ** 3
        g /= L
        c[i] = g / lam ** 1.5
    return c


def build_skew(K, block_size, xi):
    """``block_skew`` for every summarised block: K [T, D], xi [NB, r, D] (exact factors) -> [NB, r]."""
    K = np.asarray(K, dtype=np.float64)
    L = block_size
    return np.stack([block_skew(K[b * L:(b + 1) * L], xi[b]) for b in range(xi.shape[0])]) if xi.shape[0] else np.zeros((0, xi.shape[1]))


def log_mass_estimates_skew(q, mean, xi, skew, block_size):
    """Second-order estimate plus the diagonal third-cumulant term (Appendix, "Cheap diagonal skew"):
      e[g, b] = ln L + q'_g . kbar_b + 1/2 sum_i (xi_{b,i} . q'_g)^2 + 1/6 sum_i c_{b,i} (xi_{b,i} . q'_g)^3 .
    mean [NB, D], xi [NB, r, D] as stored, skew [NB, r] as stored (binary32 values)."""
    qs = scale_query(q)
    G, nb = qs.shape[0], mean.shape[0]
    e = np.zeros((G, nb))
    for g in range(G):
        for b in range(nb):
            val = np.log(block_size) + qs[g] @ mean[b]
            for i in range(xi.shape[1]):
                d = xi[b, i] @ qs[g]
                val += 0.5 * d * d + skew[b, i] * d * d * d / 6.0
            e[g, b] = val
    return e


def store_summaries(mean, xi, summary_dtype, scale_dtype="fp32"):
    """Round summaries to their storage format (Method, Quantization).

    summary_dtype "fp32": mean and factors binary32.
                  "bf16": mean and factors bf16.
                  "fp4":  mean bf16, factors E2M1 codes + one scale per factor.
    Returns a dict with the values scoring will see ("mean", "xi", float64 on
    the storage grid) and, for fp4, "codes" (uint8 0..15) and "scale" (float32).
    """
    if summary_dtype == "fp32":
        return {"mean": round_to_fp32(mean), "xi": round_to_fp32(xi)}
    if summary_dtype == "bf16":
        return {"mean": round_to_bf16(mean), "xi": round_to_bf16(xi)}
    if summary_dtype == "fp4":
        codes, scale = quantise_e2m1(xi, scale_dtype)
        return {"mean": round_to_bf16(mean), "xi": dequantise_e2m1(codes, scale),
                "codes": codes, "scale": scale}
    raise ValueError(summary_dtype)


# ---------------------------------------------------------------------------
# query subspace (Method, Subspace method; Ablations, adaptive vs. global)
# ---------------------------------------------------------------------------


def energy_rank(eigvals, fraction=0.9):
    """Smallest n such that the n largest eigenvalues hold `fraction` of the trace."""
    lam = np.sort(np.asarray(eigvals, dtype=np.float64))[::-1]
    c = np.cumsum(lam)
    return int(np.searchsorted(c, fraction * c[-1] - 1e-12 * c[-1]) + 1)


def adaptive_sub_dim(ranks90, factor=1.25):
    """s = factor x (rank holding 90 % of the query spectral energy, averaged over heads)."""
    return int(np.floor(factor * float(np.mean(ranks90)) + 0.5))


def query_subspace(q_cal, sub_dim):
    """U_Q: top `sub_dim` eigenvectors of the query second moment E[q q^T] (uncentred).

    q_cal: [n, D] calibration queries (already scaled).  Returns (U_Q [D, s], eigenvalues desc).
    """
    q_cal = np.asarray(q_cal, dtype=np.float64)
    m2 = q_cal.T @ q_cal / q_cal.shape[0]
    lam, u = np.linalg.eigh(m2)
    order = np.argsort(-lam, kind="stable")
    return u[:, order[:sub_dim]], lam[order]


# ---------------------------------------------------------------------------
# (b) block scores
# ---------------------------------------------------------------------------


def scale_query(q):
    """q' = q / sqrt(D): the attention scale absorbed into the query (Background, Notation)."""
    q = np.asarray(q, dtype=np.float64)
    return q / np.sqrt(q.shape[-1])


def log_mass_estimates(q, mean, xi, block_size, u_q=None):
    """Second-order estimate of ln m_b for every block and every head of the group.

    Eq. trunc with the curvature evaluated from the stored factors (Eq. gram):
      e[g, b] = ln L + q'_g . kbar_b + 1/2 * sum_i (xi_{b,i} . q~_g)^2,
    q~ = U_Q^T q' for the subspace descriptor, q' otherwise.
    q: [G, D] raw queries; mean [NB, D]; xi [NB, r, Ds] as stored.
    """
    qs = scale_query(q)
    qt = qs if u_q is None else qs @ np.asarray(u_q, dtype=np.float64)
    G, nb = qs.shape[0], mean.shape[0]
    e = np.zeros((G, nb))
    for g in range(G):
        for b in range(nb):
            first = qs[g] @ mean[b]
            second = 0.0
            for i in range(xi.shape[1]):
                second += (xi[b, i] @ qt[g]) ** 2
            e[g, b] = np.log(block_size) + first + 0.5 * second
    return e


def log_mass_estimates_fast(q, mean, xi, block_size, u_q=None):
    """Same quantity as ``log_mass_estimates`` with the loops handed to matmul
    (used where NB is in the thousands; tested equal to the loop version)."""
    qs = scale_query(q)
    qt = qs if u_q is None else qs @ np.asarray(u_q, dtype=np.float64)
    first = qs @ mean.T  # [G, NB]
    proj = np.einsum("bid,gd->gbi", xi, qt)
    return np.log(block_size) + first + 0.5 * np.sum(proj * proj, axis=-1)


def exact_log_masses(q, K, block_size, n_blocks):
    """ln m_b with m_b = sum_{t in b} exp(q' . k_t), by direct summation (Eq. bg-defs)."""
    qs = scale_query(q)
    K = np.asarray(K, dtype=np.float64)
    G = qs.shape[0]
    out = np.zeros((G, n_blocks))
    for g in range(G):
        for b in range(n_blocks):
            s = K[b * block_size:(b + 1) * block_size] @ qs[g]
            mx = s.max()
            out[g, b] = mx + np.log(np.sum(np.exp(s - mx)))
    return out


def group_scores(e):
    """GQA selection score (Eq. prop-gqa / Eq. gqa-secondorder).

    e: [G, NB] (estimated or exact) log masses over all summarised blocks.
    score_b = sum_g m_b^g / Z^g with Z^g = sum_b' m_b'^g, evaluated with the
    maximum subtracted.  The normaliser runs over every summarised block.
    """
    e = np.asarray(e, dtype=np.float64)
    mx = e.max(axis=1, keepdims=True)
    lse = mx + np.log(np.sum(np.exp(e - mx), axis=1, keepdims=True))
    return np.sum(np.exp(e - lse), axis=0)


# ---------------------------------------------------------------------------
# (c) selection
# ---------------------------------------------------------------------------


def window_start(seq_len, window, block_size):
    """First token of the local window, aligned down to a block boundary, so that
    selected blocks and the window never share a token (a reading; the paper
    lists a sliding-window branch beside the selection branch)."""
    return (max(0, seq_len - window) // block_size) * block_size


def select_topk(score, n_candidates, topk):
    """Indices of the topk largest scores among blocks 0..n_candidates-1.

    Larger score first, lower index on exact ties; returned in ascending index order.
    """
    cand = list(range(n_candidates))
    cand.sort(key=lambda b: (-score[b], b))
    return np.array(sorted(cand[:min(topk, n_candidates)]), dtype=np.int64)


def adaptive_count(score, n_candidates, tau, k_min, k_max):
    """Adaptive number of selected blocks.  NOT IN THE PAPER (the paper always keeps k blocks): an extension
    built on the paper's dropped mass tau = sum of the normalised block masses outside the kept set S
    (Background, the renormalisation paragraph before Eq. prop-gqa), applied to the group score of Eq. prop-gqa:

      k_adapt = the smallest k such that the k largest candidate scores hold at least (1 - tau) of the
                candidates' total score, clamped to [k_min, k_max] and to the number of candidates.

    Ties in the ordering: lower index first, as in ``select_topk``.
    """
    s = np.asarray(score, dtype=np.float64)[:n_candidates]
    if n_candidates == 0:
        return 0
    order = sorted(range(n_candidates), key=lambda b: (-s[b], b))
    total = 0.0
    for b in range(n_candidates):
        total += s[b]
    need = (1.0 - float(tau)) * total
    k, cum = n_candidates, 0.0
    for j, b in enumerate(order):
        cum += s[b]
        if cum >= need:
            k = j + 1
            break
    return int(min(max(k, k_min), k_max, n_candidates))


def select_adaptive(score, n_candidates, tau, k_min, k_max):
    """The ``adaptive_count`` largest candidate scores, ascending index order (extension, not in the paper)."""
    return select_topk(score, n_candidates, adaptive_count(score, n_candidates, tau, k_min, k_max))


# ---------------------------------------------------------------------------
# (d) attention over selected blocks + window
# ---------------------------------------------------------------------------


def token_set(sel, seq_len, window, block_size):
    ws = window_start(seq_len, window, block_size)
    toks = [np.arange(b * block_size, (b + 1) * block_size) for b in sel]
    toks.append(np.arange(ws, seq_len))
    return np.concatenate(toks) if toks else np.zeros(0, dtype=np.int64)


def attend(q, K, V, tokens):
    """Softmax attention restricted to a token set: Eq. oracle-true, the kept
    blocks renormalised among themselves.  Returns (o [G, D], lse [G])."""
    qs = scale_query(q)
    K = np.asarray(K, dtype=np.float64)[tokens]
    V = np.asarray(V, dtype=np.float64)[tokens]
    s = qs @ K.T  # [G, n]
    mx = s.max(axis=1, keepdims=True)
    p = np.exp(s - mx)
    z = p.sum(axis=1, keepdims=True)
    return (p / z) @ V, (mx + np.log(z))[:, 0]


def dense_attention(q, K, V, seq_len):
    return attend(q, K, V, np.arange(seq_len))


def decode_step(q, K, V, seq_len, stored, block_size, topk, window, u_q=None):
    """One decode step for one KV head: scores -> selection -> attention.

    stored: output of ``store_summaries`` for blocks 0..floor(seq_len/L)-1.
    Returns dict(e, score, sel, out, lse).
    """
    n_sum = seq_len // block_size
    e = log_mass_estimates_fast(q, stored["mean"][:n_sum], stored["xi"][:n_sum], block_size, u_q)
    score = group_scores(e) if n_sum > 0 else np.zeros(0)
    n_cand = window_start(seq_len, window, block_size) // block_size
    sel = select_topk(score, n_cand, topk)
    out, lse = attend(q, K, V, token_set(sel, seq_len, window, block_size))
    return {"e": e, "score": score, "sel": sel, "out": out, "lse": lse}


# ---------------------------------------------------------------------------
# traffic accounting (Experiments, KV cache read traffic study)
# ---------------------------------------------------------------------------


def factor_bytes(rank, ds, fmt):
    """Bytes of the covariance factors of one block descriptor (mean excluded)."""
    if fmt == "bf16":
        return rank * ds * 2
    if fmt == "fp4":
        return rank * ds / 2 + 4 * rank  # packed nibbles + one fp32 scale per factor
    raise ValueError(fmt)


def summary_key_kib(n_blocks, n_kv_heads, head_dim, rank, ds, fmt):
    """'Summary keys' column of the traffic table: bf16 mean + factors, all blocks, all KV heads."""
    per = 2 * head_dim + (factor_bytes(rank, ds, fmt) if rank > 0 else 0)
    return n_blocks * n_kv_heads * per / 1024.0
