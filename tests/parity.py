"""Helpers shared by the parity tests: run the oracle per (sequence, KV head) unit, upload its
summaries bit for bit into the device arrays, and the comparison rules.

Comparison rules
  scores    relative error against the oracle's double-precision score
  selection with theta = the oracle's k-th largest score and the band
            {b : |score_b - theta| <= 1e-5 * |theta|}: the device set must hold every oracle-selected
            block outside the band, no unselected block outside the band, and have the same size
  output    per (sequence, query head): max_j |o_gpu - o_ref| / max_j |o_ref| <= 2e-3
"""

from __future__ import annotations

import numpy as np
import torch

from oracle import cobs_oracle as O
from paper_2607_09052_b200 import synth

OUT_TOL = 2e-3
TIE_BAND = 1e-5
SCORE_TOL = 2e-5


def oracle_unit_summaries(wl, inp, b, h, n_blocks=None):
    """Oracle summaries of one unit, rounded to the workload's storage format."""
    K, _ = synth.unit_kv(inp, wl, b, h)
    u_q = inp["u_q"][h].double().cpu().numpy() if wl.sub_dim else None
    n_sum = int(inp["seq_lens"][b]) // wl.block_size if n_blocks is None else n_blocks
    mean, xi, lam = O.build_summaries(K.numpy(), wl.block_size, wl.rank, u_q, n_blocks=n_sum)
    st = O.store_summaries(mean, xi, wl.summary_dtype, wl.scale_dtype)
    st["lam"] = lam
    st["xi_exact"] = xi
    st["mean_exact"] = mean
    return st


def oracle_unit_step(wl, inp, b, h, stored):
    K, V = synth.unit_kv(inp, wl, b, h)
    q = synth.unit_q(inp, wl, b, h).numpy()
    u_q = inp["u_q"][h].double().cpu().numpy() if wl.sub_dim else None
    return O.decode_step(q, K.numpy(), V.numpy(), int(inp["seq_lens"][b]), stored, wl.block_size, wl.topk,
                         wl.window, u_q)


def oracle_attend(wl, inp, b, h, sel):
    K, V = synth.unit_kv(inp, wl, b, h)
    q = synth.unit_q(inp, wl, b, h).numpy()
    toks = O.token_set(np.asarray(sel, dtype=np.int64), int(inp["seq_lens"][b]), wl.window, wl.block_size)
    return O.attend(q, K.numpy(), V.numpy(), toks)


def upload_unit_summaries(binding, cfg, summ, b, h, stored):
    """Write one unit's oracle summaries into the device arrays, same bits."""
    mean_v, xi_v, scale_v = binding.summary_views(cfg, summ)
    n = stored["mean"].shape[0]
    if n == 0:
        return
    dev = mean_v.device
    mean_v[b, h, :n] = torch.from_numpy(stored["mean"]).to(mean_v.dtype).to(dev)
    if cfg.rank == 0:
        return
    if cfg.summary_dtype == 2:
        codes = torch.from_numpy(stored["codes"]).to(dev)
        xi_v[b, h, :n] = binding.pack_fp4_rows(codes, binding.cobs_padded_sub_dim(cfg))
        scale_v[b, h, :n] = torch.from_numpy(stored["scale"]).to(scale_v.dtype).to(dev)
    else:
        xi_v[b, h, :n] = torch.from_numpy(stored["xi"]).to(xi_v.dtype).to(dev)


def check_selection(gpu_sel, oracle_score, n_cand, topk):
    """Apply the tie-band rule.  Returns (ok, message, exact_match)."""
    k = min(topk, n_cand)
    gpu = [int(x) for x in gpu_sel if x >= 0]
    if len(gpu) != k:
        return False, f"count {len(gpu)} != {k}", False
    if gpu != sorted(set(gpu)):
        return False, "not ascending / not distinct", False
    if any(x >= n_cand for x in gpu):
        return False, "selected a non-candidate block", False
    ref = list(O.select_topk(oracle_score, n_cand, topk))
    if gpu == ref:
        return True, "", True
    if k == 0:
        return True, "", True
    theta = sorted(oracle_score[:n_cand], reverse=True)[k - 1]
    band = {b for b in range(n_cand) if abs(oracle_score[b] - theta) <= TIE_BAND * abs(theta)}
    missing = [b for b in ref if b not in gpu and b not in band]
    extra = [b for b in gpu if b not in ref and b not in band]
    if missing or extra:
        return False, f"outside tie band: missing {missing} extra {extra}", False
    return True, "tie swap inside band", False


def out_rel_err(o_gpu, o_ref):
    o_gpu = np.asarray(o_gpu, dtype=np.float64)
    return np.max(np.abs(o_gpu - o_ref), axis=-1) / np.max(np.abs(o_ref), axis=-1)
