"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same
seeded inputs.  Summaries for the score/select/attend checks are built by the oracle and uploaded
bit for bit, so selection can be compared exactly (up to the tie band) and outputs within 2e-3.
"""

import numpy as np
import pytest
import torch

from oracle import cobs_oracle as O
from paper_2607_09052_b200 import synth
from parity import (OUT_TOL, SCORE_TOL, check_selection, oracle_attend, oracle_unit_step, oracle_unit_summaries,
                    out_rel_err, upload_unit_summaries)

pytestmark = pytest.mark.gpu

WL = synth.named_workloads()


def _binding():
    from paper_2607_09052_b200 import binding
    return binding


def to_dev(inp):
    return {k: (v.cuda() if isinstance(v, torch.Tensor) and k != "planted" else v) for k, v in inp.items()}


def run_stage_s(wl, inp_cpu=None, units=None, inp_dev=None, summ=None):
    """Score/select/attend parity for the given units (all by default). Returns a small report."""
    B = _binding()
    if inp_dev is None:
        inp_cpu = synth.generate(wl) if inp_cpu is None else inp_cpu
        inp_dev = to_dev(inp_cpu)
    src = inp_dev if inp_cpu is None else inp_cpu      # where the oracle reads its inputs from
    cfg = B.make_config(wl)
    kv = B.make_kv(inp_dev)
    if summ is None:
        summ = B.SummaryBuffers(cfg, "cuda", inp_dev.get("u_q"))
    ws = B.alloc_workspace(cfg, "cuda")
    nb, hq, hkv, G, D = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.group, wl.head_dim
    if units is None:
        units = [(b, h) for b in range(nb) for h in range(hkv)]
    ref = {}
    for (b, h) in units:
        st = oracle_unit_summaries(wl, src, b, h)
        upload_unit_summaries(B, cfg, summ, b, h, st)
        ref[(b, h)] = oracle_unit_step(wl, src, b, h, st)

    sel_idx = torch.full((nb, hkv, wl.topk), -7, dtype=torch.int32, device="cuda")
    sel_cnt = torch.full((nb, hkv), -7, dtype=torch.int32, device="cuda")
    scores = torch.zeros((nb, hkv, wl.max_blocks), dtype=torch.float32, device="cuda")
    B.cobs_score_select(cfg, inp_dev["q"], summ, inp_dev["seq_lens"], sel_idx, sel_cnt, scores, ws)

    # attention on the ORACLE's selection, so a tie swap can neither hide nor fake an output error
    sel_ref = torch.full((nb, hkv, wl.topk), -1, dtype=torch.int32)
    cnt_ref = torch.zeros((nb, hkv), dtype=torch.int32)
    for (b, h), r in ref.items():
        sel_ref[b, h, :len(r["sel"])] = torch.from_numpy(r["sel"]).int()
        cnt_ref[b, h] = len(r["sel"])
    out_a = torch.zeros((nb, hq, D), dtype=torch.float32, device="cuda")
    lse_a = torch.zeros((nb, hq), dtype=torch.float32, device="cuda")
    B.cobs_sparse_decode(cfg, inp_dev["q"], kv, sel_ref.cuda(), cnt_ref.cuda(), out_a, lse_a, ws)

    out_f = torch.zeros_like(out_a)
    lse_f = torch.zeros_like(lse_a)
    sel_f = torch.full_like(sel_idx, -7)
    cnt_f = torch.full_like(sel_cnt, -7)
    B.cobs_decode_step(cfg, inp_dev["q"], kv, summ, out_f, lse_f, sel_f, cnt_f, ws)
    assert B.cobs_read_status(ws) == 0
    torch.cuda.synchronize()

    sel_idx, sel_cnt, scores = sel_idx.cpu(), sel_cnt.cpu(), scores.cpu().double().numpy()
    out_a, lse_a, out_f, lse_f = out_a.cpu().numpy(), lse_a.cpu().numpy(), out_f.cpu().numpy(), lse_f.cpu().numpy()
    sel_f, cnt_f = sel_f.cpu(), cnt_f.cpu()
    report = {"swaps": 0, "max_score_err": 0.0, "max_out_err": 0.0}
    for (b, h), r in ref.items():
        T = int(src["seq_lens"][b])
        n_sum = T // wl.block_size
        n_cand = O.window_start(T, wl.window, wl.block_size) // wl.block_size
        if n_sum:
            err = np.max(np.abs(scores[b, h, :n_sum] - r["score"]) / np.maximum(r["score"], 1e-30))
            report["max_score_err"] = max(report["max_score_err"], float(err))
            assert err <= SCORE_TOL, (b, h, err)
        ok, msg, exact = check_selection(sel_idx[b, h].tolist(), r["score"], n_cand, wl.topk)
        assert ok, (b, h, msg)
        assert int(sel_cnt[b, h]) == min(wl.topk, n_cand)
        assert all(int(x) == -1 for x in sel_idx[b, h, int(sel_cnt[b, h]):])
        report["swaps"] += 0 if exact else 1
        # fused step: same selection bits as the two-call path
        assert torch.equal(sel_f[b, h], sel_idx[b, h]) and int(cnt_f[b, h]) == int(sel_cnt[b, h])
        hs = slice(h * G, (h + 1) * G)
        ea = out_rel_err(out_a[b, hs], r["out"])
        assert np.all(ea <= OUT_TOL), (b, h, ea)
        assert np.allclose(lse_a[b, hs], r["lse"], atol=2e-3, rtol=0)
        if exact:
            ref_out, ref_lse = r["out"], r["lse"]
        else:
            ref_out, ref_lse = oracle_attend(wl, src, b, h, [int(x) for x in sel_f[b, h] if x >= 0])
        ef = out_rel_err(out_f[b, hs], ref_out)
        assert np.all(ef <= OUT_TOL), (b, h, ef)
        assert np.allclose(lse_f[b, hs], ref_lse, atol=2e-3, rtol=0)
        report["max_out_err"] = max(report["max_out_err"], float(ea.max()), float(ef.max()))
    return report


# --- the named workloads -------------------------------------------------------------------------------

def test_cfg1_tiny_all_entry_points():
    rep = run_stage_s(WL["cfg1_tiny"])
    assert rep["swaps"] == 0


def test_cfg2_32k_full():
    run_stage_s(WL["cfg2_32k"])


def test_cfg3a_subspace_fp4():
    run_stage_s(WL["cfg3a_32k_subspace"].replace(batch=2))


def test_cfg3b_k85_fp4():
    run_stage_s(WL["cfg3b_32k_k85"].replace(batch=2), units=[(0, 0), (0, 5), (1, 3), (1, 7)])


def test_cfg4_reduced_paged_rank8():
    wl = WL["cfg4_128k"].replace(batch=2, seq_len=16384)
    run_stage_s(wl)


def test_cfg5_reduced_g8_block128():
    wl = WL["cfg5_64k_g8"].replace(batch=2, seq_len=8192)
    run_stage_s(wl)


def test_cfg4_full_size_sampled_units():
    """Full 128k x 16 workload in the launch configuration the benchmark times: inputs drawn on the
    device, summaries built on the device for every block, then the sampled units' summaries replaced
    by the oracle's so that their selection can be compared exactly."""
    B = _binding()
    wl = WL["cfg4_128k"]
    inp = synth.generate(wl, "cuda")
    cfg = B.make_config(wl)
    summ = B.SummaryBuffers(cfg, "cuda")
    ws = B.alloc_workspace(cfg, "cuda")
    B.cobs_build_summaries(cfg, B.make_kv(inp), 0, wl.max_blocks, summ, ws)
    assert B.cobs_read_status(ws) == 0
    # the 128 units are scored in four waves of 32: the first and the last unit of every wave, and one inside
    units = [(0, 0), (3, 7), (4, 0), (7, 3), (7, 7), (8, 0), (11, 7), (12, 0), (15, 7)]
    run_stage_s(wl, inp_dev=inp, units=units, summ=summ)
    check_fused_equals_two_calls_on_every_unit(wl, inp, summ)


def check_fused_equals_two_calls_on_every_unit(wl, inp, summ):
    """For EVERY unit (no oracle time needed): cobs_decode_step selects exactly what cobs_score_select selects, and
    its output is cobs_sparse_decode's on that selection up to fp32 reassociation."""
    B = _binding()
    cfg = B.make_config(wl)
    kv = B.make_kv(inp)
    ws = B.alloc_workspace(cfg, "cuda")
    nb, hq, hkv, D = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim
    sel = torch.full((nb, hkv, wl.topk), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((nb, hkv), -7, dtype=torch.int32, device="cuda")
    B.cobs_score_select(cfg, inp["q"], summ, inp["seq_lens"], sel, cnt, None, ws)
    out_a = torch.zeros((nb, hq, D), dtype=torch.float32, device="cuda")
    lse_a = torch.zeros((nb, hq), dtype=torch.float32, device="cuda")
    B.cobs_sparse_decode(cfg, inp["q"], kv, sel, cnt, out_a, lse_a, ws)
    sel_f, cnt_f = torch.full_like(sel, -7), torch.full_like(cnt, -7)
    out_f, lse_f = torch.zeros_like(out_a), torch.zeros_like(lse_a)
    B.cobs_decode_step(cfg, inp["q"], kv, summ, out_f, lse_f, sel_f, cnt_f, ws)
    assert B.cobs_read_status(ws) == 0
    assert torch.equal(sel, sel_f) and torch.equal(cnt, cnt_f)
    lens = inp["seq_lens"].cpu().tolist()
    want = torch.tensor([min(wl.topk, O.window_start(t, wl.window, wl.block_size) // wl.block_size) for t in lens],
                        dtype=torch.int32)
    assert torch.equal(cnt.cpu(), want[:, None].expand(nb, hkv))
    s = sel.cpu()
    for b in range(nb):                                       # ascending, distinct, candidates only, -1 padding
        k = int(want[b])
        assert torch.all(s[b, :, k:] == -1)
        if k:
            assert torch.all(s[b, :, :k] >= 0) and torch.all(s[b, :, :k] < O.window_start(lens[b], wl.window, wl.block_size) // wl.block_size)
            assert torch.all(s[b, :, 1:k] > s[b, :, :k - 1])
    scale = out_a.abs().amax(dim=-1, keepdim=True).clamp_min(1e-30)
    assert float(((out_f - out_a).abs() / scale).max()) <= 1e-5
    assert float((lse_f - lse_a).abs().max()) <= 1e-5


def test_cfg5_full_size_sampled_units():
    """Configuration 5 at full size (8 sequences x 64k, blocks of 128, groups of 8 heads), as the benchmark runs it."""
    B = _binding()
    wl = WL["cfg5_64k_g8"]
    inp = synth.generate(wl, "cuda")
    cfg = B.make_config(wl)
    summ = B.SummaryBuffers(cfg, "cuda")
    ws = B.alloc_workspace(cfg, "cuda")
    B.cobs_build_summaries(cfg, B.make_kv(inp), 0, wl.max_blocks, summ, ws)
    assert B.cobs_read_status(ws) == 0
    run_stage_s(wl, inp_dev=inp, units=[(0, 0), (3, 5), (7, 7)], summ=summ)
    check_fused_equals_two_calls_on_every_unit(wl, inp, summ)


def test_cfg3a_full_batch_sampled_units():
    """Configuration 3A (subspace descriptor, packed E2M1) at its full batch of four sequences."""
    B = _binding()
    wl = WL["cfg3a_32k_subspace"]
    cpu = synth.generate(wl)
    inp = to_dev(cpu)
    cfg = B.make_config(wl)
    summ = B.SummaryBuffers(cfg, "cuda", inp.get("u_q"))
    ws = B.alloc_workspace(cfg, "cuda")
    B.cobs_build_summaries(cfg, B.make_kv(inp), 0, wl.max_blocks, summ, ws)
    assert B.cobs_read_status(ws) == 0
    run_stage_s(wl, inp_cpu=cpu, inp_dev=inp, units=[(0, 0), (1, 6), (2, 3), (3, 7)], summ=summ)
    check_fused_equals_two_calls_on_every_unit(wl, inp, summ)


# --- the opt-in tcgen05 scoring path ------------------------------------------------------------------------

@pytest.mark.parametrize("case", ["cfg2_32k_fp4_rank8", "cfg4_reduced", "ragged_g8_fp16_scales"])
def test_tcgen05_scoring_path(case, monkeypatch):
    """Same parity bar with phase S on tcgen05 (TMA-unpacked E2M1 rows x two-term E4M3 query, TMEM accumulators)."""
    B = _binding()
    if case == "cfg2_32k_fp4_rank8":
        wl = WL["cfg2_32k"].replace(summary_dtype="fp4", rank=8)
    elif case == "cfg4_reduced":
        wl = WL["cfg4_128k"].replace(batch=3, seq_len=16384)
    else:
        lens = [64 * 40 + 5, 64 * 96, 100, 64 * 33]
        wl = synth.Workload("ragged_tc", len(lens), 16, 2, 128, 64 * 96, 64, 16, rank=8, topk=12, window=200,
                            summary_dtype="fp4", scale_dtype="fp16", key_model="block_offset", planted=2,
                            shuffle_pages=True, seed=21, seq_lens=lens)
    monkeypatch.setenv("COBS_SCORE_PATH", "tcgen05")
    before = B.cobs_tcgen05_launches()
    run_stage_s(wl)
    assert B.cobs_tcgen05_launches() >= before + 2      # cobs_score_select and cobs_decode_step both took it
    monkeypatch.delenv("COBS_SCORE_PATH")
    before = B.cobs_tcgen05_launches()
    run_stage_s(wl, units=[(0, 0)])
    assert B.cobs_tcgen05_launches() == before          # and the default path does not


# --- the exact-mass selector (OSA) -----------------------------------------------------------------------------

@pytest.mark.parametrize("case", ["cfg2_32k", "paged_g8_d64_ragged"])
def test_exact_mass_selector_matches_oracle(case):
    """cobs_exact_select against the oracle's direct summation (Eq. bg-defs) + group score + top-k."""
    B = _binding()
    if case == "cfg2_32k":
        wl = WL["cfg2_32k"]
    else:
        lens = [32 * 21 + 7, 32 * 40, 19, 32 * 3]
        wl = synth.Workload("osa", len(lens), 16, 2, 64, 32 * 40, 32, 16, rank=2, topk=5, window=70, summary_dtype="bf16",
                            key_model="block_offset", planted=2, shuffle_pages=True, seed=51, seq_lens=lens)
    inp = synth.generate(wl)
    dev = to_dev(inp)
    cfg = B.make_config(wl)
    ws = B.alloc_workspace(cfg, "cuda")
    nb, hkv, G, L = wl.batch, wl.n_kv_heads, wl.group, wl.block_size
    sel = torch.full((nb, hkv, wl.topk), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((nb, hkv), -7, dtype=torch.int32, device="cuda")
    scores = torch.zeros((nb, hkv, wl.max_blocks), dtype=torch.float32, device="cuda")
    B.cobs_exact_select(cfg, dev["q"], B.make_kv(dev), sel, cnt, scores, ws)
    assert B.cobs_read_status(ws) == 0
    sel, cnt, scores = sel.cpu(), cnt.cpu(), scores.cpu().double().numpy()
    for b in range(nb):
        T = int(inp["seq_lens"][b])
        n_sum = T // L
        n_cand = O.window_start(T, wl.window, L) // L
        for h in range(hkv):
            K, _ = synth.unit_kv(inp, wl, b, h)
            q = synth.unit_q(inp, wl, b, h).numpy()
            assert int(cnt[b, h]) == min(wl.topk, n_cand)
            if n_sum == 0:
                continue
            ref = O.group_scores(O.exact_log_masses(q, K.numpy(), L, n_sum))
            err = np.max(np.abs(scores[b, h, :n_sum] - ref) / np.maximum(ref, 1e-30))
            assert err <= SCORE_TOL, (b, h, err)
            ok, msg, _ = check_selection(sel[b, h].tolist(), ref, n_cand, wl.topk)
            assert ok, (b, h, msg)


# --- shapes and edge cases ---------------------------------------------------------------------------------

@pytest.mark.parametrize("summary_dtype,scale_dtype", [("fp32", "fp32"), ("bf16", "fp32"), ("fp4", "fp32"),
                                                       ("fp4", "fp16")])
@pytest.mark.parametrize("G,D,L,P", [(1, 64, 32, 16), (2, 128, 64, 32), (4, 64, 128, 16), (8, 128, 16, 16)])
def test_shape_grid(summary_dtype, scale_dtype, G, D, L, P):
    wl = synth.Workload("grid", 2, 2 * G, 2, D, 40 * L, L, P, rank=3, topk=5, window=2 * L + 7,
                        summary_dtype=summary_dtype, scale_dtype=scale_dtype, key_model="block_offset",
                        planted=2, shuffle_pages=True, seed=11)
    run_stage_s(wl)


def test_ragged_lengths_and_degenerate_cases():
    L = 64
    # T < L (no summarised block), T inside the window only, partial last block, k larger than candidates
    lens = [37, 200, 64 * 9 + 13, 64 * 30, 1]
    wl = synth.Workload("ragged", len(lens), 8, 2, 128, 64 * 30, L, 16, rank=4, topk=12, window=130,
                        summary_dtype="bf16", key_model="block_offset", planted=1, shuffle_pages=True, seed=12,
                        seq_lens=lens)
    run_stage_s(wl)


def test_selection_exact_ties_for_every_blocks_per_thread_layout():
    """The selection team spreads a unit's blocks 4, 8 or 16 per thread depending on the unit's block count.
    Synthetic summaries with two kinds of block (every 16th block "hot", the rest "cold", identical within a kind)
    make every score one of two values, exactly: the top-k must be all hot candidates plus the LOWEST-index cold
    ones (ties -> lower index), for block counts on both sides of each layout boundary, in one batch."""
    B = _binding()
    L, D, G, NB, topk = 16, 64, 4, 2048, 48
    n_sums = [3, 100, 511, 512, 513, 1024, 1025, 2047, 2048]
    lens = [n * L + ((7 * i) % L if n < NB else 0) for i, n in enumerate(n_sums)]
    wl = synth.Workload("ties", len(lens), G, 1, D, NB * L, L, 16, rank=2, topk=topk, window=70, summary_dtype="bf16",
                        key_model="iid", seed=3, seq_lens=lens)
    inp = synth.generate(wl)
    gen = torch.Generator().manual_seed(5)
    v = torch.randn(D, generator=gen)
    q = (v[None, None, :] + 0.3 * torch.randn(len(lens), G, D, generator=gen)).to(torch.bfloat16)
    inp["q"] = q
    hot = (0.5 * v).to(torch.bfloat16)
    cold = (-0.5 * v).to(torch.bfloat16)
    f = (0.2 * torch.randn(2, D, generator=gen)).to(torch.bfloat16)
    assert float((q.float() @ (hot.float() - cold.float())).min()) > 0        # hot beats cold for every head
    dev = to_dev(inp)
    cfg = B.make_config(wl)
    summ = B.SummaryBuffers(cfg, "cuda")
    ws = B.alloc_workspace(cfg, "cuda")
    mean_v, xi_v, _ = B.summary_views(cfg, summ)
    is_hot = (torch.arange(NB) % 16 == 0)
    mean_all = torch.where(is_hot[:, None], hot[None, :], cold[None, :])
    mean_v[:, 0] = mean_all.cuda()[None]
    xi_v[:, 0] = f.cuda()[None, None]
    sel = torch.full((len(lens), 1, topk), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((len(lens), 1), -7, dtype=torch.int32, device="cuda")
    B.cobs_score_select(cfg, dev["q"], summ, dev["seq_lens"], sel, cnt, None, ws)
    out = torch.zeros((len(lens), G, D), dtype=torch.float32, device="cuda")
    sel_f, cnt_f = torch.full_like(sel, -7), torch.full_like(cnt, -7)
    B.cobs_decode_step(cfg, dev["q"], B.make_kv(dev), summ, out, None, sel_f, cnt_f, ws)
    assert B.cobs_read_status(ws) == 0
    sel, cnt, sel_f, cnt_f = sel.cpu(), cnt.cpu(), sel_f.cpu(), cnt_f.cpu()
    mean_np, f_np = mean_all.double().numpy(), f.double().numpy()
    for i, n_sum in enumerate(n_sums):
        n_cand = O.window_start(lens[i], wl.window, L) // L
        xi = np.broadcast_to(f_np[None], (n_sum, 2, D))
        e = O.log_mass_estimates(q[i].double().numpy(), mean_np[:n_sum], xi, L)
        score = O.group_scores(e)
        assert len(set(score.tolist())) <= 2                                    # two values, exactly
        ref = [int(x) for x in O.select_topk(score, n_cand, topk)]
        k = min(topk, n_cand)
        hot_c = [b for b in range(n_cand) if b % 16 == 0]
        cold_c = [b for b in range(n_cand) if b % 16 != 0]
        assert ref == sorted(hot_c[:k] + cold_c[:max(0, k - len(hot_c))])       # the oracle breaks ties by index
        assert int(cnt[i, 0]) == k and int(cnt_f[i, 0]) == k
        assert [int(x) for x in sel[i, 0, :k]] == ref, (n_sum, "cobs_score_select")
        assert [int(x) for x in sel_f[i, 0, :k]] == ref, (n_sum, "cobs_decode_step")
        assert all(int(x) == -1 for x in sel[i, 0, k:])


@pytest.mark.parametrize("key_model,planted", [("block_offset", 4), ("iid", 0)])
def test_adaptive_block_count_extension(key_model, planted):
    """cobs_score_select -> cobs_adaptive_trim -> cobs_sparse_decode against the oracle's adaptive_count /
    select_adaptive (an extension, not in the paper).  The count may differ from the oracle's only where the kept
    mass is within 5e-5 of the threshold (fp32 scores on the device, fp64 in the oracle): it must lie between the
    oracle's counts for tau +- 5e-5; the kept set is then checked with the usual tie band, and the attention output
    on the device's own trimmed selection against the oracle's attention over the same blocks."""
    B = _binding()
    L, topk, k_min = 64, 64, 3
    lens = [L * 96, L * 50 + 9, L * 3, L * 20 + 63]
    wl = synth.Workload("adapt", len(lens), 8, 2, 128, L * 96, L, 16, rank=4, topk=topk, window=130,
                        summary_dtype="bf16", key_model=key_model, planted=planted, shuffle_pages=True, seed=21,
                        seq_lens=lens)
    inp = synth.generate(wl)
    dev = to_dev(inp)
    cfg = B.make_config(wl)
    kv = B.make_kv(dev)
    summ = B.SummaryBuffers(cfg, "cuda")
    ws = B.alloc_workspace(cfg, "cuda")
    nb, hq, hkv, G, D = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.group, wl.head_dim
    ref = {}
    for b in range(nb):
        for h in range(hkv):
            st = oracle_unit_summaries(wl, inp, b, h)
            upload_unit_summaries(B, cfg, summ, b, h, st)
            ref[(b, h)] = oracle_unit_step(wl, inp, b, h, st)
    scores = torch.zeros((nb, hkv, wl.max_blocks), dtype=torch.float32, device="cuda")
    counts = []
    for tau in (0.5, 0.1, 0.01, 0.0):
        tau32 = float(np.float32(tau))
        sel = torch.full((nb, hkv, topk), -7, dtype=torch.int32, device="cuda")
        cnt = torch.full((nb, hkv), -7, dtype=torch.int32, device="cuda")
        B.cobs_score_select(cfg, dev["q"], summ, dev["seq_lens"], sel, cnt, scores, ws)
        B.cobs_adaptive_trim(cfg, scores, dev["seq_lens"], tau32, k_min, sel, cnt, ws)
        out = torch.zeros((nb, hq, D), dtype=torch.float32, device="cuda")
        lse = torch.zeros((nb, hq), dtype=torch.float32, device="cuda")
        B.cobs_sparse_decode(cfg, dev["q"], kv, sel, cnt, out, lse, ws)
        assert B.cobs_read_status(ws) == 0
        sel_c, cnt_c, out_c, lse_c = sel.cpu(), cnt.cpu(), out.cpu().numpy(), lse.cpu().numpy()
        for (b, h), r in ref.items():
            n_cand = O.window_start(lens[b], wl.window, L) // L
            k_gpu = int(cnt_c[b, h])
            k_lo = O.adaptive_count(r["score"], n_cand, min(tau32 + 5e-5, 1.0), k_min, topk)
            k_hi = O.adaptive_count(r["score"], n_cand, max(tau32 - 5e-5, 0.0), k_min, topk)
            assert k_lo <= k_gpu <= k_hi, (tau, b, h, k_gpu, k_lo, k_hi)
            gpu_sel = [int(x) for x in sel_c[b, h, :k_gpu]]
            assert all(int(x) == -1 for x in sel_c[b, h, k_gpu:])
            ok, msg, _ = check_selection(gpu_sel, r["score"], n_cand, k_gpu)
            assert ok, (tau, b, h, msg)
            ref_out, ref_lse = oracle_attend(wl, inp, b, h, gpu_sel)
            hs = slice(h * G, (h + 1) * G)
            assert np.all(out_rel_err(out_c[b, hs], ref_out) <= OUT_TOL), (tau, b, h)
            assert np.allclose(lse_c[b, hs], ref_lse, atol=2e-3, rtol=0)
            counts.append((tau, k_gpu, n_cand))
    # the rule does something: tau = 0 keeps everything it may, a large tau keeps fewer blocks where there are many
    assert all(k == min(topk, n) for t, k, n in counts if t == 0.0)
    assert any(k < min(topk, n) for t, k, n in counts if t == 0.5 and n > topk)
    if planted:
        # four planted blocks hold most of the mass: half of it needs only a few blocks
        assert all(k <= 8 for t, k, n in counts if t == 0.5 and n > topk)


@pytest.mark.parametrize("summary_dtype", ["bf16", "fp4"])
def test_diagonal_skew_variant_scores_and_step(summary_dtype):
    """The paper's diagonal-skew variant (Appendix, Cheap diagonal skew): with skew scalars given, scores carry the
    cubic term.  Oracle summaries and oracle skew scalars are uploaded bit for bit; scores, selection and the step's
    output are compared with the oracle's skew estimate."""
    B = _binding()
    L = 32
    lens = [L * 40, L * 23 + 5, L * 2]
    wl = synth.Workload("skew", len(lens), 8, 2, 64, L * 40, L, 16, rank=4, topk=6, window=70,
                        summary_dtype=summary_dtype, key_model="block_offset", planted=2, shuffle_pages=True, seed=9,
                        seq_lens=lens)
    inp = synth.generate(wl)
    dev = to_dev(inp)
    cfg = B.make_config(wl)
    kv = B.make_kv(dev)
    summ = B.SummaryBuffers(cfg, "cuda", skew=True)
    ws = B.alloc_workspace(cfg, "cuda")
    nb, hq, hkv, G, D = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.group, wl.head_dim
    ref, differs = {}, 0
    for b in range(nb):
        for h in range(hkv):
            st = oracle_unit_summaries(wl, inp, b, h)
            upload_unit_summaries(B, cfg, summ, b, h, st)
            K, _ = synth.unit_kv(inp, wl, b, h)
            n = st["mean"].shape[0]
            c = O.build_skew(K.numpy(), L, st["xi_exact"]).astype(np.float32)
            if n:
                summ.skew[b, h, :n] = torch.from_numpy(c).cuda()
            q = synth.unit_q(inp, wl, b, h).numpy()
            e = O.log_mass_estimates_skew(q, st["mean"], st["xi"], c.astype(np.float64), L)
            score = O.group_scores(e) if n else np.zeros(0)
            plain = O.group_scores(O.log_mass_estimates(q, st["mean"], st["xi"], L)) if n else np.zeros(0)
            differs += int(np.sum(np.abs(score - plain) > 1e-3 * np.maximum(plain, 1e-30)))
            ref[(b, h)] = score
    assert differs > 0                                            # the cubic term moves the scores
    sel = torch.full((nb, hkv, wl.topk), -7, dtype=torch.int32, device="cuda")
    cnt = torch.full((nb, hkv), -7, dtype=torch.int32, device="cuda")
    scores = torch.zeros((nb, hkv, wl.max_blocks), dtype=torch.float32, device="cuda")
    B.cobs_score_select(cfg, dev["q"], summ, dev["seq_lens"], sel, cnt, scores, ws)
    out = torch.zeros((nb, hq, D), dtype=torch.float32, device="cuda")
    lse = torch.zeros((nb, hq), dtype=torch.float32, device="cuda")
    sel_f, cnt_f = torch.full_like(sel, -7), torch.full_like(cnt, -7)
    B.cobs_decode_step(cfg, dev["q"], kv, summ, out, lse, sel_f, cnt_f, ws)
    assert B.cobs_read_status(ws) == 0
    sel, cnt, scores = sel.cpu(), cnt.cpu(), scores.cpu().double().numpy()
    out, lse, sel_f, cnt_f = out.cpu().numpy(), lse.cpu().numpy(), sel_f.cpu(), cnt_f.cpu()
    for (b, h), score in ref.items():
        n_sum = lens[b] // L
        n_cand = O.window_start(lens[b], wl.window, L) // L
        if n_sum:
            err = np.max(np.abs(scores[b, h, :n_sum] - score) / np.maximum(score, 1e-30))
            assert err <= SCORE_TOL, (b, h, err)
        ok, msg, _ = check_selection(sel[b, h].tolist(), score, n_cand, wl.topk)
        assert ok, (b, h, msg)
        assert torch.equal(sel_f[b, h], sel[b, h]) and int(cnt_f[b, h]) == int(cnt[b, h]) == min(wl.topk, n_cand)
        ref_out, ref_lse = oracle_attend(wl, inp, b, h, [int(x) for x in sel_f[b, h] if x >= 0])
        hs = slice(h * G, (h + 1) * G)
        assert np.all(out_rel_err(out[b, hs], ref_out) <= OUT_TOL), (b, h)
        assert np.allclose(lse[b, hs], ref_lse, atol=2e-3, rtol=0)


def test_builder_writes_skew_scalars():
    """cobs_build_summaries with a skew buffer (fp32 summaries): the scalars against the oracle's block_skew, directly
    where the factor's eigenvalue is well separated (elsewhere the eigenvector itself is not unique to rounding), and
    for every factor against block_skew evaluated on the factor the device stored."""
    B = _binding()
    L, D, r = 32, 64, 4
    wl = synth.Workload("skewb", 2, 4, 2, D, L * 12, L, 16, rank=r, topk=2, window=40, summary_dtype="fp32",
                        key_model="lowrank16", shuffle_pages=True, seed=17, seq_lens=[L * 12, L * 7 + 3])
    inp = synth.generate(wl)
    dev = to_dev(inp)
    cfg = B.make_config(wl)
    summ = B.SummaryBuffers(cfg, "cuda", skew=True)
    ws = B.alloc_workspace(cfg, "cuda")
    B.cobs_build_summaries(cfg, B.make_kv(dev), 0, wl.max_blocks, summ, ws)
    assert B.cobs_read_status(ws) == 0
    _, xi_v, _ = B.summary_views(cfg, summ)
    xi_gpu, skew_gpu = xi_v.cpu().double().numpy(), summ.skew.cpu().double().numpy()
    direct = 0
    for b in range(wl.batch):
        for h in range(wl.n_kv_heads):
            K, _ = synth.unit_kv(inp, wl, b, h)
            K = K.numpy()
            n = int(inp["seq_lens"][b]) // L
            _, xi, lam = O.build_summaries(K, L, r, n_blocks=n)
            c_ref = O.build_skew(K, L, xi)
            for blk in range(n):
                own = O.block_skew(K[blk * L:(blk + 1) * L], xi_gpu[b, h, blk])
                assert np.all(np.abs(skew_gpu[b, h, blk] - own) <= 2e-3 * np.maximum(1.0, np.abs(own))), (b, h, blk)
                for i in range(r):
                    gaps = [abs(lam[blk, i] - lam[blk, j]) for j in range(r) if j != i]
                    if lam[blk, i] > 0 and min(gaps) > 0.2 * lam[blk, i] and i < r - 1:
                        assert abs(skew_gpu[b, h, blk, i] - c_ref[blk, i]) <= 5e-3 * max(1.0, abs(c_ref[blk, i])), (b, h, blk, i)
                        direct += 1
    assert direct >= 20


def test_context_beyond_the_fused_selection_capacity():
    """4096 blocks per unit: more than the step kernel's selection team holds (2048), so scoring and selection
    take the generic kernels and only attention runs in the persistent kernel; same parity bar."""
    wl = synth.Workload("long", 1, 4, 1, 128, 4096 * 64, 64, 64, rank=4, topk=16, window=512, summary_dtype="fp4",
                        key_model="block_offset", planted=4, shuffle_pages=False, seed=41)
    run_stage_s(wl)


def test_rank_zero_is_first_order_mean_pool():
    wl = WL["cfg1_tiny"].replace(rank=0, summary_dtype="bf16")
    run_stage_s(wl)


def test_subspace_odd_dimension_bf16_and_fp32():
    for dt in ("bf16", "fp32"):
        wl = synth.Workload("sub", 1, 8, 2, 128, 64 * 24, 64, 64, rank=4, topk=6, window=128, summary_dtype=dt,
                            sub_dim=53, key_model="block_offset", query_model="spectrum", planted=2, seed=13)
        run_stage_s(wl)


def test_invalid_selection_is_reported_not_faulted():
    """An out-of-range block index is skipped by the kernel and surfaces as a status code."""
    B = _binding()
    wl = WL["cfg1_tiny"]
    inp = to_dev(synth.generate(wl))
    cfg = B.make_config(wl)
    ws = B.alloc_workspace(cfg, "cuda")
    sel = torch.tensor([[[0, 5, 31, 99]]], dtype=torch.int32, device="cuda")   # 31 lies in the window, 99 is outside
    cnt = torch.tensor([[4]], dtype=torch.int32, device="cuda")
    out = torch.zeros((1, 4, 64), dtype=torch.float32, device="cuda")
    B.cobs_sparse_decode(cfg, inp["q"], B.make_kv(inp), sel, cnt, out, None, ws)
    assert B.cobs_read_status(ws) == 6
    B.cobs_reset_status(ws)
    assert B.cobs_read_status(ws) == 0
    # the valid part of the request was still served: equals the oracle on blocks {0, 5}
    cpu = synth.generate(wl)
    o_ref, _ = oracle_attend(wl, cpu, 0, 0, [0, 5])
    assert np.all(out_rel_err(out[0].cpu().numpy(), o_ref) <= OUT_TOL)


def test_host_buffer_entry_point_matches_device_entry_point():
    B = _binding()
    wl = WL["cfg2_32k"].replace(seq_len=4096)
    cpu = synth.generate(wl)
    inp = to_dev(cpu)
    cfg = B.make_config(wl)
    summ = B.SummaryBuffers(cfg, "cuda")
    ws = B.alloc_workspace(cfg, "cuda")
    kv = B.make_kv(inp)
    B.cobs_build_summaries(cfg, kv, 0, wl.max_blocks, summ, ws)
    out_d = torch.zeros((1, 32, 128), dtype=torch.float32, device="cuda")
    sel_d = torch.zeros((1, 8, wl.topk), dtype=torch.int32, device="cuda")
    cnt_d = torch.zeros((1, 8), dtype=torch.int32, device="cuda")
    B.cobs_decode_step(cfg, inp["q"], kv, summ, out_d, None, sel_d, cnt_d, ws)
    q_h = cpu["q"].pin_memory()
    out_h = torch.zeros((1, 32, 128), dtype=torch.float32).pin_memory()
    sel_h = torch.zeros((1, 8, wl.topk), dtype=torch.int32).pin_memory()
    cnt_h = torch.zeros((1, 8), dtype=torch.int32).pin_memory()
    B.cobs_decode_step_host(cfg, q_h, kv, summ, out_h, sel_h, cnt_h, ws)
    assert torch.equal(out_h, out_d.cpu()) and torch.equal(sel_h, sel_d.cpu()) and torch.equal(cnt_h, cnt_d.cpu())
    # pinned output memory is written by the kernel itself; pageable memory goes through the staging buffer
    out_p = torch.zeros((1, 32, 128), dtype=torch.float32)
    assert not out_p.is_pinned()
    B.cobs_decode_step_host(cfg, q_h, kv, summ, out_p, None, None, ws)
    assert torch.equal(out_p, out_d.cpu())
    assert B.cobs_read_status(ws) == 0


# --- quantiser (bit exact) -----------------------------------------------------------------------------------

@pytest.mark.parametrize("scale_dtype", ["fp32", "fp16"])
@pytest.mark.parametrize("ds", [128, 85, 64])
def test_quantiser_bit_exact(scale_dtype, ds):
    B = _binding()
    wl = WL["cfg4_128k"].replace(sub_dim=0 if ds == 128 else ds, scale_dtype=scale_dtype, rank=4)
    cfg = B.make_config(wl)
    r = np.random.default_rng(ds)
    n = 4 * 300
    xi = (r.normal(size=(n, ds)) * np.exp(r.normal(size=(n, 1)) * 2)).astype(np.float32)
    grid = np.array([6, 0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, -0.25, -2.5, 0.0, -0.0, 5.999, 0.2499, 6.0], np.float32)
    xi[0, :len(grid)] = grid; xi[0, len(grid):] = 0
    xi[1] = 0.0
    xi[2] = 1e-30
    xi[3, :] = np.linspace(-6, 6, ds)
    codes_ref, scale_ref = O.quantise_e2m1(xi, scale_dtype)
    ds_pad = B.cobs_padded_sub_dim(cfg)
    codes = torch.full((n, ds_pad // 2), 0xEE, dtype=torch.uint8, device="cuda")
    scale = torch.zeros(n, dtype=torch.float16 if scale_dtype == "fp16" else torch.float32, device="cuda")
    B.cobs_quantise_xi(cfg, torch.from_numpy(xi).cuda(), codes, scale)
    got = B.unpack_fp4_rows(codes, ds_pad).cpu().numpy()
    assert np.array_equal(got[:, :ds], codes_ref)
    assert np.all(got[:, ds:] == 0)
    assert np.array_equal(scale.float().cpu().numpy(), scale_ref)


def test_e2m1_rounding_rule_agrees_with_the_hardware_conversion():
    """The oracle's E2M1 rounding (nearest, ties to the even mantissa bit, saturating at 6) against the GPU's own
    conversion instruction on a dense fp32 grid over [-6, 6], every tie point with both fp32 neighbours, and
    values beyond the range.  Every row holds a 6, so the oracle's scale is exactly 1 and t = x."""
    B = _binding()
    ties = np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0], np.float32)
    near = np.concatenate([ties, np.nextafter(ties, np.float32(0)), np.nextafter(ties, np.float32(10))])
    special = np.concatenate([near, -near, np.array([0.0, 0.5, 1, 1.5, 2, 3, 4, 6, -0.5, -1, -1.5, -2, -3, -4, -6,
                                                      1e-30, 1e-45, 0.2499999, 5.9999995], np.float32)])
    dense = np.linspace(-6.0, 6.0, 400001).astype(np.float32)
    rnd = (np.random.default_rng(0).uniform(-6, 6, 200000)).astype(np.float32)
    vals = np.concatenate([special, dense, rnd])
    cols = 127
    vals = np.concatenate([vals, np.zeros((-len(vals)) % cols, np.float32)]).reshape(-1, cols)
    rows = np.concatenate([np.full((vals.shape[0], 1), 6.0, np.float32), vals], axis=1)     # max |x| = 6 -> scale 1
    codes_ref, scale_ref = O.quantise_e2m1(rows, "fp32")
    assert np.all(scale_ref == 1.0)
    x = torch.from_numpy(rows.reshape(-1)).cuda()
    hw = torch.zeros(x.numel(), dtype=torch.uint8, device="cuda")
    B.cobs_hw_e2m1_codes(x, hw)
    hw = hw.cpu().numpy().reshape(rows.shape)
    assert np.array_equal(hw & 7, codes_ref & 7)                  # the magnitude index, everywhere
    nz = (codes_ref & 7) != 0
    assert np.array_equal(hw[nz] >> 3, codes_ref[nz] >> 3)        # the sign wherever the value is not zero
    # beyond the largest magnitude the conversion saturates, as the oracle's last threshold does (t > 5 -> 6)
    big = torch.tensor([6.5, 7.0, 100.0, 3e38, -6.5, -7.0, -1e9], dtype=torch.float32, device="cuda")
    hb = torch.zeros(big.numel(), dtype=torch.uint8, device="cuda")
    B.cobs_hw_e2m1_codes(big, hb)
    assert hb.cpu().tolist() == [7, 7, 7, 7, 15, 15, 15]
    # codes that are zero in magnitude: +0 and tiny positives give code 0 on both sides.  Negative values that
    # round to zero keep their sign bit in the oracle's rule (code 8, which decodes to the same 0)
    zero_neg = torch.tensor([-0.0, -1e-30, -0.2], dtype=torch.float32, device="cuda")
    hz = torch.zeros(3, dtype=torch.uint8, device="cuda")
    B.cobs_hw_e2m1_codes(zero_neg, hz)
    assert all(int(c) & 7 == 0 for c in hz.cpu().tolist())


@pytest.mark.parametrize("topk", [16, 64])
@pytest.mark.parametrize("G", [1, 2, 4, 8])
def test_selection_with_few_heavy_blocks_over_a_flat_background(G, topk):
    """Units of 513 ... 1024 summarised blocks whose scores are a handful of heavy blocks over a nearly uniform
    background: at some bisection round of the top-k more than 512 keys lie above the lowest trial value while
    fewer than k lie above the others (the case in which a packed count once overflowed its field).  Selection
    against the oracle, and nothing may be written outside a unit's own row of sel_idx (guard rows)."""
    B = _binding()
    L, D, NB = 16, 64, 1024
    n_sums = [600, 1023, 1024, 513, 512, 700]
    lens = [n * L + (3 if n < NB else 0) for n in n_sums]
    wl = synth.Workload("flat", len(lens), G, 1, D, NB * L, L, 16, rank=2, topk=topk, window=L + 5, summary_dtype="bf16",
                        key_model="iid", seed=31 + G, seq_lens=lens)
    inp = synth.generate(wl)
    gen = torch.Generator().manual_seed(100 + G)
    v = torch.randn(D, generator=gen)
    inp["q"] = (v[None, None, :] + 0.2 * torch.randn(len(lens), G, D, generator=gen)).to(torch.bfloat16)
    dev = to_dev(inp)
    cfg = B.make_config(wl)
    summ = B.SummaryBuffers(cfg, "cuda")
    ws = B.alloc_workspace(cfg, "cuda")
    mean_v, xi_v, _ = B.summary_views(cfg, summ)
    # background: means -0.3 v plus a little noise (scores within a few per cent of each other); 4 heavy blocks
    mean_all = (-0.3 * v[None, None, :] + 0.004 * torch.randn(len(lens), NB, D, generator=gen))
    heavy = [[int(x) for x in torch.randperm(n - 4, generator=gen)[:4]] for n in n_sums]
    for i, hb in enumerate(heavy):
        mean_all[i, hb] = 0.6 * v
    mean_bf = mean_all.to(torch.bfloat16)
    xi_bf = (0.05 * torch.randn(len(lens), NB, 2, D, generator=gen)).to(torch.bfloat16)
    mean_v[:, 0] = mean_bf.cuda()
    xi_v[:, 0] = xi_bf.cuda()
    guard = torch.full((len(lens) + 2, topk), -7, dtype=torch.int32, device="cuda")
    sel = guard[1:-1].view(len(lens), 1, topk)
    cnt = torch.full((len(lens), 1), -7, dtype=torch.int32, device="cuda")
    B.cobs_score_select(cfg, dev["q"], summ, dev["seq_lens"], sel, cnt, None, ws)
    guard_f = torch.full_like(guard, -7)
    sel_f = guard_f[1:-1].view(len(lens), 1, topk)
    cnt_f = torch.full_like(cnt, -7)
    out = torch.zeros((len(lens), G, D), dtype=torch.float32, device="cuda")
    B.cobs_decode_step(cfg, dev["q"], B.make_kv(dev), summ, out, None, sel_f, cnt_f, ws)
    assert B.cobs_read_status(ws) == 0
    for g_ in (guard, guard_f):
        assert torch.all(g_[0] == -7) and torch.all(g_[-1] == -7)
    sel_c, sel_fc = sel.cpu(), sel_f.cpu()
    for i, n_sum in enumerate(n_sums):
        n_cand = O.window_start(lens[i], wl.window, L) // L
        e = O.log_mass_estimates(inp["q"][i].double().numpy(), mean_bf[i, :n_sum].double().numpy(),
                                 xi_bf[i, :n_sum].double().numpy(), L)
        score = O.group_scores(e)
        ref = set(int(x) for x in O.select_topk(score, n_cand, topk))
        assert set(heavy[i]) <= ref                               # the heavy blocks are the top of the list
        for which, got in (("cobs_score_select", sel_c[i, 0]), ("cobs_decode_step", sel_fc[i, 0])):
            ok, msg, _ = check_selection(got.tolist(), score, n_cand, topk)
            assert ok, (which, n_sum, msg)


def test_length_beyond_the_page_table_is_reported_not_followed():
    """T = NB * L + L - 1 with a page table that covers exactly NB * L tokens: the window's last tokens have no
    page-table entry.  The kernel must not read past the row: it skips them and leaves COBS_ERR_BOUNDS."""
    B = _binding()
    wl = WL["cfg1_tiny"].replace(summary_dtype="bf16")
    assert wl.max_pages_per_seq * wl.page_size == wl.max_blocks * wl.block_size
    cpu = synth.generate(wl)
    inp = to_dev(cpu)
    cfg = B.make_config(wl)
    summ = B.SummaryBuffers(cfg, "cuda")
    ws = B.alloc_workspace(cfg, "cuda")
    kv = B.make_kv(inp)
    B.cobs_build_summaries(cfg, kv, 0, wl.max_blocks, summ, ws)
    # the page table is the last thing in its allocation's row: put a poisoned row behind it
    table = torch.full((wl.batch + 1, wl.max_pages_per_seq), 2 ** 30, dtype=torch.int32, device="cuda")
    table[:wl.batch] = inp["page_table"]
    inp["page_table"] = table[:wl.batch]
    kv = B.make_kv(inp)
    inp["seq_lens"].fill_(wl.max_blocks * wl.block_size + wl.block_size - 1)
    out = torch.zeros((wl.batch, wl.n_q_heads, wl.head_dim), dtype=torch.float32, device="cuda")
    B.cobs_decode_step(cfg, inp["q"], kv, summ, out, None, None, None, ws)
    assert B.cobs_read_status(ws) == 6
    B.cobs_reset_status(ws)
    # the tokens that do have a page were served: same result as the full-capacity length, whose window is those tokens
    assert torch.isfinite(out).all()
    inp["seq_lens"].fill_(wl.max_blocks * wl.block_size)
    out2 = torch.zeros_like(out)
    B.cobs_decode_step(cfg, inp["q"], kv, summ, out2, None, None, None, ws)
    assert B.cobs_read_status(ws) == 0


def test_one_workspace_serves_calls_of_different_shapes():
    """A workspace as large as the largest of three shapes needs, used by their steps in a mixed order: every step
    gives the bits it gives on a workspace of its own (the hand-off counters of the persistent kernel live at the same
    places for every shape, and each launch clears what the previous one left, however many units that one had)."""
    B = _binding()

    def setup(wl):
        inp = to_dev(synth.generate(wl))
        cfg = B.make_config(wl)
        kv = B.make_kv(inp)
        summ = B.SummaryBuffers(cfg, "cuda")
        own = B.alloc_workspace(cfg, "cuda")
        B.cobs_build_summaries(cfg, kv, 0, wl.max_blocks, summ, own)
        nb, hq, hkv, D = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim
        x = dict(wl=wl, inp=inp, cfg=cfg, kv=kv, summ=summ,
                 out=torch.zeros((nb, hq, D), dtype=torch.float32, device="cuda"),
                 lse=torch.zeros((nb, hq), dtype=torch.float32, device="cuda"),
                 sel=torch.zeros((nb, hkv, wl.topk), dtype=torch.int32, device="cuda"),
                 cnt=torch.zeros((nb, hkv), dtype=torch.int32, device="cuda"))
        B.cobs_decode_step(cfg, inp["q"], kv, summ, x["out"], x["lse"], x["sel"], x["cnt"], own)
        torch.cuda.synchronize()
        x["ref_out"], x["ref_sel"] = x["out"].clone(), x["sel"].clone()
        return x

    a = setup(WL["cfg2_32k"].replace(seq_len=8192, batch=4))                      # 32 units
    b = setup(WL["cfg2_32k"].replace(seq_len=4096, batch=1))                      # 8 units
    c = setup(WL["cfg4_128k"].replace(seq_len=4096, batch=9))                     # 72 units, another descriptor
    size = max(B.cobs_workspace_bytes(x["cfg"]) for x in (a, b, c))
    raw = torch.zeros(size + 256, dtype=torch.uint8, device="cuda")
    off = (-raw.data_ptr()) % 256
    ws = raw[off:off + size]
    B.cobs_reset_status(ws)
    for x in (a, b, c, a, a, c, b, b, a, c, b, a):
        x["out"].zero_(); x["sel"].zero_()
        B.cobs_decode_step(x["cfg"], x["inp"]["q"], x["kv"], x["summ"], x["out"], x["lse"], x["sel"], x["cnt"], ws)
        torch.cuda.synchronize()
        assert torch.equal(x["out"], x["ref_out"]) and torch.equal(x["sel"], x["ref_sel"])
        assert B.cobs_read_status(ws) == 0


def test_step_replays_from_a_cuda_graph():
    """The fused step captured once and replayed: its hand-off counters alternate between two sets by themselves
    (no host state), so odd and even replays give the bits of a plain call; the status word stays clear."""
    B = _binding()
    wl = WL["cfg2_32k"].replace(seq_len=8192)
    inp = to_dev(synth.generate(wl))
    cfg = B.make_config(wl)
    kv = B.make_kv(inp)
    summ = B.SummaryBuffers(cfg, "cuda")
    ws = B.alloc_workspace(cfg, "cuda")
    B.cobs_build_summaries(cfg, kv, 0, wl.max_blocks, summ, ws)
    nb, hq, hkv, D = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim
    out = torch.zeros((nb, hq, D), dtype=torch.float32, device="cuda")
    lse = torch.zeros((nb, hq), dtype=torch.float32, device="cuda")
    sel = torch.zeros((nb, hkv, wl.topk), dtype=torch.int32, device="cuda")
    cnt = torch.zeros((nb, hkv), dtype=torch.int32, device="cuda")
    B.cobs_decode_step(cfg, inp["q"], kv, summ, out, lse, sel, cnt, ws)
    torch.cuda.synchronize()
    ref_out, ref_sel, ref_lse = out.clone(), sel.clone(), lse.clone()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        B.cobs_decode_step(cfg, inp["q"], kv, summ, out, lse, sel, cnt, ws)
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=side):
            B.cobs_decode_step(cfg, inp["q"], kv, summ, out, lse, sel, cnt, ws)
    for _ in range(5):
        out.zero_(); sel.zero_(); lse.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, ref_out) and torch.equal(sel, ref_sel) and torch.equal(lse, ref_lse)
    # and a plain call after the replays
    out.zero_()
    B.cobs_decode_step(cfg, inp["q"], kv, summ, out, lse, sel, cnt, ws)
    torch.cuda.synchronize()
    assert torch.equal(out, ref_out)
    assert B.cobs_read_status(ws) == 0


# --- builder (backward error; eigenvectors of close eigenvalues are not unique to rounding) ---------------------

def check_builder(wl, units):
    B = _binding()
    cpu = synth.generate(wl)
    inp = to_dev(cpu)
    cfg32 = B.make_config(wl.replace(summary_dtype="fp32"))
    s32 = B.SummaryBuffers(cfg32, "cuda", inp.get("u_q"))
    ws = B.alloc_workspace(cfg32, "cuda")
    kv = B.make_kv(inp)
    B.cobs_build_summaries(cfg32, kv, 0, wl.max_blocks, s32, ws)
    assert B.cobs_read_status(ws) == 0
    mean32, xi32, _ = B.summary_views(cfg32, s32)
    # determinism: a second build gives the same bits
    s32b = B.SummaryBuffers(cfg32, "cuda", inp.get("u_q"))
    B.cobs_build_summaries(cfg32, kv, 0, wl.max_blocks, s32b, ws)
    assert torch.equal(s32.xi, s32b.xi) and torch.equal(s32.mean, s32b.mean)

    r, L = wl.rank, wl.block_size
    for (b, h) in units:
        K, _ = synth.unit_kv(cpu, wl, b, h)
        K = K.numpy()
        u_q = cpu["u_q"][h].double().numpy() if wl.sub_dim else None
        q = synth.unit_q(cpu, wl, b, h).numpy()
        qt = O.scale_query(q) if u_q is None else O.scale_query(q) @ u_q
        n_sum = int(cpu["seq_lens"][b]) // L
        xi_g = xi32[b, h, :n_sum].double().cpu().numpy()
        mean_g = mean32[b, h, :n_sum].double().cpu().numpy()
        for blk in range(n_sum):
            kb = K[blk * L:(blk + 1) * L]
            kbar, sigma = O.block_mean_and_covariance(kb)
            if u_q is not None:
                sigma = u_q.T @ sigma @ u_q
            lam = np.sort(np.linalg.eigvalsh(sigma))[::-1]
            lam0 = lam[0]
            assert np.max(np.abs(mean_g[blk] - kbar)) <= 1e-6 * max(1.0, np.max(np.abs(kbar)))
            x = xi_g[blk]
            for i in range(r):
                n2 = x[i] @ x[i]
                assert abs(n2 - lam[i]) <= 2e-5 * lam0, (b, h, blk, i, n2, lam[i])
                resid = np.linalg.norm(sigma @ x[i] - n2 * x[i])
                assert resid <= 1e-4 * lam0 * np.sqrt(n2), (b, h, blk, i, resid)
                j = int(np.argmax(np.abs(x[i])))
                assert x[i, j] > 0
                for k2 in range(i):
                    assert abs(x[i] @ x[k2]) <= 1e-4 * np.sqrt(n2 * (x[k2] @ x[k2]))
            # the quadratic form the scorer will see
            for g in range(q.shape[0]):
                got = sum((x[i] @ qt[g]) ** 2 for i in range(r))
                _, xr, _ = O.scaled_eigenvectors_gram(kb, r, u_q)
                want = sum((xr[i] @ qt[g]) ** 2 for i in range(r))
                slack = 1e-4 * lam0 * (qt[g] @ qt[g]) + (lam[r - 1] - lam[r] if (lam[r - 1] - lam[r]) < 1e-3 * lam0 else 0) * (qt[g] @ qt[g])
                assert abs(got - want) <= slack, (b, h, blk, g, got, want)

    # storage formats: the device's bf16 / FP4 outputs are its own fp32 factors pushed through the
    # storage rounding (bf16: RNE; FP4: the quantiser, itself bit-exact against the oracle elsewhere)
    if wl.summary_dtype != "fp32":
        cfg = B.make_config(wl)
        s = B.SummaryBuffers(cfg, "cuda", inp.get("u_q"))
        B.cobs_build_summaries(cfg, kv, 0, wl.max_blocks, s, ws)
        mean_s, xi_s, scale_s = B.summary_views(cfg, s)
        assert torch.equal(mean_s, mean32.to(torch.bfloat16))
        if wl.summary_dtype == "bf16":
            assert torch.equal(xi_s, xi32.to(torch.bfloat16))
        else:
            ds = wl.sub_dim or wl.head_dim
            flat = xi32.reshape(-1, ds).contiguous()
            codes = torch.zeros((flat.shape[0], xi_s.shape[-1]), dtype=torch.uint8, device="cuda")
            scale = torch.zeros(flat.shape[0], dtype=scale_s.dtype, device="cuda")
            B.cobs_quantise_xi(cfg, flat, codes, scale)
            assert torch.equal(codes.view_as(xi_s), xi_s) and torch.equal(scale.view_as(scale_s), scale_s)
            # and the ORACLE's quantiser applied to the device's fp32 factors gives the device's codes and scales,
            # bit for bit (the builder's own FP4 output against the paper-side definition of the format)
            codes_ref, scale_ref = O.quantise_e2m1(flat.cpu().numpy(), wl.scale_dtype)
            ds_pad = B.cobs_padded_sub_dim(cfg)
            got = B.unpack_fp4_rows(xi_s.reshape(-1, ds_pad // 2), ds_pad).cpu().numpy()
            assert np.array_equal(got[:, :ds], codes_ref)
            assert np.all(got[:, ds:] == 0)
            assert np.array_equal(scale_s.reshape(-1).float().cpu().numpy(), scale_ref)
    assert B.cobs_read_status(ws) == 0


def test_builder_cfg1_fp32():
    check_builder(WL["cfg1_tiny"], [(0, 0)])


def test_builder_cfg2_like_bf16():
    check_builder(WL["cfg2_32k"].replace(seq_len=4096), [(0, 0), (0, 7)])


def test_builder_cfg4_like_fp4_paged():
    check_builder(WL["cfg4_128k"].replace(batch=2, seq_len=4096), [(0, 1), (1, 6)])


def test_builder_cfg3a_like_subspace():
    check_builder(WL["cfg3a_32k_subspace"].replace(batch=1, seq_len=2048), [(0, 2)])


def test_builder_cfg5_like_block128():
    check_builder(WL["cfg5_64k_g8"].replace(batch=1, seq_len=4096), [(0, 4)])


@pytest.mark.parametrize("case", ["cfg1_tiny", "cfg4_like", "cfg5_like", "subspace"])
def test_builder_jacobi_route(case, monkeypatch):
    """The builder's second eigen-solver (taken by a block whose tridiagonal route fails its residual check), forced
    for every block: the same checks against the oracle's definitions."""
    monkeypatch.setenv("COBS_BUILD_SOLVER", "jacobi")
    if case == "cfg1_tiny":
        check_builder(WL["cfg1_tiny"], [(0, 0)])
    elif case == "cfg4_like":
        check_builder(WL["cfg4_128k"].replace(batch=1, seq_len=2048), [(0, 3)])
    elif case == "cfg5_like":
        check_builder(WL["cfg5_64k_g8"].replace(batch=1, seq_len=2048), [(0, 4)])
    else:
        check_builder(WL["cfg3a_32k_subspace"].replace(batch=1, seq_len=1024), [(0, 2)])


@pytest.mark.parametrize("solver", ["tridiagonal", "jacobi"])
@pytest.mark.parametrize("rank,L,D", [(12, 64, 128), (16, 128, 64), (15, 32, 64)])
def test_builder_ranks_above_eight(rank, L, D, solver, monkeypatch):
    """More factors than the builder has warps: two eigenvectors per warp in the inverse iteration."""
    if solver == "jacobi":
        monkeypatch.setenv("COBS_BUILD_SOLVER", "jacobi")
    wl = synth.Workload("highrank", 1, 4, 2, D, 6 * L, L, 16, rank=rank, topk=2, window=L, summary_dtype="fp32",
                        key_model="block_offset", planted=1, shuffle_pages=True, seed=21)
    check_builder(wl, [(0, 0), (0, 1)])


@pytest.mark.parametrize("solver", ["tridiagonal", "jacobi"])
@pytest.mark.parametrize("L", [16, 32, 64, 128])
def test_builder_structured_spectra(L, solver, monkeypatch):
    """Blocks whose Gram matrices are not generic: rank one, two equal leading eigenvalues, a few distinct tokens
    repeated (a reducible tridiagonal form), a spectrum of well separated and of nearly equal eigenvalues, tokens
    equal in pairs.  Errors are measured against the largest eigenvalue (backward error): factors of numerically
    null directions are rounding noise in fp32 and exact zeros in the oracle's fp64."""
    if solver == "jacobi":
        monkeypatch.setenv("COBS_BUILD_SOLVER", "jacobi")
    B = _binding()
    D, r, nblk = 64, 4, 6
    wl = WL["cfg1_tiny"].replace(block_size=L, page_size=16, seq_len=nblk * L, window=L, topk=2, rank=r)
    cpu = synth.generate(wl)
    g = torch.Generator().manual_seed(1234 + L)
    blocks = []
    u = torch.linalg.qr(torch.randn(D, D, generator=g))[0]                       # orthonormal directions
    t = torch.randn(L, generator=g)
    blocks.append(1.5 + t[:, None] * u[:, 0][None, :] * 2.0)                     # rank one
    a = torch.linalg.qr(torch.randn(L, 2, generator=g) - 0.0)[0]
    a = a - a.mean(0, keepdim=True)
    a = torch.linalg.qr(a)[0] * (L ** 0.5)
    blocks.append(a[:, :1] * u[:, 1][None, :] + a[:, 1:2] * u[:, 2][None, :] + 0.01 * torch.randn(L, D, generator=g))  # two equal
    few = torch.randn(3, D, generator=g)
    blocks.append(few[torch.arange(L) % 3])                                      # three distinct tokens
    sv = torch.tensor([4.0, 2.0, 1.0, 0.5] + [0.01] * (D - 4))
    blocks.append(torch.randn(L, D, generator=g) @ (u * sv[None, :]).T)          # separated
    sv = torch.tensor([1.0, 0.9999, 0.9998, 0.5, 0.4999] + [0.05] * (D - 5))
    blocks.append(torch.randn(L, D, generator=g) @ (u * sv[None, :]).T)          # nearly equal
    half = torch.randn(L // 2, D, generator=g)
    blocks.append(half.repeat_interleave(2, dim=0))                              # tokens equal in pairs
    kp = cpu["k_pages"]                                                          # [n_pages][Hkv][P][D]
    assert kp.shape[1] == 1 and kp.shape[3] == D
    ppb = L // wl.page_size
    for i, blk in enumerate(blocks):
        pages = cpu["page_table"][0, i * ppb:(i + 1) * ppb].long()
        kp[pages, 0] = blk.to(torch.bfloat16).reshape(ppb, wl.page_size, D)
    inp = to_dev(cpu)
    cfg = B.make_config(wl)
    s = B.SummaryBuffers(cfg, "cuda")
    ws = B.alloc_workspace(cfg, "cuda")
    B.cobs_build_summaries(cfg, B.make_kv(inp), 0, wl.max_blocks, s, ws)
    assert B.cobs_read_status(ws) == 0
    _, xi, _ = B.summary_views(cfg, s)
    K, _ = synth.unit_kv(cpu, wl, 0, 0)
    K = K.numpy()
    for i in range(nblk):
        kb = K[i * L:(i + 1) * L]
        _, sigma = O.block_mean_and_covariance(kb)
        lam = np.sort(np.linalg.eigvalsh(sigma))[::-1]
        lam0 = lam[0]
        x = xi[0, 0, i].double().cpu().numpy()
        for f in range(r):
            n2 = x[f] @ x[f]
            assert abs(n2 - lam[f]) <= 2e-5 * lam0, (i, f, n2, lam[f])
            assert np.linalg.norm(sigma @ x[f] - n2 * x[f]) <= 1e-4 * lam0 * np.sqrt(lam0), (i, f)
            for f2 in range(f):
                assert abs(x[f] @ x[f2]) <= 1e-4 * lam0, (i, f, f2)
        # the rank-r approximation the scorer uses, as a matrix
        approx = x.T @ x
        w, v = np.linalg.eigh(sigma)
        want = (v[:, -r:] * w[-r:]) @ v[:, -r:].T
        gap = lam[r - 1] - lam[r]
        slack = 2e-4 * lam0 + (gap if gap < 1e-3 * lam0 else 0.0)
        assert np.linalg.norm(approx - want, 2) <= slack, (i, np.linalg.norm(approx - want, 2), slack)


def test_builder_constant_key_block_gives_zero_factors():
    B = _binding()
    wl = WL["cfg1_tiny"].replace(summary_dtype="fp4")
    inp = to_dev(synth.generate(wl))
    inp["k_pages"][3] = inp["k_pages"][3, :, :1, :]          # every key of block 3 equal
    cfg = B.make_config(wl)
    s = B.SummaryBuffers(cfg, "cuda")
    ws = B.alloc_workspace(cfg, "cuda")
    B.cobs_build_summaries(cfg, B.make_kv(inp), 0, wl.max_blocks, s, ws)
    mean, xi, scale = B.summary_views(cfg, s)
    assert torch.all(xi[0, 0, 3] == 0) and torch.all(scale[0, 0, 3] == 0)
    assert torch.equal(mean[0, 0, 3], inp["k_pages"][3, 0, 0])
    assert torch.any(xi[0, 0, 2] != 0)
