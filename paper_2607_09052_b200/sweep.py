"""Variants of the descriptor on one shape, through the same kernels: rank 0 (mean-pool score), 4, 6, 8; full key
space or a query subspace of several widths; bf16 or FP4 factors (the paper's ablation axes: Table "bandwidth",
Table "quant", the per-layer subspace widths, and the appendix's diagonal-skew variant).  For every variant: the record bytes per block and KV head, the
algorithmic bytes of a decode step, the measured step time on the GPU, and the recall of its selection against the
exact-mass selector (cobs_exact_select, the paper's OSA reference).  Prints a markdown table.

    python -m paper_2607_09052_b200.sweep [--batch 4] [--steps 30]

Each variant also checks that the fused step selects exactly what cobs_score_select selects."""

from __future__ import annotations

import argparse

import torch

from . import binding as B
from . import synth


def algorithmic_bytes(wl: synth.Workload, record: int) -> int:
    L, D = wl.block_size, wl.head_dim
    total = 0
    for t in wl.lens():
        n_sum = t // L
        ws = (max(0, t - wl.window) // L) * L
        n_cand = ws // L
        toks = min(wl.topk, n_cand) * L + (t - ws)
        total += wl.n_kv_heads * (n_sum * record + toks * 2 * D * 2)
    total += wl.batch * wl.n_q_heads * D * (2 + 4)
    if wl.sub_dim:
        total += wl.n_kv_heads * D * wl.sub_dim * 4
    return total


def time_variant(wl: synth.Workload, steps: int, skew: bool = False):
    dev = "cuda"
    inp = synth.generate(wl, dev)
    cfg = B.make_config(wl)
    kv = B.make_kv(inp)
    summ = B.SummaryBuffers(cfg, dev, inp.get("u_q"), skew=skew)
    ws = B.alloc_workspace(cfg, dev)
    B.cobs_build_summaries(cfg, kv, 0, wl.max_blocks, summ, ws)
    nb, hq, hkv, D = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim
    out = torch.zeros((nb, hq, D), dtype=torch.float32, device=dev)
    sel = torch.zeros((nb, hkv, wl.topk), dtype=torch.int32, device=dev)
    cnt = torch.zeros((nb, hkv), dtype=torch.int32, device=dev)
    sel2, cnt2 = torch.zeros_like(sel), torch.zeros_like(cnt)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    B.cobs_score_select(cfg, inp["q"], summ, inp["seq_lens"], sel2, cnt2, None, ws)
    for _ in range(3):
        B.cobs_decode_step(cfg, inp["q"], kv, summ, out, None, sel, cnt, ws)
    torch.cuda.synchronize()
    if B.cobs_read_status(ws) != 0 or not (torch.equal(sel, sel2) and torch.equal(cnt, cnt2)):
        raise RuntimeError(f"{wl.name}: fused step and cobs_score_select disagree")
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in evs:
        flush.zero_()                                  # the L2 holds nothing of the step when it starts
        a.record()
        B.cobs_decode_step(cfg, inp["q"], kv, summ, out, None, sel, cnt, ws)
        b.record()
    torch.cuda.synchronize()
    us = sorted(a.elapsed_time(b) * 1e3 for a, b in evs)[len(evs) // 2]
    mb, xb, sb = B.cobs_summary_bytes(cfg)
    record = (mb + xb + sb) // (nb * hkv * wl.max_blocks) + (4 * wl.rank if skew else 0)
    # recall of the estimator's selection against the exact-mass selector (the paper's OSA reference)
    sel_x, cnt_x = torch.zeros_like(sel), torch.zeros_like(cnt)
    B.cobs_exact_select(cfg, inp["q"], kv, sel_x, cnt_x, None, ws)
    torch.cuda.synchronize()
    hits = total = 0
    for a, b in zip(sel.cpu().reshape(-1, wl.topk).tolist(), sel_x.cpu().reshape(-1, wl.topk).tolist()):
        want = {x for x in b if x >= 0}
        hits += len(want & {x for x in a if x >= 0})
        total += len(want)
    return record, algorithmic_bytes(wl, record), us, hits / max(total, 1)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=4)
    ap.add_argument("--steps", type=int, default=30)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("the sweep times CUDA kernels: no GPU here")
    base = synth.named_workloads()["cfg3a_32k_subspace"].replace(batch=args.batch)
    variants = []
    for dtype in ("bf16", "fp4"):
        for rank in (0, 4, 6, 8):
            variants.append((f"full space, r={rank}, {dtype}", base.replace(sub_dim=0, query_model="iid", rank=rank,
                                                                            summary_dtype=dtype)))
    for s in (42, 56, 71, 85, 108):
        variants.append((f"subspace s={s}, r=4, fp4", base.replace(sub_dim=s, rank=4, summary_dtype="fp4")))
    variants.append(("subspace s=85, r=4, bf16", base.replace(sub_dim=85, rank=4, summary_dtype="bf16")))
    # the diagonal-skew variant (Appendix, Cheap diagonal skew): r more scalars per block, scored by the generic kernels
    skewed = [(f"full space, r={rank}, bf16 + skew", base.replace(sub_dim=0, query_model="iid", rank=rank,
                                                                  summary_dtype="bf16")) for rank in (4, 8)]
    print(f"shape: B={base.batch}, {base.n_q_heads} query / {base.n_kv_heads} KV heads, D={base.head_dim}, "
          f"T={base.seq_len}, L={base.block_size}, k={base.topk}, W={base.window}")
    print("| descriptor | record B / block / KV head | algorithmic MiB / step | step (median, us) | GB/s | "
          "recall of the exact-mass top-k |")
    print("|---|---|---|---|---|---|")
    for label, wl in variants + skewed:
        record, nbytes, us, recall = time_variant(wl.replace(name=label), args.steps, skew=(label, wl) in skewed)
        print(f"| {label} | {record} | {nbytes / 2**20:.1f} | {us:.1f} | {nbytes / us / 1e3:.0f} | {recall:.3f} |")


if __name__ == "__main__":
    main()
