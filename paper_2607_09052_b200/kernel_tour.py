"""One call of every entry point of the library on a small paged workload.

    python -m paper_2607_09052_b200.kernel_tour [--batch 4] [--context 32768]

A usage example of the whole API in order (build the summaries, score and select, attend, the fused step, the
exact-mass selector, the adaptive trim, appending a token, the host-buffer step), and the command the per-kernel
launch lists under profiles/ are taken from: every kernel of the library runs at least once here.  Prints one line
per call with its device time (CUDA events).  Needs a CUDA device; there is no CPU fallback.
"""

from __future__ import annotations

import argparse
import os

import torch

from . import binding as B
from . import build as build_mod
from . import synth


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=4)
    ap.add_argument("--context", type=int, default=32768)
    args = ap.parse_args()
    build_mod.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    stream = torch.cuda.current_stream()

    def timed(name, fn):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record(stream)
        fn()
        b.record(stream)
        torch.cuda.synchronize()
        print(f"{name:58s} {a.elapsed_time(b) * 1e3:10.1f} us")

    base = synth.named_workloads()["cfg4_128k"].replace(batch=args.batch, seq_len=args.context)
    variants = [
        ("packed E2M1, rank 8 (step kernel scores)", base),
        ("bf16, rank 4 (step kernel scores)", base.replace(summary_dtype="bf16", rank=4)),
        ("fp32, rank 4 (generic scoring + selection kernels)", base.replace(summary_dtype="fp32", rank=4)),
        ("packed E2M1 subspace 85, rank 4 (projection prologue)", base.replace(sub_dim=85, rank=4, query_model="spectrum")),
    ]
    for label, wl in variants:
        print(f"--- {label}: {wl.batch} x {wl.seq_len} tokens, {wl.n_q_heads}/{wl.n_kv_heads} heads, top-{wl.topk}")
        inp = synth.generate(wl, dev)
        cfg = B.make_config(wl)
        kv = B.make_kv(inp)
        summ = B.SummaryBuffers(cfg, dev, inp.get("u_q"))
        ws = B.alloc_workspace(cfg, dev)
        nb, hq, hkv, D = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim
        out = torch.zeros((nb, hq, D), dtype=torch.float32, device=dev)
        lse = torch.zeros((nb, hq), dtype=torch.float32, device=dev)
        sel = torch.zeros((nb, hkv, wl.topk), dtype=torch.int32, device=dev)
        cnt = torch.zeros((nb, hkv), dtype=torch.int32, device=dev)
        scores = torch.zeros((nb, hkv, wl.max_blocks), dtype=torch.float32, device=dev)
        timed("cobs_build_summaries (every block)", lambda: B.cobs_build_summaries(cfg, kv, 0, wl.max_blocks, summ, ws))
        timed("cobs_score_select", lambda: B.cobs_score_select(cfg, inp["q"], summ, inp["seq_lens"], sel, cnt, scores, ws))
        timed("cobs_sparse_decode", lambda: B.cobs_sparse_decode(cfg, inp["q"], kv, sel, cnt, out, lse, ws))
        timed("cobs_decode_step", lambda: B.cobs_decode_step(cfg, inp["q"], kv, summ, out, lse, sel, cnt, ws))
        if wl is base:
            timed("cobs_adaptive_trim (tau 0.1)", lambda: B.cobs_adaptive_trim(cfg, scores, inp["seq_lens"], 0.1, 4, sel, cnt, ws))
            timed("cobs_sparse_decode on the trimmed selection", lambda: B.cobs_sparse_decode(cfg, inp["q"], kv, sel, cnt, out, lse, ws))
            timed("cobs_sparse_decode_static", lambda: B.cobs_sparse_decode_static(cfg, inp["q"], kv, sel, cnt, out, lse))
            timed("cobs_exact_select (reads every key)", lambda: B.cobs_exact_select(cfg, inp["q"], kv, sel, cnt, scores, ws))
            # the quantiser on its own: fp32 factors -> packed codes + scales
            xi = torch.randn((4096 * wl.rank, wl.head_dim), dtype=torch.float32, device=dev)
            codes = torch.zeros((xi.shape[0], B.cobs_padded_sub_dim(cfg) // 2), dtype=torch.uint8, device=dev)
            scale = torch.zeros(xi.shape[0], dtype=torch.float32, device=dev)
            timed("cobs_quantise_xi (32768 factor rows)", lambda: B.cobs_quantise_xi(cfg, xi, codes, scale))
            hw = torch.zeros(xi.numel(), dtype=torch.uint8, device=dev)
            timed("cobs_hw_e2m1_codes (test hook)", lambda: B.cobs_hw_e2m1_codes(xi.reshape(-1), hw))
            # one more token per sequence (the cache has room: lengths are set one block short first)
            inp["seq_lens"].fill_(wl.seq_len - wl.block_size)
            k_new = torch.randn((nb, hkv, D), device=dev).to(torch.bfloat16)
            v_new = torch.randn((nb, hkv, D), device=dev).to(torch.bfloat16)
            timed("cobs_append_token", lambda: B.cobs_append_token(cfg, k_new, v_new, inp, ws))
            q_host = inp["q"].cpu().pin_memory()
            out_host = torch.zeros((nb, hq, D), dtype=torch.float32).pin_memory()
            timed("cobs_decode_step_host (pinned host q / out)", lambda: B.cobs_decode_step_host(cfg, q_host, kv, summ, out_host, None, None, ws))
            os.environ["COBS_SCORE_PATH"] = "tcgen05"
            before = B.cobs_tcgen05_launches()
            timed("cobs_decode_step, scoring on tcgen05 (opt-in)", lambda: B.cobs_decode_step(cfg, inp["q"], kv, summ, out, lse, sel, cnt, ws))
            del os.environ["COBS_SCORE_PATH"]
            print(f"    tcgen05 launches: {B.cobs_tcgen05_launches() - before}")
        status = B.cobs_read_status(ws)
        if status != 0:
            raise RuntimeError(f"device status {status} ({B.status_string(status)})")
        del inp, kv, summ, ws
        torch.cuda.empty_cache()
    print(f"kernels launched: {B.cobs_kernel_launches()}")


if __name__ == "__main__":
    main()
