"""Consecutive decode steps on the GPU (append a token, rebuild the summary of a block that just filled, fused
step) against the oracle run on a host mirror of the same cache, step by step: lengths that are not multiples of
the block size, blocks filling at different steps in different sequences, the window growing over a partial block."""

import numpy as np
import pytest
import torch

from oracle import cobs_oracle as O
from paper_2607_09052_b200 import synth
from parity import OUT_TOL, check_selection, oracle_attend, oracle_unit_step, oracle_unit_summaries, out_rel_err

pytestmark = pytest.mark.gpu


def _bf16_rows(gen, *shape):
    return torch.randn(*shape, generator=gen, dtype=torch.float32).to(torch.bfloat16)


@pytest.mark.parametrize("summary_dtype,P", [("fp32", 16), ("fp4", 16), ("bf16", 32)])
def test_decode_loop_matches_oracle_step_by_step(summary_dtype, P):
    from paper_2607_09052_b200 import binding as B
    from paper_2607_09052_b200.decode_loop import DecodeLoop

    L, D, G, Hkv = 32, 64, 2, 2
    start = [150, 97, 64]                        # mid-block, mid-block, exactly on a block boundary
    steps = 2 * L + 5
    wl = synth.Workload("loop", len(start), G * Hkv, Hkv, D, 12 * L, L, P, rank=4, topk=3, window=40,
                        summary_dtype=summary_dtype, key_model="block_offset", planted=1, shuffle_pages=True, seed=31,
                        seq_lens=start)
    host = synth.generate(wl)                    # CPU tensors: the oracle's mirror of the cache
    dev = {k: (v.cuda() if isinstance(v, torch.Tensor) and k != "planted" else v) for k, v in host.items()}
    loop = DecodeLoop(wl, dev)
    nb, hq = wl.batch, wl.n_q_heads
    out = torch.zeros((nb, hq, D), dtype=torch.float32, device="cuda")
    lse = torch.zeros((nb, hq), dtype=torch.float32, device="cuda")
    sel = torch.zeros((nb, Hkv, wl.topk), dtype=torch.int32, device="cuda")
    cnt = torch.zeros((nb, Hkv), dtype=torch.int32, device="cuda")
    gen = torch.Generator().manual_seed(77)
    swaps = 0
    for step in range(steps):
        q, k_new, v_new = _bf16_rows(gen, nb, hq, D), _bf16_rows(gen, nb, Hkv, D), _bf16_rows(gen, nb, Hkv, D)
        # the oracle's side: the same append on the host mirror
        for b in range(nb):
            t = int(host["seq_lens"][b])
            pg = int(host["page_table"][b, t // P])
            host["k_pages"][pg, :, t % P] = k_new[b]
            host["v_pages"][pg, :, t % P] = v_new[b]
            host["seq_lens"][b] = t + 1
        host["q"] = q
        loop.step(q.cuda(), k_new.cuda(), v_new.cuda(), out, lse, sel, cnt)
        assert B.cobs_read_status(loop.ws) == 0
        assert loop.lens == [int(t) for t in host["seq_lens"]]
        if step % 8 != 0 and step < steps - 3:    # compare every 8th step and the last three (the oracle is slow)
            continue
        o_gpu, l_gpu, s_gpu, c_gpu = out.cpu().numpy(), lse.cpu().numpy(), sel.cpu(), cnt.cpu()
        for b in range(nb):
            for h in range(Hkv):
                T = int(host["seq_lens"][b])
                n_cand = O.window_start(T, wl.window, L) // L
                hs = slice(h * G, (h + 1) * G)
                gpu_sel = [int(x) for x in s_gpu[b, h] if x >= 0]
                assert int(c_gpu[b, h]) == min(wl.topk, n_cand) == len(gpu_sel)
                assert all(0 <= x < n_cand for x in gpu_sel)
                # attention is exact given the selection: compare on the device's own selection
                ref_out, ref_lse = oracle_attend(wl, host, b, h, gpu_sel)
                assert np.all(out_rel_err(o_gpu[b, hs], ref_out) <= OUT_TOL), (step, b, h)
                assert np.allclose(l_gpu[b, hs], ref_lse, atol=2e-3, rtol=0)
                if summary_dtype == "fp32":
                    # the device built these summaries itself, in fp32: its selection must agree with the
                    # oracle's (own fp64 summaries) up to the tie band
                    st = oracle_unit_summaries(wl, host, b, h)
                    ref = oracle_unit_step(wl, host, b, h, st)
                    ok, msg, exact = check_selection(s_gpu[b, h].tolist(), ref["score"], n_cand, wl.topk)
                    assert ok, (step, b, h, msg)
                    swaps += 0 if exact else 1
    assert loop.rebuilds >= 4                     # three sequences crossed block boundaries at different steps
    torch.cuda.synchronize()
    # the cache on the device is the host mirror, bit for bit
    assert torch.equal(dev["seq_lens"].cpu(), host["seq_lens"])
    assert torch.equal(dev["k_pages"].cpu().view(torch.int16), host["k_pages"].view(torch.int16))
    assert torch.equal(dev["v_pages"].cpu().view(torch.int16), host["v_pages"].view(torch.int16))
    # and the summaries kept up to date block by block equal a rebuild of everything from the final cache
    fresh = B.SummaryBuffers(loop.cfg, "cuda")
    B.cobs_build_summaries(loop.cfg, loop.kv, 0, wl.max_blocks, fresh, loop.ws)
    mv, xv, sv = B.summary_views(loop.cfg, loop.summ)
    mf, xf, sf = B.summary_views(loop.cfg, fresh)
    for b in range(nb):
        n = int(host["seq_lens"][b]) // L
        assert torch.equal(mv[b, :, :n].contiguous().view(torch.uint8), mf[b, :, :n].contiguous().view(torch.uint8))
        assert torch.equal(xv[b, :, :n].contiguous().view(torch.uint8), xf[b, :, :n].contiguous().view(torch.uint8))
        if sv is not None and sf is not None:
            assert torch.equal(sv[b, :, :n].contiguous().view(torch.uint8), sf[b, :, :n].contiguous().view(torch.uint8))


def test_append_beyond_the_page_table_is_reported_not_faulted():
    from paper_2607_09052_b200 import binding as B
    wl = synth.Workload("full", 2, 4, 2, 64, 4 * 32, 32, 16, rank=2, topk=2, window=40, summary_dtype="bf16",
                        key_model="block_offset", planted=1, shuffle_pages=False, seed=5)
    host = synth.generate(wl)                    # both sequences are full: no position left in the page table
    dev = {k: (v.cuda() if isinstance(v, torch.Tensor) and k != "planted" else v) for k, v in host.items()}
    cfg = B.make_config(wl)
    ws = B.alloc_workspace(cfg, "cuda")
    k_before = dev["k_pages"].clone()
    new = torch.ones((2, 2, 64), dtype=torch.bfloat16, device="cuda")
    B.cobs_append_token(cfg, new, new, dev, ws)
    assert B.cobs_read_status(ws) == 6
    assert torch.equal(dev["seq_lens"].cpu(), host["seq_lens"])
    assert torch.equal(dev["k_pages"].view(torch.int16), k_before.view(torch.int16))
