"""cobs_sparse_decode_static: the attention step for callers that are not allowed to allocate device memory
(its scratch is a fixed array inside the library).  It must give what cobs_sparse_decode gives, call after call,
although every call reuses the same scratch and finds the previous call's leftovers in it."""

import numpy as np
import pytest
import torch

from paper_2607_09052_b200 import synth
from parity import OUT_TOL, oracle_attend, out_rel_err

pytestmark = pytest.mark.gpu


def test_static_scratch_variant_matches_workspace_variant_on_two_calls_in_a_row():
    from paper_2607_09052_b200 import binding as B
    base = synth.named_workloads()["cfg4_128k"]
    # the second call has another batch, context and top-k: it finds the first call's counters and partials laid
    # out differently in the shared scratch
    for call, (seed, batch, seq_len, topk) in enumerate(((41, 3, 8192, 64), (42, 2, 4096, 24))):
        wl = base.replace(batch=batch, seq_len=seq_len, topk=topk)
        cfg = B.make_config(wl)
        ws = B.alloc_workspace(cfg, "cuda")
        cpu = synth.generate(wl.replace(seed=seed))
        inp = {k: (v.cuda() if k != "planted" else v) for k, v in cpu.items()}
        kv = B.make_kv(inp)
        # a selection to attend over: the library's own, from summaries it builds (any valid selection would do)
        summ = B.SummaryBuffers(cfg, "cuda")
        B.cobs_build_summaries(cfg, kv, 0, wl.max_blocks, summ, ws)
        sel = torch.zeros((wl.batch, wl.n_kv_heads, wl.topk), dtype=torch.int32, device="cuda")
        cnt = torch.zeros((wl.batch, wl.n_kv_heads), dtype=torch.int32, device="cuda")
        B.cobs_score_select(cfg, inp["q"], summ, inp["seq_lens"], sel, cnt, None, ws)
        shape = (wl.batch, wl.n_q_heads, wl.head_dim)
        out_ws = torch.zeros(shape, dtype=torch.float32, device="cuda")
        lse_ws = torch.zeros(shape[:2], dtype=torch.float32, device="cuda")
        B.cobs_sparse_decode(cfg, inp["q"], kv, sel, cnt, out_ws, lse_ws, ws)
        out_st = torch.full(shape, float("nan"), dtype=torch.float32, device="cuda")
        lse_st = torch.full(shape[:2], float("nan"), dtype=torch.float32, device="cuda")
        B.cobs_sparse_decode_static(cfg, inp["q"], kv, sel, cnt, out_st, lse_st)
        torch.cuda.synchronize()
        assert B.cobs_read_status(ws) == 0
        err = out_rel_err(out_st.cpu().numpy(), out_ws.cpu().double().numpy())
        assert np.all(err <= OUT_TOL), (call, err.max())
        assert np.allclose(lse_st.cpu().numpy(), lse_ws.cpu().numpy(), atol=2e-3, rtol=0), call
        # and against the CPU oracle's attention over the same blocks, on two units
        G = wl.group
        for (b, h) in ((0, 0), (batch - 1, wl.n_kv_heads - 1)):
            chosen = [int(x) for x in sel[b, h].cpu() if x >= 0]
            ref_out, ref_lse = oracle_attend(wl, cpu, b, h, chosen)
            hs = slice(h * G, (h + 1) * G)
            assert np.all(out_rel_err(out_st[b, hs].cpu().numpy(), ref_out) <= OUT_TOL), (call, b, h)
            assert np.allclose(lse_st[b, hs].cpu().numpy(), ref_lse, atol=2e-3, rtol=0), (call, b, h)


def test_static_scratch_variant_refuses_what_does_not_fit():
    from paper_2607_09052_b200 import binding as B
    wl = synth.named_workloads()["cfg5_64k_g8"].replace(batch=64)      # 512 units x G = 8: more than 4 MiB of partials
    cfg = B.make_config(wl)
    fake = torch.zeros(64, dtype=torch.uint8, device="cuda")
    kv = B.KV(fake.data_ptr(), fake.data_ptr(), fake.data_ptr(), fake.data_ptr(), 1)
    with pytest.raises(B.CobsError) as e:
        B.cobs_sparse_decode_static(cfg, fake, kv, fake, fake, fake, None)
    assert e.value.status == 3
