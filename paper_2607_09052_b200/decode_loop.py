"""Consecutive decode steps: append the new token, rebuild the summary of a block that just filled, run the
fused step.  Host orchestration only: every step of the path runs in the library's kernels
(cobs_append_token, cobs_build_summaries, cobs_decode_step).

A block gets its summary when it fills (Method, Cost: the Gram-trick build is paid once per block, i.e. once per
L decode steps per sequence); the partial last block has no summary and lies in the local window."""

from __future__ import annotations

from typing import Optional

import torch

from . import binding as B


class DecodeLoop:
    def __init__(self, wl, inputs, summ: Optional[B.SummaryBuffers] = None, ws: Optional[torch.Tensor] = None):
        """`wl`: the decode problem (any object binding.make_config accepts).  `inputs`: device tensors k_pages, v_pages, page_table, seq_lens (and u_q for a subspace descriptor) of a
        cache with room for the tokens to come: max_blocks * block_size tokens per sequence at most."""
        self.wl = wl
        self.inputs = inputs
        self.cfg = B.make_config(wl)
        self.kv = B.make_kv(inputs)
        self.summ = summ if summ is not None else B.SummaryBuffers(self.cfg, inputs["k_pages"].device, inputs.get("u_q"))
        self.ws = ws if ws is not None else B.alloc_workspace(self.cfg, inputs["k_pages"].device)
        self.lens = [int(t) for t in inputs["seq_lens"].cpu().tolist()]      # host mirror of the lengths
        self.rebuilds = 0
        if summ is None:
            B.cobs_build_summaries(self.cfg, self.kv, 0, wl.max_blocks, self.summ, self.ws)

    def step(self, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, out: torch.Tensor,
             lse: Optional[torch.Tensor] = None, sel_idx: Optional[torch.Tensor] = None,
             sel_cnt: Optional[torch.Tensor] = None, stream=None):
        """One decode step: the new token's key / value rows [B][Hkv][D] go into the cache, then q [B][Hq][D]
        attends over the selected blocks and the window, the new token included."""
        L = self.wl.block_size
        if max(self.lens) + 1 > self.wl.max_blocks * L:
            raise ValueError("the cache has no room for another token")
        B.cobs_append_token(self.cfg, k_new, v_new, self.inputs, self.ws, stream)
        self.lens = [t + 1 for t in self.lens]
        filled = sorted({t // L - 1 for t in self.lens if t % L == 0})
        if filled:
            # blocks [first, last] of every sequence, clipped per sequence to its full blocks: the block that just
            # filled is new; a sequence that did not fill one gets the same bits again (the build is deterministic)
            B.cobs_build_summaries(self.cfg, self.kv, filled[0], filled[-1] + 1, self.summ, self.ws, stream)
            self.rebuilds += 1
        B.cobs_decode_step(self.cfg, q, self.kv, self.summ, out, lse, sel_idx, sel_cnt, self.ws, stream)
