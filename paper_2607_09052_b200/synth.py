"""Seeded synthetic decode workloads (inputs only).

This module draws queries, a paged bf16 KV cache, a page table and, for the
query-subspace descriptor, an orthonormal basis.  It holds none of the method's
arithmetic (no summaries, scores, selection or attention) and is the one module
that both the CUDA path's tests and the CPU oracle's tests read inputs from.

Every tensor is a pure function of (workload, seed, batch index, tensor name)
and of the device the generator runs on (torch's CPU and CUDA generators give
different streams for the same seed; tests that compare against the CPU oracle
either generate on the CPU and upload, or generate on the device and download
the units they check).
"""

from __future__ import annotations

import dataclasses
import math
from dataclasses import dataclass, field
from typing import List, Optional

import torch


@dataclass
class Workload:
    name: str
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    seq_len: int                     # tokens in cache (capacity; per-sequence lengths in seq_lens)
    block_size: int
    page_size: int
    rank: int
    topk: int
    window: int
    summary_dtype: str = "bf16"      # "fp32" | "bf16" | "fp4"
    scale_dtype: str = "fp32"        # "fp32" | "fp16"
    sub_dim: int = 0                 # 0 = full-space descriptor
    key_model: str = "iid"           # "iid" | "block_offset" | "lowrank16" | "cov_perturb"
    query_model: str = "iid"         # "iid" | "spectrum"
    planted: int = 0                 # planted high-mass blocks per KV head
    shuffle_pages: bool = False
    seed: int = 0
    seq_lens: Optional[List[int]] = None   # defaults to [seq_len] * batch

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def max_blocks(self) -> int:
        return self.seq_len // self.block_size

    @property
    def max_pages_per_seq(self) -> int:
        return (self.seq_len + self.page_size - 1) // self.page_size

    def lens(self) -> List[int]:
        return list(self.seq_lens) if self.seq_lens is not None else [self.seq_len] * self.batch

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def named_workloads():
    """The decode workloads this project measures and tests, by name."""
    w = {}
    w["cfg1_tiny"] = Workload("cfg1_tiny", 1, 4, 1, 64, 2048, 64, 64, rank=4, topk=4, window=64,
                              summary_dtype="fp32", key_model="iid", planted=2, seed=0)
    w["cfg2_32k"] = Workload("cfg2_32k", 1, 32, 8, 128, 32768, 64, 64, rank=4, topk=16, window=512,
                             summary_dtype="bf16", key_model="block_offset", planted=4, seed=2)
    w["cfg3a_32k_subspace"] = Workload("cfg3a_32k_subspace", 4, 32, 8, 128, 32768, 64, 64, rank=4, topk=16,
                                       window=512, summary_dtype="fp4", sub_dim=85,
                                       key_model="block_offset", query_model="spectrum", planted=4, seed=3)
    w["cfg3b_32k_k85"] = Workload("cfg3b_32k_k85", 4, 32, 8, 128, 32768, 64, 64, rank=4, topk=85, window=512,
                                  summary_dtype="fp4", key_model="block_offset", planted=4, seed=3)
    w["cfg4_128k"] = Workload("cfg4_128k", 16, 32, 8, 128, 131072, 64, 16, rank=8, topk=64, window=512,
                              summary_dtype="fp4", key_model="lowrank16", shuffle_pages=True, seed=4)
    w["cfg5_64k_g8"] = Workload("cfg5_64k_g8", 8, 64, 8, 128, 65536, 128, 128, rank=4, topk=16, window=512,
                                summary_dtype="fp4", key_model="cov_perturb", seed=5)
    return w


def _gen(device, *key) -> torch.Generator:
    g = torch.Generator(device=device)
    h = 0x9E3779B97F4A7C15
    for k in key:
        h = (h * 6364136223846793005 + (hash(k) if not isinstance(k, int) else k) + 1442695040888963407) % (1 << 63)
    g.manual_seed(h)
    return g


_TENSOR_IDS = {"q": 1, "k": 2, "v": 3, "perm": 4, "plant": 5, "basis": 6, "koff": 7, "voff": 8, "mix": 9,
               "z": 10, "cov_u": 11, "cov_c": 12, "noise": 13}


def _randn(shape, device, wl: Workload, b: int, name: str):
    return torch.randn(shape, generator=_gen(device, wl.seed, b, _TENSOR_IDS[name]), device=device,
                       dtype=torch.float32)


def window_start_tokens(seq_len: int, window: int, block_size: int) -> int:
    """First token of the block-aligned local window (an input-layout fact the
    planted-block recipe needs: planted blocks are never placed under the window)."""
    return (max(0, seq_len - window) // block_size) * block_size


def spectrum_for_rank90(dim: int, rank90: int):
    """Geometric eigenvalue sequence rho**i (i < dim) such that exactly `rank90` leading
    eigenvalues are needed to hold 90 % of the trace (rho in the middle of the interval
    of ratios with that property, found by bisection); scaled to trace `dim`."""
    def need(rho):
        lam = [rho ** i for i in range(dim)]
        tot, acc = sum(lam), 0.0
        for n, x in enumerate(lam, 1):
            acc += x
            if acc >= 0.9 * tot:
                return n
        return dim

    def smallest_rho_needing(n):
        lo, hi = 0.5, 0.999999
        for _ in range(60):
            mid = 0.5 * (lo + hi)
            if need(mid) < n:
                lo = mid
            else:
                hi = mid
        return hi

    rho = 0.5 * (smallest_rho_needing(rank90) + smallest_rho_needing(rank90 + 1))
    assert need(rho) == rank90
    lam = torch.tensor([rho ** i for i in range(dim)], dtype=torch.float64)
    return lam * (dim / lam.sum())


def query_basis(wl: Workload, device="cpu"):
    """Per-KV-head orthogonal matrix [Hkv, D, D] whose columns are the eigenvectors of the
    query second moment used by query_model == "spectrum" (column i pairs with eigenvalue i)."""
    out = []
    for h in range(wl.n_kv_heads):
        a = torch.randn((wl.head_dim, wl.head_dim), generator=_gen("cpu", wl.seed, 1000 + h, _TENSOR_IDS["basis"]),
                        dtype=torch.float64)
        qmat, _ = torch.linalg.qr(a)
        out.append(qmat)
    return torch.stack(out).to(device)


def calibration_queries(wl: Workload, n: int, h: int, device="cpu"):
    """n unscaled calibration queries for KV head h under query_model == "spectrum" ([n, D] float64)."""
    lam = spectrum_for_rank90(wl.head_dim, 68)
    basis = query_basis(wl, "cpu")[h]
    z = torch.randn((n, wl.head_dim), generator=_gen("cpu", wl.seed, 2000 + h, _TENSOR_IDS["z"]), dtype=torch.float64)
    return ((z * lam.sqrt()) @ basis.T).to(device)


def generate(wl: Workload, device="cpu"):
    """Draw one workload.  Returns a dict of torch tensors on `device`:

    q           [B, Hq, D]             bf16
    k_pages     [n_pages, Hkv, P, D]   bf16   (n_pages = B * max_pages_per_seq)
    v_pages     [n_pages, Hkv, P, D]   bf16
    page_table  [B, max_pages_per_seq] int32
    seq_lens    [B]                    int32
    u_q         [Hkv, D, sub_dim]      fp32   (only when wl.sub_dim > 0)
    planted     [B, Hkv, planted]      int64  block indices of the planted blocks
    """
    B, Hq, Hkv, D, T, L, P = wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.seq_len, wl.block_size, wl.page_size
    G = wl.group
    mpp = wl.max_pages_per_seq
    n_pages = B * mpp
    lens = wl.lens()
    assert len(lens) == B and max(lens) <= T and L % P == 0

    # page table: identity, or a seeded permutation of all pages
    if wl.shuffle_pages:
        perm = torch.randperm(n_pages, generator=_gen("cpu", wl.seed, 0, _TENSOR_IDS["perm"]))
    else:
        perm = torch.arange(n_pages)
    page_table = perm.view(B, mpp).to(torch.int32).to(device)

    # queries
    if wl.query_model == "spectrum":
        lam = spectrum_for_rank90(D, 68).to(device)
        basis = query_basis(wl, device)  # [Hkv, D, D]
    q = torch.empty((B, Hq, D), dtype=torch.bfloat16, device=device)
    for b in range(B):
        z = _randn((Hq, D), device, wl, b, "q")
        if wl.query_model == "spectrum":
            z = z.double().view(Hkv, G, D) * lam.sqrt()
            z = torch.einsum("hgi,hdi->hgd", z, basis).reshape(Hq, D).float()
        q[b] = z.to(torch.bfloat16)

    k_pages = torch.empty((n_pages, Hkv, P, D), dtype=torch.bfloat16, device=device)
    v_pages = torch.empty((n_pages, Hkv, P, D), dtype=torch.bfloat16, device=device)
    planted = torch.zeros((B, Hkv, max(wl.planted, 0)), dtype=torch.int64)
    n_tok_alloc = mpp * P
    nb_alloc = (n_tok_alloc + L - 1) // L

    for b in range(B):
        k = _randn((n_tok_alloc, Hkv, D), device, wl, b, "k")
        v = _randn((n_tok_alloc, Hkv, D), device, wl, b, "v")
        if wl.key_model == "block_offset":
            koff = 0.5 * _randn((nb_alloc, Hkv, D), device, wl, b, "koff")
            voff = 0.5 * _randn((nb_alloc, Hkv, D), device, wl, b, "voff")
            k = k + koff.repeat_interleave(L, dim=0)[:n_tok_alloc]
            v = v + voff.repeat_interleave(L, dim=0)[:n_tok_alloc]
        elif wl.key_model == "lowrank16":
            mix = _randn((Hkv, D, 16), device, wl, 10_000, "mix") / 4.0     # per head, shared by the batch
            z = _randn((n_tok_alloc, Hkv, 16), device, wl, b, "z")
            k = torch.einsum("thr,hdr->thd", z, mix) + 0.25 * k
        elif wl.key_model == "cov_perturb":
            u = _randn((nb_alloc, Hkv, D), device, wl, b, "cov_u")
            u = u / u.norm(dim=-1, keepdim=True)
            c = torch.rand((nb_alloc, Hkv, 1), generator=_gen(device, wl.seed, b, _TENSOR_IDS["cov_c"]),
                           device=device) * 4.0
            # rows ~ N(0, I + c u u^T):  x + (sqrt(1+c) - 1) (x.u) u
            ur = u.repeat_interleave(L, dim=0)[:n_tok_alloc]
            cr = c.repeat_interleave(L, dim=0)[:n_tok_alloc]
            k = k + ((1.0 + cr).sqrt() - 1.0) * (k * ur).sum(-1, keepdim=True) * ur
        elif wl.key_model != "iid":
            raise ValueError(wl.key_model)

        if wl.planted > 0:
            n_cand = window_start_tokens(lens[b], wl.window, L) // L
            for h in range(Hkv):
                pick = torch.randperm(n_cand, generator=_gen("cpu", wl.seed, b * 4096 + h, _TENSOR_IDS["plant"]))
                pick = pick[:min(wl.planted, n_cand)]
                planted[b, h, :len(pick)] = pick
                for p, blk in enumerate(pick.tolist()):
                    qh = q[b, h * G + (p % G)].float()
                    direction = qh / qh.norm() * math.sqrt(D)
                    noise = torch.randn((L, D), generator=_gen(device, wl.seed, (b * 4096 + h) * 64 + p,
                                                               _TENSOR_IDS["noise"]), device=device)
                    k[blk * L:(blk + 1) * L, h, :] = 0.8 * direction + 0.6 * noise

        kp = k.view(mpp, P, Hkv, D).permute(0, 2, 1, 3).to(torch.bfloat16)
        vp = v.view(mpp, P, Hkv, D).permute(0, 2, 1, 3).to(torch.bfloat16)
        idx = page_table[b].long()
        k_pages[idx] = kp
        v_pages[idx] = vp
        del k, v, kp, vp

    out = {"q": q, "k_pages": k_pages, "v_pages": v_pages, "page_table": page_table,
           "seq_lens": torch.tensor(lens, dtype=torch.int32, device=device), "planted": planted}
    if wl.sub_dim > 0:
        if wl.query_model == "spectrum":
            out["u_q"] = basis[:, :, :wl.sub_dim].float().contiguous()
        else:
            out["u_q"] = query_basis(wl, device)[:, :, :wl.sub_dim].float().contiguous()
    return out


def unit_kv(inputs, wl: Workload, b: int, h: int):
    """Logical K, V [T_b, D] of sequence b, KV head h, gathered through the page table
    (returned as float64 CPU tensors holding the exact bf16 values)."""
    t = int(inputs["seq_lens"][b])
    n_pg = (t + wl.page_size - 1) // wl.page_size
    idx = inputs["page_table"][b, :n_pg].long()
    k = inputs["k_pages"][idx, h].reshape(-1, wl.head_dim)[:t]
    v = inputs["v_pages"][idx, h].reshape(-1, wl.head_dim)[:t]
    return k.double().cpu(), v.double().cpu()


def unit_q(inputs, wl: Workload, b: int, h: int):
    """The G raw queries of KV head h in sequence b, [G, D] float64 CPU."""
    g = wl.group
    return inputs["q"][b, h * g:(h + 1) * g].double().cpu()
