"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header declares, and its
host-only entry points (sizes, validation) behave as documented.  No kernel is launched here."""

import ctypes as C
import os
import re

import pytest

from conftest import ROOT
from oracle import cobs_oracle as O
from paper_2607_09052_b200 import binding as B
from paper_2607_09052_b200 import build as build_mod
from paper_2607_09052_b200 import synth


@pytest.fixture(scope="module", autouse=True)
def built():
    build_mod.build()


def header_symbols():
    text = open(os.path.join(ROOT, "include", "cobs.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cobs_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    syms = header_symbols()
    assert len(syms) >= 12
    lib = B.lib()
    for s in syms:
        assert hasattr(lib, s), s
    assert sorted(B.EXPORTS) == syms


def test_status_strings():
    assert B.status_string(0) == "ok"
    assert "workspace" in B.status_string(3)
    assert B.status_string(99) == "unknown status"


def record_bytes(wl):
    cfg = B.make_config(wl)
    m, x, s = B.cobs_summary_bytes(cfg)
    n = wl.batch * wl.n_kv_heads * wl.max_blocks
    return (m + x + s) // n, (x + s) // n


def test_summary_record_bytes_follow_the_papers_accounting():
    wl = synth.named_workloads()
    assert record_bytes(wl["cfg2_32k"]) == (1280, 1024)            # bf16 mean 256 + 4 x 128 x 2
    assert record_bytes(wl["cfg3b_32k_k85"]) == (528, 272)         # 256 + (4 x 64 + 4 x 4): the table's 272
    assert record_bytes(wl["cfg4_128k"]) == (800, 544)             # r = 8
    assert record_bytes(wl["cfg3a_32k_subspace"]) == (464, 208)    # 85 -> 96 codes (48 B) per row
    assert record_bytes(wl["cfg4_128k"].replace(scale_dtype="fp16")) == (784, 528)
    # the factor bytes agree with the oracle's accounting wherever no padding is involved
    for r, d in ((4, 128), (4, 64), (6, 128)):
        w = wl["cfg3b_32k_k85"].replace(rank=r, sub_dim=0 if d == 128 else d)
        assert record_bytes(w)[1] == O.factor_bytes(r, d, "fp4")
    assert B.cobs_padded_sub_dim(B.make_config(wl["cfg3a_32k_subspace"])) == 96


def test_workspace_size_and_alignment_rules():
    wl = synth.named_workloads()["cfg4_128k"]
    cfg = B.make_config(wl)
    n = B.cobs_workspace_bytes(cfg)
    assert n % 256 == 0 and n > 4 * wl.batch * wl.n_q_heads * wl.max_blocks


@pytest.mark.parametrize("field,value,status", [
    ("head_dim", 96, 2), ("n_q_heads", 33, 1), ("n_q_heads", 24, 2), ("block_size", 48, 2), ("page_size", 8, 1),
    ("page_size", 128, 1), ("rank", 17, 1), ("sub_dim", 4, 1), ("sub_dim", 200, 1), ("topk", 0, 1), ("topk", 129, 1),
    ("window", 0, 1), ("summary_dtype", 3, 1), ("max_blocks", 0, 1), ("max_pages_per_seq", 3, 1), ("batch", 0, 1)])
def test_config_validation(field, value, status):
    wl = synth.named_workloads()["cfg2_32k"]
    cfg = B.make_config(wl)
    setattr(cfg, field, value)
    n = C.c_size_t()
    assert B.lib().cobs_workspace_bytes(C.byref(cfg), C.byref(n)) == status


def test_entry_points_reject_bad_pointers_before_launching():
    """NULL or misaligned pointers are refused on the host (nothing is launched, no GPU needed)."""
    wl = synth.named_workloads()["cfg1_tiny"]
    cfg = B.make_config(wl)
    lib = B.lib()
    kv = B.KV(0, 0, 0, 0, 0)
    sm = B.Summaries(0, 0, 0, 0)
    null = C.c_void_p(0)
    big = C.c_size_t(1 << 30)
    fake = C.c_void_p(0x10000)          # aligned, never dereferenced by the host code
    assert lib.cobs_decode_step(C.byref(cfg), null, C.byref(kv), C.byref(sm), null, null, null, null, fake, big, null) == 1
    assert lib.cobs_decode_step(C.byref(cfg), fake, C.byref(kv), C.byref(sm), fake, null, null, null, null, big, null) == 1
    assert lib.cobs_decode_step(C.byref(cfg), fake, C.byref(kv), C.byref(sm), fake, null, null, null, fake,
                                C.c_size_t(64), null) == 3
    assert lib.cobs_decode_step(C.byref(cfg), fake, C.byref(kv), C.byref(sm), fake, null, null, null,
                                C.c_void_p(0x10010), big, null) == 1
    assert lib.cobs_score_select(C.byref(cfg), fake, C.byref(sm), fake, fake, fake, null, fake, big, null) == 1
    assert lib.cobs_sparse_decode(C.byref(cfg), fake, C.byref(kv), fake, fake, fake, null, fake, big, null) == 1
    assert lib.cobs_build_summaries(C.byref(cfg), C.byref(kv), 0, 4, C.byref(sm), fake, big, null) == 1
    kv2 = B.KV(0x10000, 0x20000, 0x30000, 0x40000, 32)
    assert lib.cobs_build_summaries(C.byref(cfg), C.byref(kv2), 5, 4, C.byref(sm), fake, big, null) == 1
    assert lib.cobs_build_summaries(C.byref(cfg), C.byref(kv2), 0, 33, C.byref(sm), fake, big, null) == 1
    assert lib.cobs_quantise_xi(C.byref(cfg), fake, C.c_int64(3), fake, fake, null) == 1
    assert lib.cobs_read_status(null, big, null, null) == 1


def test_pack_unpack_fp4_layout():
    import torch
    codes = torch.arange(16, dtype=torch.uint8).repeat(2)[:21].view(1, 21)
    packed = B.pack_fp4_rows(codes, 32)
    assert packed.shape == (1, 16)
    assert packed[0, 0] == (0 | (1 << 4)) and packed[0, 10] == 4 and packed[0, 11] == 0
    assert torch.equal(B.unpack_fp4_rows(packed, 21), codes)
