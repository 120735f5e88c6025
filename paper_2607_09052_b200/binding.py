"""ctypes binding of libcobs.so: the same entry points as include/cobs.h, taking torch tensors.

Argument marshalling only.  Every step of the path runs in the CUDA library; there is no CPU or
PyTorch fallback: if the library is missing or a call returns a nonzero status this module raises.
"""

from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcobs.so")

SUMM_DTYPES = {"fp32": 0, "bf16": 1, "fp4": 2}
SCALE_DTYPES = {"fp32": 0, "fp16": 1}

EXPORTS = [
    "cobs_status_string", "cobs_padded_sub_dim", "cobs_summary_bytes", "cobs_workspace_bytes", "cobs_reset_status",
    "cobs_read_status", "cobs_build_summaries", "cobs_quantise_xi", "cobs_score_select", "cobs_sparse_decode",
    "cobs_decode_step", "cobs_decode_step_host", "cobs_kernel_launches", "cobs_tcgen05_launches", "cobs_sparse_decode_static", "cobs_append_token", "cobs_exact_select",
    "cobs_adaptive_trim", "cobs_hw_e2m1_codes",
]


class CobsError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


class Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "batch", "n_q_heads", "n_kv_heads", "head_dim", "block_size", "page_size", "rank", "sub_dim", "topk",
        "window", "summary_dtype", "scale_dtype", "max_blocks", "max_pages_per_seq")]


class KV(C.Structure):
    _fields_ = [("k_pages", C.c_void_p), ("v_pages", C.c_void_p), ("page_table", C.c_void_p),
                ("seq_lens", C.c_void_p), ("n_pages", C.c_int64)]


class Summaries(C.Structure):
    _fields_ = [("mean", C.c_void_p), ("xi", C.c_void_p), ("scale", C.c_void_p), ("u_q", C.c_void_p),
                ("skew", C.c_void_p)]


_lib = None


def use_library(path: str):
    """Load the library from `path` instead of the default build (before the first call): used by the benchmark's
    phase-timing mode, which runs the build that carries the timing code."""
    global _lib, LIB_PATH
    if _lib is not None:
        raise RuntimeError("the library is already loaded")
    LIB_PATH = path


def lib():
    """Load libcobs.so once.  Raises if it has not been built (python -m paper_2607_09052_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2607_09052_b200.build`; "
                               "there is no fallback path")
        l = C.CDLL(LIB_PATH)
        l.cobs_status_string.restype = C.c_char_p
        l.cobs_status_string.argtypes = [C.c_int32]
        for name in EXPORTS[1:]:
            getattr(l, name).restype = C.c_int32
        l.cobs_kernel_launches.restype = C.c_int64
        l.cobs_tcgen05_launches.restype = C.c_int64
        _lib = l
    return _lib


def cobs_kernel_launches() -> int:
    return int(lib().cobs_kernel_launches())


def cobs_tcgen05_launches() -> int:
    return int(lib().cobs_tcgen05_launches())


def status_string(status: int) -> str:
    return lib().cobs_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != 0:
        raise CobsError(status, where)


def _ptr(t: Optional[torch.Tensor]):
    return C.c_void_p(t.data_ptr()) if t is not None else C.c_void_p(0)


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def make_config(wl) -> Config:
    """The library's configuration struct from any object that names a decode problem by the attributes batch,
    n_q_heads, n_kv_heads, head_dim, block_size, page_size, rank, sub_dim, topk, window, summary_dtype
    ("fp32" | "bf16" | "fp4"), scale_dtype ("fp32" | "fp16"), max_blocks and max_pages_per_seq."""
    return Config(wl.batch, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.block_size, wl.page_size, wl.rank, wl.sub_dim,
                  wl.topk, wl.window, SUMM_DTYPES[wl.summary_dtype], SCALE_DTYPES[wl.scale_dtype], wl.max_blocks,
                  wl.max_pages_per_seq)


def make_kv(inputs) -> KV:
    return KV(inputs["k_pages"].data_ptr(), inputs["v_pages"].data_ptr(), inputs["page_table"].data_ptr(),
              inputs["seq_lens"].data_ptr(), inputs["k_pages"].shape[0])


def cobs_padded_sub_dim(cfg: Config) -> int:
    v = lib().cobs_padded_sub_dim(C.byref(cfg))
    if v < 0:
        raise CobsError(1, "cobs_padded_sub_dim")
    return v


def cobs_summary_bytes(cfg: Config):
    a, b, c = C.c_size_t(), C.c_size_t(), C.c_size_t()
    _check(lib().cobs_summary_bytes(C.byref(cfg), C.byref(a), C.byref(b), C.byref(c)), "cobs_summary_bytes")
    return a.value, b.value, c.value


def cobs_workspace_bytes(cfg: Config) -> int:
    n = C.c_size_t()
    _check(lib().cobs_workspace_bytes(C.byref(cfg), C.byref(n)), "cobs_workspace_bytes")
    return n.value


class SummaryBuffers:
    """Device buffers for the summary arrays of one workload, sized by the library."""

    def __init__(self, cfg: Config, device, u_q: Optional[torch.Tensor] = None, skew: bool = False):
        mb, xb, sb = cobs_summary_bytes(cfg)
        self.mean = torch.zeros(max(mb, 16), dtype=torch.uint8, device=device)
        self.xi = torch.zeros(max(xb, 16), dtype=torch.uint8, device=device)
        self.scale = torch.zeros(max(sb, 16), dtype=torch.uint8, device=device)
        self.u_q = u_q
        # the diagonal-skew variant: one fp32 scalar per stored factor, [B][Hkv][NB][r]
        self.skew = (torch.zeros((cfg.batch, cfg.n_kv_heads, cfg.max_blocks, max(cfg.rank, 1)), dtype=torch.float32,
                                 device=device) if skew else None)
        self.nbytes = (mb, xb, sb)

    def struct(self) -> Summaries:
        return Summaries(self.mean.data_ptr(), self.xi.data_ptr(), self.scale.data_ptr(),
                         self.u_q.data_ptr() if self.u_q is not None else 0,
                         self.skew.data_ptr() if self.skew is not None else 0)


def alloc_workspace(cfg: Config, device) -> torch.Tensor:
    ws = torch.empty(cobs_workspace_bytes(cfg) + 256, dtype=torch.uint8, device=device)
    off = (-ws.data_ptr()) % 256
    ws = ws[off:off + cobs_workspace_bytes(cfg)]
    cobs_reset_status(ws)
    return ws


def cobs_reset_status(ws: torch.Tensor, stream=None):
    _check(lib().cobs_reset_status(_ptr(ws), C.c_size_t(ws.numel()), _stream(stream)), "cobs_reset_status")


def cobs_read_status(ws: torch.Tensor, stream=None) -> int:
    code = C.c_int32(-1)
    _check(lib().cobs_read_status(_ptr(ws), C.c_size_t(ws.numel()), _stream(stream), C.byref(code)),
           "cobs_read_status")
    return code.value


def cobs_build_summaries(cfg: Config, kv: KV, block_begin: int, block_end: int, summ: SummaryBuffers,
                         ws: torch.Tensor, stream=None):
    s = summ.struct()
    _check(lib().cobs_build_summaries(C.byref(cfg), C.byref(kv), C.c_int32(block_begin), C.c_int32(block_end),
                                      C.byref(s), _ptr(ws), C.c_size_t(ws.numel()), _stream(stream)),
           "cobs_build_summaries")


def cobs_append_token(cfg: Config, k_new: torch.Tensor, v_new: torch.Tensor, inputs, ws: torch.Tensor, stream=None):
    """Write one new token per sequence into the paged cache of `inputs` (k_pages, v_pages, page_table, seq_lens)
    and advance seq_lens on the device."""
    _check(lib().cobs_append_token(C.byref(cfg), _ptr(k_new), _ptr(v_new), _ptr(inputs["k_pages"]), _ptr(inputs["v_pages"]),
                                   _ptr(inputs["page_table"]), _ptr(inputs["seq_lens"]),
                                   C.c_int64(inputs["k_pages"].shape[0]), _ptr(ws), C.c_size_t(ws.numel()),
                                   _stream(stream)), "cobs_append_token")


def cobs_quantise_xi(cfg: Config, xi_fp32: torch.Tensor, codes: torch.Tensor, scale: torch.Tensor, stream=None):
    n_vectors = xi_fp32.shape[0]
    _check(lib().cobs_quantise_xi(C.byref(cfg), _ptr(xi_fp32), C.c_int64(n_vectors), _ptr(codes), _ptr(scale),
                                  _stream(stream)), "cobs_quantise_xi")


def cobs_hw_e2m1_codes(x: torch.Tensor, codes: torch.Tensor, stream=None):
    """codes[i] = the E2M1 code the GPU's own conversion instruction gives x[i] (test hook for the rounding rule)."""
    assert x.dtype == torch.float32 and codes.dtype == torch.uint8 and x.numel() == codes.numel()
    _check(lib().cobs_hw_e2m1_codes(_ptr(x), C.c_int64(x.numel()), _ptr(codes), _stream(stream)), "cobs_hw_e2m1_codes")


def cobs_score_select(cfg: Config, q: torch.Tensor, summ: SummaryBuffers, seq_lens: torch.Tensor,
                      sel_idx: torch.Tensor, sel_cnt: torch.Tensor, scores: Optional[torch.Tensor],
                      ws: torch.Tensor, stream=None):
    s = summ.struct()
    _check(lib().cobs_score_select(C.byref(cfg), _ptr(q), C.byref(s), _ptr(seq_lens), _ptr(sel_idx), _ptr(sel_cnt),
                                   _ptr(scores), _ptr(ws), C.c_size_t(ws.numel()), _stream(stream)),
           "cobs_score_select")


def cobs_exact_select(cfg: Config, q: torch.Tensor, kv: KV, sel_idx: torch.Tensor, sel_cnt: torch.Tensor,
                      scores: Optional[torch.Tensor], ws: torch.Tensor, stream=None):
    """Selection by exact block masses (reads every key): the quality reference for cobs_score_select."""
    _check(lib().cobs_exact_select(C.byref(cfg), _ptr(q), C.byref(kv), _ptr(sel_idx), _ptr(sel_cnt), _ptr(scores),
                                   _ptr(ws), C.c_size_t(ws.numel()), _stream(stream)), "cobs_exact_select")


def cobs_adaptive_trim(cfg: Config, scores: torch.Tensor, seq_lens: torch.Tensor, tau: float, k_min: int,
                       sel_idx: torch.Tensor, sel_cnt: torch.Tensor, ws: torch.Tensor, stream=None):
    """Trim a selection, in place, to the smallest count that holds (1 - tau) of the candidates' total score
    (an extension, not in the paper; see include/cobs.h)."""
    _check(lib().cobs_adaptive_trim(C.byref(cfg), _ptr(scores), _ptr(seq_lens), C.c_float(tau), C.c_int32(k_min),
                                    _ptr(sel_idx), _ptr(sel_cnt), _ptr(ws), C.c_size_t(ws.numel()), _stream(stream)),
           "cobs_adaptive_trim")


def cobs_sparse_decode(cfg: Config, q: torch.Tensor, kv: KV, sel_idx: torch.Tensor, sel_cnt: torch.Tensor,
                       out: torch.Tensor, lse: Optional[torch.Tensor], ws: torch.Tensor, stream=None):
    _check(lib().cobs_sparse_decode(C.byref(cfg), _ptr(q), C.byref(kv), _ptr(sel_idx), _ptr(sel_cnt), _ptr(out),
                                    _ptr(lse), _ptr(ws), C.c_size_t(ws.numel()), _stream(stream)),
           "cobs_sparse_decode")


def cobs_sparse_decode_static(cfg: Config, q: torch.Tensor, kv: KV, sel_idx: torch.Tensor, sel_cnt: torch.Tensor,
                              out: torch.Tensor, lse: Optional[torch.Tensor], stream=None):
    """cobs_sparse_decode without a workspace: the scratch is a fixed device array inside the library, so the
    call allocates nothing (for callers that are not allowed to allocate device memory).  Raises CobsError(3)
    when the configuration needs more scratch than the library holds."""
    _check(lib().cobs_sparse_decode_static(C.byref(cfg), _ptr(q), C.byref(kv), _ptr(sel_idx), _ptr(sel_cnt),
                                           _ptr(out), _ptr(lse), _stream(stream)), "cobs_sparse_decode_static")


def cobs_decode_step(cfg: Config, q: torch.Tensor, kv: KV, summ: SummaryBuffers, out: torch.Tensor,
                     lse: Optional[torch.Tensor], sel_idx: Optional[torch.Tensor], sel_cnt: Optional[torch.Tensor],
                     ws: torch.Tensor, stream=None):
    s = summ.struct()
    _check(lib().cobs_decode_step(C.byref(cfg), _ptr(q), C.byref(kv), C.byref(s), _ptr(out), _ptr(lse),
                                  _ptr(sel_idx), _ptr(sel_cnt), _ptr(ws), C.c_size_t(ws.numel()), _stream(stream)),
           "cobs_decode_step")


def cobs_decode_step_host(cfg: Config, q_host: torch.Tensor, kv: KV, summ: SummaryBuffers, out_host: torch.Tensor,
                          sel_idx_host: Optional[torch.Tensor], sel_cnt_host: Optional[torch.Tensor],
                          ws: torch.Tensor, stream=None):
    assert not q_host.is_cuda and not out_host.is_cuda
    s = summ.struct()
    _check(lib().cobs_decode_step_host(C.byref(cfg), _ptr(q_host), C.byref(kv), C.byref(s), _ptr(out_host),
                                       _ptr(sel_idx_host), _ptr(sel_cnt_host), _ptr(ws), C.c_size_t(ws.numel()),
                                       _stream(stream)), "cobs_decode_step_host")


# ---------------------------------------------------------------------------------------------------
# Summary array layout <-> plain tensors (layout only; no arithmetic).
# ---------------------------------------------------------------------------------------------------

def pack_fp4_rows(codes: torch.Tensor, ds_pad: int) -> torch.Tensor:
    """codes [..., Ds] uint8 (one E2M1 code per element) -> packed [..., Ds_pad / 2] bytes:
    element 2j in the low nibble of byte j, element 2j + 1 in the high nibble, padding codes 0."""
    ds = codes.shape[-1]
    padded = torch.zeros(codes.shape[:-1] + (ds_pad,), dtype=torch.uint8, device=codes.device)
    padded[..., :ds] = codes
    return (padded[..., 0::2] | (padded[..., 1::2] << 4)).contiguous()


def unpack_fp4_rows(packed: torch.Tensor, ds: int) -> torch.Tensor:
    lo, hi = packed & 15, packed >> 4
    return torch.stack([lo, hi], dim=-1).reshape(packed.shape[:-1] + (-1,))[..., :ds].contiguous()


def summary_views(cfg: Config, summ: SummaryBuffers):
    """Typed views of the raw summary buffers: (mean [B,Hkv,NB,D], xi, scale).

    xi is [B,Hkv,NB,r,Ds] fp32/bf16, or packed bytes [B,Hkv,NB,r,Ds_pad/2] for FP4 (scale [B,Hkv,NB,r])."""
    B, H, NB, D, r = cfg.batch, cfg.n_kv_heads, cfg.max_blocks, cfg.head_dim, cfg.rank
    ds = cfg.sub_dim or D
    mb, xb, sb = summ.nbytes
    if cfg.summary_dtype == 0:
        mean = summ.mean[:mb].view(torch.float32).view(B, H, NB, D)
        xi = summ.xi[:xb].view(torch.float32).view(B, H, NB, r, ds)
        return mean, xi, None
    mean = summ.mean[:mb].view(torch.bfloat16).view(B, H, NB, D)
    if cfg.summary_dtype == 1:
        return mean, summ.xi[:xb].view(torch.bfloat16).view(B, H, NB, r, ds), None
    ds_pad = cobs_padded_sub_dim(cfg)
    xi = summ.xi[:xb].view(B, H, NB, r, ds_pad // 2)
    sdt = torch.float16 if cfg.scale_dtype == 1 else torch.float32
    return mean, xi, summ.scale[:sb].view(sdt).view(B, H, NB, r)
