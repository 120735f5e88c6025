// Shared device helpers and the kernel parameter block of the COBS decode library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "cobs.h"

namespace cobs {

constexpr int kStatusBytes = 256;          // status word lives in the first 256 bytes of the workspace
constexpr int kMaxSplits = 64;             // upper bound on split-KV partials per (sequence, KV head)
constexpr int kMaxUnits = 65535;           // (sequence, KV head) units a workspace has counters for
constexpr int kCtlBytes = kStatusBytes + 6 * kMaxUnits * 4;   // status block + two sets of counters, zeroed by cobs_reset_status

// Everything a kernel needs, passed by value.
struct Params {
  int B, Hq, Hkv, G, D, L, P;
  int r, Ds, Ds_pad;          // Ds = sub_dim or D; Ds_pad = packed FP4 row length in elements
  int topk, window, NB, mpp;
  int summ_dtype, scale_dtype;
  int n_splits;               // split-KV partials per unit
  long long n_pages;
  // inputs
  const __nv_bfloat16 *q;
  const __nv_bfloat16 *k_pages, *v_pages;
  const int32_t *page_table, *seq_lens;
  // summaries
  void *mean, *xi, *scale;
  const float *u_q;
  float *skew;                // optional [B][Hkv][NB][r] fp32: third-cumulant scalar per stored factor (full-space descriptors)
  // workspace pieces
  int32_t *status;
  // hand-off counters of the persistent kernel: two sets, used by alternate launches (bit 31 of the epoch word names
  // the set of the next launch; set 1 lies 3 ints after set 0 for the two words, ctl_set_stride ints for the arrays)
  int *ctl_epoch;             // set of the next launch (bit 31) | CTAs of the running launch that have begun
  int *ctl_item;              // next attention item to hand out
  int *ctl_bar;               // CTAs that have passed the grid barrier after the query projection
  int *ctl_score;             // [B * Hkv] scored chunks per unit
  int *ctl_ready;             // [B * Hkv] 1 once the unit's selection is written
  int *ctl_att;               // [B * Hkv] attention slices finished per unit
  int ctl_set_stride;         // ints from a per-unit array of set 0 to the same array of set 1 (the same for every shape)
  const float *qtilde;        // [B][Hq][Ds_pad] projected subspace query (what the scoring reads), or NULL
  float *qtilde_out;          // where the step kernel's prologue writes it (workspace)
  float *e;                   // [B][Hkv][G][NB]
  float *lse_part;            // [B][Hkv][G][ceil(NB / 16)][2] per-chunk (max, sum-exp) of e
  float *partial;             // [B][Hkv][n_splits] slices of [G][D] accumulators + [G] (max, sum) pairs
  int32_t *sel_idx;           // [B][Hkv][topk]
  int32_t *sel_cnt;           // [B][Hkv]
  float *scores;              // optional [B][Hkv][NB]
  float *out;                 // [B][Hq][D]
  float *lse;                 // optional [B][Hq]
};

// host-side count of kernel launches (see cobs_kernel_launches)
void count_launch(int n = 1);
void count_tcgen05_launch();

__device__ __forceinline__ void report(int32_t *status, int code) {
  if (status) atomicCAS(status, 0, code);
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// E2M1 code (bit 3 sign, bits 2..0 magnitude index) -> value, exact.
__device__ __forceinline__ float e2m1_value(uint32_t code) {
  uint32_t e = (code >> 1) & 3u, f = code & 1u;
  float mag = (e == 0) ? 0.5f * (float)f : __uint_as_float((e + 126u) << 23) * (1.0f + 0.5f * (float)f);
  return (code & 8u) ? -mag : mag;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// window start (tokens), aligned down to a block boundary
__device__ __forceinline__ int window_start(int T, int window, int L) {
  int a = T - window;
  if (a < 0) a = 0;
  return (a / L) * L;
}

}  // namespace cobs
