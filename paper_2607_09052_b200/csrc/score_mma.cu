// Fast scoring kernels for bf16 and FP4 summaries (step (b): Eq. trunc evaluated from the stored
// factors, Eq. gram).
//
// The summary stream is the HBM-bound part of scoring; the arithmetic is a skinny contraction
// [rows of mean / xi] x [q of the G heads of the group], K = D.  It runs on mma.sync m16n8k16 with
// fp32 accumulation so that the FP4 decode (integer ops) and the loads are all the CUDA cores do:
//   * a warp takes 16 consecutive blocks; thread (gid = lane / 4, tig = lane % 4) owns blocks
//     2 gid and 2 gid + 1, which are rows gid and gid + 8 of every A tile: tile 0 holds the 16 block
//     means, tile 1 + i holds factor i of the 16 blocks.  All results of one block therefore land in
//     one thread (heads 2 tig, 2 tig + 1) and no cross-lane reduction is needed.
//   * the k index of the contraction is permuted freely (the same permutation is applied when the
//     query fragments are built), so each thread reads its quarter of a row with 16-byte loads and
//     feeds the registers to the tensor core as they are.
//   * bf16 means and bf16 factors multiply the raw bf16 query (exact products); FP4 codes are turned
//     into f16 bit patterns (magnitude bits placed at exponent-LSBs / mantissa-MSB: value * 2^-14,
//     exact, subnormals included) and multiply the query scaled by a per-head power of two and
//     rounded to f16 (NT = 1), or split into an f16 high and low part for the fp32 subspace query
//     (NT = 2).
#include "common.cuh"

namespace cobs {

constexpr int kScoreWarps = 4;
constexpr int kScoreThreads = kScoreWarps * 32;
constexpr int kBlocksPerItem = kScoreWarps * 16;

__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint4 ldg_stream(const uint4 *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ uint32_t ldg_stream32(const uint32_t *p) {
  uint32_t v;
  asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];\n" : "=r"(v) : "l"(p));
  return v;
}

// Eight E2M1 codes in a word -> four f16x2 registers holding value * 2^-14.
// h[i] = (code i in the low half, code i + 4 in the high half).
__device__ __forceinline__ void decode_e2m1x8(uint32_t w, uint32_t (&h)[4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint32_t x = w << (12 - 4 * i);
    h[i] = (x & 0x80008000u) | ((x >> 3) & 0x0E000E00u);
  }
}
constexpr float kDecodeScale = 16384.0f;   // 2^14

__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t *>(&h);
}

// DT: COBS_SUMM_BF16 or COBS_SUMM_FP4_E2M1.  D: head dim.  WPT: 32-bit words of packed codes per
// thread per factor row (= Ds_pad / 32), FP4 only.  NT: number of f16 terms the query is split into.
template <int DT, int D, int WPT, int NT>
__global__ void __launch_bounds__(kScoreThreads, 4) score_mma_kernel(Params p, int items_per_unit, int total_items) {
  constexpr int KSM = D / 16;          // k-steps of the mean (and bf16 factor) tiles
  constexpr int KSQ = WPT * 2;         // k-steps of an FP4 factor tile
  constexpr int RU = 4;                // FP4 factor rows loaded ahead
  extern __shared__ float smem[];
  float *qs = smem;                    // [G][D]      q / sqrt(D)
  float *qt = smem + p.G * D;          // [G][Ds_pad] q~ (zero padded)
  __shared__ float mult[8];            // per head: factor applied to an FP4 tile result

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gid = lane >> 2, tig = lane & 3;
  const int G = p.G, r = p.r, NB = p.NB;
  const float inv_sqrt_d = 1.0f / sqrtf((float)D);
  const float ln_l = logf((float)p.L);

  const int per = (total_items + gridDim.x - 1) / gridDim.x;
  const int item0 = blockIdx.x * per, item1 = min(item0 + per, total_items);
  int cur_u = -1;
  uint32_t bm[KSM][2];                 // bf16 raw query fragments
  uint32_t bq[(DT == COBS_SUMM_FP4_E2M1) ? NT : 1][(DT == COBS_SUMM_FP4_E2M1) ? KSQ : 1][2];
  float m0 = 0.f, m1 = 0.f;

  for (int item = item0; item < item1; ++item) {
    const int u = item / items_per_unit, chunk = item - u * items_per_unit;
    const int b_idx = u / p.Hkv, h = u - b_idx * p.Hkv;
    const int n_sum = min(p.seq_lens[b_idx] / p.L, NB);
    if (u != cur_u) {
      cur_u = u;
      // ---- query fragments of this (sequence, KV head) ---------------------------------------
      const __nv_bfloat16 *qg = p.q + ((size_t)b_idx * p.Hq + h * G) * D;
#pragma unroll
      for (int m = 0; m < KSM / 2; ++m) {
        uint4 v = make_uint4(0, 0, 0, 0);
        if (gid < G) v = *reinterpret_cast<const uint4 *>(qg + gid * D + (tig + 4 * m) * 8);
        bm[2 * m][0] = v.x; bm[2 * m][1] = v.y; bm[2 * m + 1][0] = v.z; bm[2 * m + 1][1] = v.w;
      }
      if (DT == COBS_SUMM_FP4_E2M1) {
        __syncthreads();
        for (int i = tid; i < G * D; i += kScoreThreads) qs[i] = __bfloat162float(qg[i]) * inv_sqrt_d;
        __syncthreads();
        for (int i = tid; i < G * p.Ds_pad; i += kScoreThreads) {
          const int g = i / p.Ds_pad, s = i - g * p.Ds_pad;
          // full space: the raw bf16 query (exact in f16 after the power-of-two scaling below; the
          // 1/sqrt(D) factor is applied to the tile result instead); subspace: q~ = U_Q^T q / sqrt(D)
          float v = 0.f;
          if (s < p.Ds) {
            if (p.u_q) {
              const float *uq = p.u_q + (size_t)h * D * p.Ds + s;
              for (int d = 0; d < D; ++d) v = fmaf(uq[(size_t)d * p.Ds], qs[g * D + d], v);
            } else {
              v = __bfloat162float(qg[g * D + s]);
            }
          }
          qt[i] = v;
        }
        __syncthreads();
        // per-head power-of-two scale that brings max |q~| into [1, 2): keeps the f16 copy accurate
        if (warp < 2) {
          for (int g = warp; g < 8; g += 2) {
            float mx = 0.f;
            if (g < G)
              for (int s = lane; s < p.Ds_pad; s += 32) mx = fmaxf(mx, fabsf(qt[g * p.Ds_pad + s]));
            mx = warp_max(mx);
            int ex = 0;
            if (mx > 0.f) frexpf(mx, &ex);
            if (lane == 0) mult[g] = ldexpf(1.0f, ex - 1);     // = 1 / s_g
          }
        }
        __syncthreads();
        const float inv_s = (gid < G) ? 1.0f / mult[gid] : 0.f;  // s_g, exact power of two
#pragma unroll
        for (int j = 0; j < WPT; ++j) {
          float e[8];
#pragma unroll
          for (int n = 0; n < 8; ++n) e[n] = (gid < G) ? qt[gid * p.Ds_pad + tig * (WPT * 8) + j * 8 + n] * inv_s : 0.f;
#pragma unroll
          for (int t = 0; t < NT; ++t) {
            float hi[8];
#pragma unroll
            for (int n = 0; n < 8; ++n) {
              hi[n] = __half2float(__float2half_rn(e[n]));
              e[n] -= hi[n];
            }
            bq[t][2 * j][0] = pack_f16(hi[0], hi[4]); bq[t][2 * j][1] = pack_f16(hi[1], hi[5]);
            bq[t][2 * j + 1][0] = pack_f16(hi[2], hi[6]); bq[t][2 * j + 1][1] = pack_f16(hi[3], hi[7]);
          }
        }
        const float post = p.u_q ? kDecodeScale : kDecodeScale * inv_sqrt_d;
        m0 = (2 * tig < G) ? mult[2 * tig] * post : 0.f;
        m1 = (2 * tig + 1 < G) ? mult[2 * tig + 1] * post : 0.f;
      }
    }
    const int base = chunk * kBlocksPerItem + warp * 16;
    if (base >= n_sum) continue;
    const int bA = base + 2 * gid, bB = bA + 1;
    const size_t recA = (size_t)u * NB + min(bA, NB - 1), recB = (size_t)u * NB + min(bB, NB - 1);

    // ---- first-order term: the 16 block means against the raw bf16 query -------------------------
    float c[4] = {0.f, 0.f, 0.f, 0.f};
    {
      // 16-byte chunk tig + 4 m of each row: the four lanes of a quad read 64 contiguous bytes
      const uint4 *ma = reinterpret_cast<const uint4 *>((const __nv_bfloat16 *)p.mean + recA * D) + tig;
      const uint4 *mb = reinterpret_cast<const uint4 *>((const __nv_bfloat16 *)p.mean + recB * D) + tig;
      uint4 va[KSM / 2], vb[KSM / 2];
#pragma unroll
      for (int m = 0; m < KSM / 2; ++m) { va[m] = ldg_stream(ma + 4 * m); vb[m] = ldg_stream(mb + 4 * m); }
#pragma unroll
      for (int m = 0; m < KSM / 2; ++m) {
        mma_bf16(c, va[m].x, vb[m].x, va[m].y, vb[m].y, bm[2 * m][0], bm[2 * m][1]);
        mma_bf16(c, va[m].z, vb[m].z, va[m].w, vb[m].w, bm[2 * m + 1][0], bm[2 * m + 1][1]);
      }
    }
    const float fA0 = c[0] * inv_sqrt_d, fA1 = c[1] * inv_sqrt_d, fB0 = c[2] * inv_sqrt_d, fB1 = c[3] * inv_sqrt_d;
    float sA0 = 0.f, sA1 = 0.f, sB0 = 0.f, sB1 = 0.f;

    // ---- curvature term: sum_i (xi_i . q~)^2 ----------------------------------------------------------
    if (DT == COBS_SUMM_BF16) {
      const __nv_bfloat16 *xa = (const __nv_bfloat16 *)p.xi + recA * r * D + tig * 8;
      const __nv_bfloat16 *xb = (const __nv_bfloat16 *)p.xi + recB * r * D + tig * 8;
      for (int i = 0; i < r; ++i) {
        const uint4 *pa = reinterpret_cast<const uint4 *>(xa + (size_t)i * D);
        const uint4 *pb = reinterpret_cast<const uint4 *>(xb + (size_t)i * D);
        uint4 va[KSM / 2], vb[KSM / 2];
#pragma unroll
        for (int m = 0; m < KSM / 2; ++m) { va[m] = ldg_stream(pa + 4 * m); vb[m] = ldg_stream(pb + 4 * m); }
        float d[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int m = 0; m < KSM / 2; ++m) {
          mma_bf16(d, va[m].x, vb[m].x, va[m].y, vb[m].y, bm[2 * m][0], bm[2 * m][1]);
          mma_bf16(d, va[m].z, vb[m].z, va[m].w, vb[m].w, bm[2 * m + 1][0], bm[2 * m + 1][1]);
        }
        const float t0 = d[0] * inv_sqrt_d, t1 = d[1] * inv_sqrt_d, t2 = d[2] * inv_sqrt_d, t3 = d[3] * inv_sqrt_d;
        sA0 = fmaf(t0, t0, sA0); sA1 = fmaf(t1, t1, sA1); sB0 = fmaf(t2, t2, sB0); sB1 = fmaf(t3, t3, sB1);
      }
    } else {
      const int row_words = p.Ds_pad / 8;
      const uint32_t *xa = (const uint32_t *)p.xi + recA * r * row_words + tig * WPT;
      const uint32_t *xb = (const uint32_t *)p.xi + recB * r * row_words + tig * WPT;
      for (int i0 = 0; i0 < r; i0 += RU) {
        uint32_t wa[RU][WPT], wb[RU][WPT];
        float sca[RU], scb[RU];
#pragma unroll
        for (int k = 0; k < RU; ++k) {
          const int i = min(i0 + k, r - 1);
          if (WPT == 4) {
            const uint4 a = ldg_stream(reinterpret_cast<const uint4 *>(xa + (size_t)i * row_words));
            const uint4 b = ldg_stream(reinterpret_cast<const uint4 *>(xb + (size_t)i * row_words));
            wa[k][0] = a.x; wa[k][1 % WPT] = a.y; wa[k][2 % WPT] = a.z; wa[k][3 % WPT] = a.w;
            wb[k][0] = b.x; wb[k][1 % WPT] = b.y; wb[k][2 % WPT] = b.z; wb[k][3 % WPT] = b.w;
          } else {
#pragma unroll
            for (int j = 0; j < WPT; ++j) {
              wa[k][j] = ldg_stream32(xa + (size_t)i * row_words + j);
              wb[k][j] = ldg_stream32(xb + (size_t)i * row_words + j);
            }
          }
          if (p.scale_dtype == COBS_SCALE_FP16) {
            sca[k] = __half2float(((const __half *)p.scale)[recA * r + i]);
            scb[k] = __half2float(((const __half *)p.scale)[recB * r + i]);
          } else {
            sca[k] = ((const float *)p.scale)[recA * r + i];
            scb[k] = ((const float *)p.scale)[recB * r + i];
          }
        }
#pragma unroll
        for (int k = 0; k < RU; ++k) {
          if (i0 + k < r) {
            float d[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int j = 0; j < WPT; ++j) {
              uint32_t ha[4], hb[4];
              decode_e2m1x8(wa[k][j], ha);
              decode_e2m1x8(wb[k][j], hb);
#pragma unroll
              for (int t = 0; t < NT; ++t) {
                mma_f16(d, ha[0], hb[0], ha[1], hb[1], bq[t][2 * j][0], bq[t][2 * j][1]);
                mma_f16(d, ha[2], hb[2], ha[3], hb[3], bq[t][2 * j + 1][0], bq[t][2 * j + 1][1]);
              }
            }
            const float t0 = d[0] * (sca[k] * m0), t1 = d[1] * (sca[k] * m1);
            const float t2 = d[2] * (scb[k] * m0), t3 = d[3] * (scb[k] * m1);
            sA0 = fmaf(t0, t0, sA0); sA1 = fmaf(t1, t1, sA1); sB0 = fmaf(t2, t2, sB0); sB1 = fmaf(t3, t3, sB1);
          }
        }
      }
    }

    // ---- e[g][b] = ln L + first + second / 2 ------------------------------------------------------------
    const int g0 = 2 * tig, g1 = g0 + 1;
    float *e0 = p.e + ((size_t)u * G + g0) * NB, *e1 = p.e + ((size_t)u * G + g1) * NB;
    if (g0 < G) {
      if (bA < n_sum) e0[bA] = ln_l + fA0 + 0.5f * sA0;
      if (bB < n_sum) e0[bB] = ln_l + fB0 + 0.5f * sB0;
    }
    if (g1 < G) {
      if (bA < n_sum) e1[bA] = ln_l + fA1 + 0.5f * sA1;
      if (bB < n_sum) e1[bB] = ln_l + fB1 + 0.5f * sB1;
    }
  }
}

template <int DT, int D, int WPT, int NT>
static cudaError_t launch_one(const Params &p, cudaStream_t stream) {
  const int items_per_unit = (p.NB + kBlocksPerItem - 1) / kBlocksPerItem;
  const int total = items_per_unit * p.B * p.Hkv;
  int grid = 148 * 4;
  if (grid > total) grid = total;
  const size_t smem = (size_t)p.G * (D + p.Ds_pad) * sizeof(float);
  score_mma_kernel<DT, D, WPT, NT><<<grid, kScoreThreads, smem, stream>>>(p, items_per_unit, total);
  count_launch();
  return cudaGetLastError();
}

// Runs the tensor-core scoring kernel when the configuration is one it covers.
// *handled tells the caller whether it did.
cudaError_t launch_score_fast(const Params &p, cudaStream_t stream, bool *handled) {
  *handled = false;
  if (p.r < 1) return cudaSuccess;
  if (p.summ_dtype == COBS_SUMM_BF16 && p.u_q == nullptr) {
    *handled = true;
    return p.D == 128 ? launch_one<COBS_SUMM_BF16, 128, 1, 1>(p, stream) : launch_one<COBS_SUMM_BF16, 64, 1, 1>(p, stream);
  }
  if (p.summ_dtype == COBS_SUMM_FP4_E2M1 && p.Ds_pad % 32 == 0) {
    const int wpt = p.Ds_pad / 32;
    const bool sub = p.u_q != nullptr;
    *handled = true;
#define COBS_CASE(DD, WW)                                                                            \
  if (p.D == DD && wpt == WW)                                                                        \
    return sub ? launch_one<COBS_SUMM_FP4_E2M1, DD, WW, 2>(p, stream) : launch_one<COBS_SUMM_FP4_E2M1, DD, WW, 1>(p, stream);
    COBS_CASE(128, 4) COBS_CASE(128, 3) COBS_CASE(128, 2) COBS_CASE(128, 1)
    COBS_CASE(64, 2) COBS_CASE(64, 1)
#undef COBS_CASE
    *handled = false;
  }
  return cudaSuccess;
}

}  // namespace cobs
