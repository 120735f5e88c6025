// Step (a): per-block summaries.
//
//   mean   = (1/L) sum_t k_t                                  (Eq. cgf-cumulants)
//   K~     = rows k_t - mean  (times U_Q for the subspace descriptor)
//   C      = K~ K~^T / L      (L x L Gram matrix)             (Method, Cost: Gram trick)
//   (lambda_i, w_i) = eigenpairs of C, lambda descending
//   xi_i   = K~^T w_i / sqrt(L)  = sqrt(lambda_i) u_i         (Eq. lowrank)
// computed without forming C: one-sided (Hestenes) Jacobi rotates pairs of ROWS of K~ until all rows are mutually
// orthogonal.  The product of the rotations is W^T, so the rows end up as K~^T w_i = sqrt(L) xi_i with squared
// norms L lambda_i: the same O(L^2 D) work per sweep as the Gram route, the L x L matrices never exist, and a
// rotation is one dot product and one update of two rows held by a warp.
//   store  : fp32 | bf16 (RNE) | FP4 E2M1 + one scale per factor (Method, Quantization)
//
// One CTA per (sequence, KV head, block); everything stays in shared memory.  All reductions run in
// a fixed order, so the output bits are a function of the input bits only.
#include "common.cuh"

namespace cobs {

constexpr int kBuildThreads = 256;
constexpr int kMaxSweeps = 16;

// row stride of the centred keys in shared memory: a multiple of 4 floats (rows are read 16 bytes per lane), plus
// 4 so that consecutive rows start in different banks
__host__ __device__ inline int build_ldk(const Params &p) { return (((p.D > p.Ds) ? p.D : p.Ds) + 3) / 4 * 4 + 4; }

// --- FP4 quantiser -------------------------------------------------------------------------------
// code = sign bit of x, nearest E2M1 magnitude to |x| / scale with ties to the even mantissa bit.
__device__ __forceinline__ uint32_t e2m1_encode(float x, float scale) {
  const float t = __fdiv_rn(fabsf(x), scale);
  uint32_t m = 0;
  m += (t > 0.25f);
  m += (t >= 0.75f);
  m += (t > 1.25f);
  m += (t >= 1.75f);
  m += (t > 2.5f);
  m += (t >= 3.5f);
  m += (t > 5.0f);
  return (signbit(x) ? 8u : 0u) | m;
}

// Quantise one factor row held in `row` (Ds floats, shared or global) by one warp.
// codes: packed row of Ds_pad / 2 bytes (word-aligned); scale_out: element `vec` of the scale array.
__device__ void quantise_row_warp(const float *row, int Ds, int Ds_pad, uint32_t *codes_words, void *scale_arr,
                                  size_t vec, int scale_dtype, int lane) {
  float a = 0.f;
  for (int j = lane; j < Ds; j += 32) a = fmaxf(a, fabsf(row[j]));
  a = warp_max(a);
  float scale = __fdiv_rn(a, 6.0f);
  if (scale_dtype == COBS_SCALE_FP16) scale = __half2float(__float2half_rn(scale));
  for (int w = lane; w < Ds_pad / 8; w += 32) {
    uint32_t word = 0;
    if (scale > 0.f) {
#pragma unroll
      for (int n = 0; n < 8; ++n) {
        const int j = w * 8 + n;
        if (j < Ds) word |= e2m1_encode(row[j], scale) << (4 * n);
      }
    }
    codes_words[w] = word;
  }
  if (lane == 0) {
    if (scale_dtype == COBS_SCALE_FP16) ((__half *)scale_arr)[vec] = __float2half_rn(scale);
    else ((float *)scale_arr)[vec] = scale;
  }
}

__global__ void quantise_kernel(const float *xi, long long n_vectors, int Ds, int Ds_pad, int scale_dtype,
                                uint8_t *codes, void *scale) {
  const int lane = threadIdx.x & 31;
  const long long vec = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (vec >= n_vectors) return;
  quantise_row_warp(xi + vec * Ds, Ds, Ds_pad, reinterpret_cast<uint32_t *>(codes + vec * (Ds_pad / 2)), scale,
                    (size_t)vec, scale_dtype, lane);
}

// --- builder ---------------------------------------------------------------------------------------
// Shared memory:  Kc [L][Dk + 1]  centred (projected) keys, Dk = Ds
//                 C  [L][L + 1]   Gram matrix, rotated towards diagonal
//                 W  [L][L + 1]   accumulated rotations (columns = eigenvectors)
//                 small arrays
__global__ void __launch_bounds__(kBuildThreads) build_kernel(Params p, int block_begin, int block_end) {
  extern __shared__ __align__(16) float sm[];
  const int L = p.L, D = p.D, Dk = p.Ds, ldk = build_ldk(p);
  float *Kc = sm;                        // [L][ldk] centred keys; rotated in place into sqrt(L) xi rows
  float *nrm = Kc + L * ldk;             // [L] squared row norms
  float *vec = nrm + L;                  // [max(D, L)] scratch: mean, then eigenvalues
  float *red = vec + ((D > L) ? D : L);  // [kBuildThreads / 32]
  int *top = reinterpret_cast<int *>(red + kBuildThreads / 32);       // [r]
  int *flag = top + COBS_MAX_RANK;                                     // [1] a rotation was applied in this sweep

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int NW = kBuildThreads / 32;
  const int n_range = block_end - block_begin;
  const int blk = block_begin + (int)(blockIdx.x % n_range);
  const int u = blockIdx.x / n_range, b_idx = u / p.Hkv, h = u - b_idx * p.Hkv;
  const int T = p.seq_lens[b_idx];
  if (blk >= min(T / L, p.NB)) return;
  const size_t rec = (size_t)u * p.NB + blk;

  // ---- load the block's keys as fp32 -----------------------------------------------------------
  for (int c = tid; c < L * (D / 2); c += kBuildThreads) {
    const int t = c / (D / 2), dp = c - t * (D / 2);
    const int tok = blk * L + t;
    int pg = p.page_table[(size_t)b_idx * p.mpp + tok / p.P];
    uint32_t w = 0;
    if (pg < 0 || pg >= p.n_pages) report(p.status, COBS_ERR_BOUNDS);
    else w = reinterpret_cast<const uint32_t *>(p.k_pages)[((((size_t)pg * p.Hkv + h) * p.P + (tok % p.P)) * D) / 2 + dp];
    Kc[t * ldk + 2 * dp] = bf16_lo(w);
    Kc[t * ldk + 2 * dp + 1] = bf16_hi(w);
  }
  __syncthreads();

  // ---- mean (fixed summation order) and mean squared norm ---------------------------------------
  float sq = 0.f;
  if (tid < D) {
    float s = 0.f;
    for (int t = 0; t < L; ++t) { const float x = Kc[t * ldk + tid]; s += x; sq = fmaf(x, x, sq); }
    const float m = s / (float)L;
    vec[tid] = m;
    if (p.summ_dtype == COBS_SUMM_FP32) ((float *)p.mean)[rec * D + tid] = m;
    else ((__nv_bfloat16 *)p.mean)[rec * D + tid] = __float2bfloat16_rn(m);
  }
  sq = warp_sum(sq);
  if (lane == 0) red[warp] = sq;
  __syncthreads();
  float meansq = 0.f;
  for (int w = 0; w < NW; ++w) meansq += red[w];
  meansq /= (float)L;
  for (int c = tid; c < L * D; c += kBuildThreads) {
    const int t = c / D, d = c - t * D;
    Kc[t * ldk + d] -= vec[d];
  }
  __syncthreads();

  // ---- subspace projection K~ <- K~ U_Q, one warp per row, in place ----------------------------
  if (p.u_q) {
    const float *uq = p.u_q + (size_t)h * D * Dk;
    for (int t = warp; t < L; t += NW) {
      float rowreg[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) rowreg[i] = (lane + 32 * i < D) ? Kc[t * ldk + lane + 32 * i] : 0.f;
      float o[4] = {0.f, 0.f, 0.f, 0.f};
      for (int d = 0; d < D; ++d) {
        const float x = __shfl_sync(0xffffffffu, rowreg[d >> 5], d & 31);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int s = lane + 32 * i;
          if (s < Dk) o[i] = fmaf(x, uq[(size_t)d * Dk + s], o[i]);
        }
      }
      __syncwarp();
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int s = lane + 32 * i;
        if (s < D) Kc[t * ldk + s] = (s < Dk) ? o[i] : 0.f;        // columns past the subspace are cleared
      }
    }
    __syncthreads();
  }

  // ---- one-sided Jacobi on the rows of K~ (round-robin pairing: L / 2 disjoint pairs per round) --------
  // A half-warp owns a pair: lane l (of 16) holds columns 4 l .. 4 l + 3 and 64 + 4 l .. 64 + 4 l + 3 of both rows.
  // Pair slot s of round R joins rows (R + s) mod (L - 1) and (R - s) mod (L - 1); slot 0 joins row L - 1 and row R.
  const int half = L / 2, Dk4 = (Dk + 3) / 4 * 4;
  const int hw = lane >> 4, l16 = lane & 15;
  const bool col0 = 4 * l16 < Dk4, col1 = 64 + 4 * l16 < Dk4;
  constexpr int NI = 4;                                   // pair slots per half-warp per round (L <= 128)
  for (int sweep = 0; sweep < kMaxSweeps; ++sweep) {
    // exact squared norms at the start of every sweep (they are updated by formula inside it)
    for (int t = warp; t < L; t += NW) {
      float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
      if (4 * lane < Dk4) x = *reinterpret_cast<const float4 *>(Kc + t * ldk + 4 * lane);
      const float s = warp_sum(fmaf(x.x, x.x, fmaf(x.y, x.y, fmaf(x.z, x.z, x.w * x.w))));
      if (lane == 0) nrm[t] = s;
    }
    if (tid == 0) *flag = 0;
    __syncthreads();
    float nmax = 0.f;
    for (int t = 0; t < L; ++t) nmax = fmaxf(nmax, nrm[t]);
    const float floor2 = 1e-20f * nmax * nmax;            // rows below 1e-10 of the largest norm count as zero
    int pi_[NI], qi_[NI];                                 // this half-warp's pairs, advanced round by round
#pragma unroll
    for (int j = 0; j < NI; ++j) {
      const int slot = 2 * warp + hw + 2 * NW * j;
      pi_[j] = (slot == 0) ? L - 1 : slot;
      qi_[j] = (slot == 0) ? 0 : L - 1 - slot;
    }
    for (int round = 0; round < L - 1; ++round) {
#pragma unroll
      for (int j = 0; j < NI; ++j) {
        if (2 * NW * j >= half) break;                      // no slot of this index in a round (uniform)
        const int slot = 2 * warp + hw + 2 * NW * j;
        const bool on = slot < half;
        const int pi = on ? min(pi_[j], qi_[j]) : 0, qi = on ? max(pi_[j], qi_[j]) : 0;
        float4 x0 = make_float4(0.f, 0.f, 0.f, 0.f), x1 = x0, y0 = x0, y1 = x0;
        if (on && col0) {
          x0 = *reinterpret_cast<const float4 *>(Kc + pi * ldk + 4 * l16);
          y0 = *reinterpret_cast<const float4 *>(Kc + qi * ldk + 4 * l16);
        }
        if (on && col1) {
          x1 = *reinterpret_cast<const float4 *>(Kc + pi * ldk + 64 + 4 * l16);
          y1 = *reinterpret_cast<const float4 *>(Kc + qi * ldk + 64 + 4 * l16);
        }
        float g = fmaf(x0.x, y0.x, fmaf(x0.y, y0.y, fmaf(x0.z, y0.z, x0.w * y0.w))) +
                  fmaf(x1.x, y1.x, fmaf(x1.y, y1.y, fmaf(x1.z, y1.z, x1.w * y1.w)));
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) g += __shfl_xor_sync(0xffffffffu, g, o);
        const float a = nrm[pi], b = nrm[qi];
        __syncwarp();
        // rotate unless the rows are orthogonal to 4e-6 (the dot product of D terms is itself only good to ~1e-6)
        if (on && a * b > floor2 && g * g > 1.6e-11f * (a * b)) {
          // the angle may be approximate (any near-optimal rotation converges); c and s must satisfy
          // c^2 + s^2 = 1 to an unbiased rounding, or the row norms drift: c comes from a correctly rounded rsqrt
          const float zeta = __fdividef(b - a, 2.f * g);
          const float az = fabsf(zeta), rt = (az < 1e18f) ? sqrtf(fmaf(zeta, zeta, 1.f)) : az;
          const float tt = copysignf(__fdividef(1.f, az + rt), zeta);
          const float cs = __frsqrt_rn(fmaf(tt, tt, 1.f)), sn = tt * cs;
          if (col0) {
            *reinterpret_cast<float4 *>(Kc + pi * ldk + 4 * l16) =
                make_float4(cs * x0.x - sn * y0.x, cs * x0.y - sn * y0.y, cs * x0.z - sn * y0.z, cs * x0.w - sn * y0.w);
            *reinterpret_cast<float4 *>(Kc + qi * ldk + 4 * l16) =
                make_float4(sn * x0.x + cs * y0.x, sn * x0.y + cs * y0.y, sn * x0.z + cs * y0.z, sn * x0.w + cs * y0.w);
          }
          if (col1) {
            *reinterpret_cast<float4 *>(Kc + pi * ldk + 64 + 4 * l16) =
                make_float4(cs * x1.x - sn * y1.x, cs * x1.y - sn * y1.y, cs * x1.z - sn * y1.z, cs * x1.w - sn * y1.w);
            *reinterpret_cast<float4 *>(Kc + qi * ldk + 64 + 4 * l16) =
                make_float4(sn * x1.x + cs * y1.x, sn * x1.y + cs * y1.y, sn * x1.z + cs * y1.z, sn * x1.w + cs * y1.w);
          }
          if (l16 == 0) { nrm[pi] = fmaxf(a - tt * g, 0.f); nrm[qi] = b + tt * g; *flag = 1; }
        }
        // next round's rows of this slot
        if (slot == 0) { qi_[j] = round + 1; }
        else {
          pi_[j] = (pi_[j] + 1 == L - 1) ? 0 : pi_[j] + 1;
          qi_[j] = (qi_[j] + 1 == L - 1) ? 0 : qi_[j] + 1;
        }
      }
      __syncthreads();
    }
    if (*flag == 0) break;
    __syncthreads();
  }
  __syncthreads();

  // ---- eigenvalues = squared row norms / L; the top r (descending, lower index on ties), by warp 0 -----
  for (int t = warp; t < L; t += NW) {
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    if (4 * lane < Dk4) x = *reinterpret_cast<const float4 *>(Kc + t * ldk + 4 * lane);
    const float s = warp_sum(fmaf(x.x, x.x, fmaf(x.y, x.y, fmaf(x.z, x.z, x.w * x.w))));
    if (lane == 0) vec[t] = s / (float)L;
  }
  __syncthreads();
  if (warp == 0) {
    for (int i = 0; i < p.r; ++i) {
      float best = -INFINITY; int bi = 0x7fffffff;
      for (int j = lane; j < L; j += 32) {
        const float v = vec[j];
        if (v > best) { best = v; bi = j; }
      }
      for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
        if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
      }
      if (lane == 0) {
        if (i < L) { top[i] = (best > 1e-12f * meansq) ? bi : -1; vec[bi] = -INFINITY; }
        else top[i] = -1;
      }
      __syncwarp();
    }
  }
  __syncthreads();

  // ---- factors xi_i = (rotated row) / sqrt(L), gathered into the first rows' place holder ----------------
  float *xi_s = nrm + L + ((D > L) ? D : L) + kBuildThreads / 32 + 2 * COBS_MAX_RANK;   // [r][Dk] after the small arrays
  const float inv_sqrt_l = 1.0f / sqrtf((float)L);
  for (int c = tid; c < p.r * Dk; c += kBuildThreads) {
    const int i = c / Dk, d = c - i * Dk;
    const int col = top[i];
    xi_s[c] = (col >= 0) ? Kc[col * ldk + d] * inv_sqrt_l : 0.f;
  }
  __syncthreads();

  // ---- sign rule + store, one warp per factor ---------------------------------------------------------
  for (int i = warp; i < p.r; i += NW) {
    float *row = xi_s + i * Dk;
    float best = -1.f; int bi = 0x7fffffff;
    for (int j = lane; j < Dk; j += 32) {
      const float v = fabsf(row[j]);
      if (v > best) { best = v; bi = j; }
    }
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ov > best || (ov == best && oi < bi)) { best = ov; bi = oi; }
    }
    const bool flip = row[bi] < 0.f;
    __syncwarp();
    if (flip)
      for (int j = lane; j < Dk; j += 32) row[j] = -row[j];
    __syncwarp();
    const size_t v = rec * p.r + i;
    if (p.summ_dtype == COBS_SUMM_FP32) {
      for (int j = lane; j < Dk; j += 32) ((float *)p.xi)[v * Dk + j] = row[j];
    } else if (p.summ_dtype == COBS_SUMM_BF16) {
      for (int j = lane; j < Dk; j += 32) ((__nv_bfloat16 *)p.xi)[v * Dk + j] = __float2bfloat16_rn(row[j]);
    } else {
      quantise_row_warp(row, Dk, p.Ds_pad, reinterpret_cast<uint32_t *>((uint8_t *)p.xi + v * (p.Ds_pad / 2)),
                        p.scale, v, p.scale_dtype, lane);
    }
  }

  // ---- diagonal of the third cumulant in the stored eigenbasis (Appendix, Cheap diagonal skew) -------------------
  // c_i = g_i / lam_i^(3/2) with g_i = 1/L sum_t (u_i . (k_t - kbar))^3 and xi_i = sqrt(lam_i) u_i, i.e.
  // c_i = [1/L sum_t p_t^3] / lam_i^3 for p_t = xi_i . (k_t - kbar).  The projections are taken on the raw keys and
  // centred afterwards (xi_i . kbar is their mean), from the unrounded, sign-fixed factors.  Full space only (Dk = D).
  if (p.skew) {
    __syncthreads();
    float *proj = Kc;                            // [r][L]: the rotated rows are no longer needed
    for (int t = warp; t < L; t += NW) {
      const int tok = blk * L + t;
      const int pg = p.page_table[(size_t)b_idx * p.mpp + tok / p.P];
      const bool okp = pg >= 0 && pg < p.n_pages;           // a bad page was reported when the keys were loaded
      const __nv_bfloat16 *kr = p.k_pages + (((size_t)(okp ? pg : 0) * p.Hkv + h) * p.P + (tok % p.P)) * D;
      float kreg[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) kreg[i] = (okp && lane + 32 * i < D) ? __bfloat162float(kr[lane + 32 * i]) : 0.f;
      for (int f = 0; f < p.r; ++f) {
        float a = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (lane + 32 * i < D) a = fmaf(kreg[i], xi_s[f * Dk + lane + 32 * i], a);
        a = warp_sum(a);
        if (lane == 0) proj[f * L + t] = a;
      }
    }
    __syncthreads();
    for (int f = warp; f < p.r; f += NW) {
      const float *row = xi_s + f * Dk;
      float lam = 0.f, sum = 0.f;
      for (int j = lane; j < Dk; j += 32) lam = fmaf(row[j], row[j], lam);
      for (int t = lane; t < L; t += 32) sum += proj[f * L + t];
      lam = warp_sum(lam);
      const float m = warp_sum(sum) / (float)L;
      float c3 = 0.f;
      for (int t = lane; t < L; t += 32) {
        const float x = proj[f * L + t] - m;
        c3 = fmaf(x * x, x, c3);
      }
      c3 = warp_sum(c3) / (float)L;
      if (lane == 0) p.skew[rec * p.r + f] = (top[f] >= 0 && lam > 0.f) ? c3 / (lam * lam * lam) : 0.f;
    }
  }
}

size_t build_smem_bytes(const Params &p) {
  const int L = p.L;
  size_t f = (size_t)L * build_ldk(p) + L + ((p.D > L) ? p.D : L) + kBuildThreads / 32 + 2 * COBS_MAX_RANK +
             (size_t)COBS_MAX_RANK * p.Ds;
  return f * sizeof(float);
}

cudaError_t launch_build(const Params &p, int block_begin, int block_end, cudaStream_t stream) {
  const int n_range = block_end - block_begin;
  if (n_range <= 0) return cudaSuccess;
  const size_t smem = build_smem_bytes(p);
  cudaError_t e = cudaFuncSetAttribute(build_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const long long n_cta = (long long)p.B * p.Hkv * n_range;
  build_kernel<<<(unsigned)n_cta, kBuildThreads, smem, stream>>>(p, block_begin, block_end);
  count_launch();
  return cudaGetLastError();
}

// One new token per sequence into the paged cache: 16 bytes per thread, one CTA per (sequence, KV head); the
// CTAs of KV head 0 also advance the sequence lengths once every CTA of the sequence has read the old one.
__global__ void append_kernel(Params p, const __nv_bfloat16 *k_new, const __nv_bfloat16 *v_new, __nv_bfloat16 *k_pages,
                              __nv_bfloat16 *v_pages, int32_t *seq_lens, const int32_t *old_lens) {
  const int b = blockIdx.x / p.Hkv, h = blockIdx.x - b * p.Hkv;
  const int T = old_lens[b];
  if (T < 0 || T >= p.mpp * p.P) { if (threadIdx.x == 0) report(p.status, COBS_ERR_BOUNDS); return; }
  const int pg = p.page_table[(size_t)b * p.mpp + T / p.P];
  if (pg < 0 || pg >= p.n_pages) { if (threadIdx.x == 0) report(p.status, COBS_ERR_BOUNDS); return; }
  const size_t dst = (((size_t)pg * p.Hkv + h) * p.P + (T % p.P)) * p.D, src = ((size_t)b * p.Hkv + h) * p.D;
  for (int i = threadIdx.x; i < p.D / 8; i += blockDim.x) {
    reinterpret_cast<uint4 *>(k_pages + dst)[i] = reinterpret_cast<const uint4 *>(k_new + src)[i];
    reinterpret_cast<uint4 *>(v_pages + dst)[i] = reinterpret_cast<const uint4 *>(v_new + src)[i];
  }
  if (h == 0 && threadIdx.x == 0) seq_lens[b] = T + 1;
}

// old_lens: a snapshot of the lengths taken on the stream before the launch (the kernel reads the snapshot and
// writes the live array, so no CTA can see a length another CTA has already advanced).
cudaError_t launch_append(const Params &p, const void *k_new, const void *v_new, void *k_pages, void *v_pages, int32_t *seq_lens,
                          int32_t *old_lens, cudaStream_t stream) {
  cudaError_t e = cudaMemcpyAsync(old_lens, seq_lens, sizeof(int32_t) * p.B, cudaMemcpyDeviceToDevice, stream);
  if (e != cudaSuccess) return e;
  append_kernel<<<p.B * p.Hkv, 32, 0, stream>>>(p, static_cast<const __nv_bfloat16 *>(k_new), static_cast<const __nv_bfloat16 *>(v_new),
                                                 static_cast<__nv_bfloat16 *>(k_pages), static_cast<__nv_bfloat16 *>(v_pages), seq_lens,
                                                 old_lens);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_quantise(const float *xi, long long n_vectors, int Ds, int Ds_pad, int scale_dtype, void *codes,
                            void *scale, cudaStream_t stream) {
  if (n_vectors <= 0) return cudaSuccess;
  const int wpb = 8;
  quantise_kernel<<<(unsigned)((n_vectors + wpb - 1) / wpb), wpb * 32, 0, stream>>>(xi, n_vectors, Ds, Ds_pad,
                                                                                 scale_dtype, (uint8_t *)codes, scale);
  count_launch();
  return cudaGetLastError();
}

// The GPU's own float -> E2M1 conversion instruction, one code per input value: what the threshold chain of
// e2m1_encode is checked against (a test hook; nothing on the path calls it).
__global__ void hw_e2m1_kernel(const float *x, long long n, uint8_t *codes) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  uint32_t r;
  // the instruction packs two codes in a byte; the partner value is +0 (code 0), so the OR of the byte's two
  // nibbles is the code of x[i] whichever nibble the instruction puts it in
  asm("{\n .reg .b8 t;\n cvt.rn.satfinite.e2m1x2.f32 t, %1, %2;\n cvt.u32.u8 %0, t;\n}\n" : "=r"(r) : "f"(x[i]), "f"(0.0f));
  codes[i] = (uint8_t)(((r >> 4) | r) & 15u);
}

}  // namespace cobs

extern "C" int32_t cobs_hw_e2m1_codes(const float *x, int64_t n, uint8_t *codes, void *stream) {
  if (!x || !codes || n < 0) return COBS_ERR_INVALID_ARG;
  if (n == 0) return COBS_OK;
  if (n > ((int64_t)1 << 31)) return COBS_ERR_UNSUPPORTED;
  cobs::hw_e2m1_kernel<<<(unsigned)((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(x, n, codes);
  cobs::count_launch();
  return cudaGetLastError() == cudaSuccess ? COBS_OK : COBS_ERR_CUDA;
}
