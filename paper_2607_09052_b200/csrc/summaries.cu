// Step (a): per-block summaries.
//
//   mean   = (1/L) sum_t k_t                                  (Eq. cgf-cumulants)
//   K~     = rows k_t - mean  (times U_Q for the subspace descriptor)
//   C      = K~ K~^T / L      (L x L Gram matrix)             (Method, Cost: Gram trick)
//   (lambda_i, w_i) = eigenpairs of C by parallel cyclic Jacobi, lambda descending
//   xi_i   = K~^T w_i / sqrt(L)  = sqrt(lambda_i) u_i         (Eq. lowrank)
//   store  : fp32 | bf16 (RNE) | FP4 E2M1 + one scale per factor (Method, Quantization)
//
// One CTA per (sequence, KV head, block); everything stays in shared memory.  All reductions run in
// a fixed order, so the output bits are a function of the input bits only.
#include "common.cuh"

namespace cobs {

constexpr int kBuildThreads = 256;
constexpr int kMaxSweeps = 16;

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
  const int L = p.L, D = p.D, Dk = p.Ds, ldk = ((D > Dk) ? D : Dk) + 1, ldc = L + 1;
  float *Kc = sm;                        // [L][ldk]
  float *C = Kc + L * ldk;               // [L][ldc]
  float *W = C + L * ldc;                // [L][ldc]
  float *rot_c = W + L * ldc;            // [L / 2]
  float *rot_s = rot_c + L / 2;          // [L / 2]
  float *vec = rot_s + L / 2;            // [max(D, L)] scratch: mean, then eigenvalues
  float *red = vec + ((D > L) ? D : L);  // [2 * kBuildThreads / 32]
  float *wnorm = red + 2 * (kBuildThreads / 32);                      // [r] 1 / |w_i|
  int *top = reinterpret_cast<int *>(wnorm + COBS_MAX_RANK);          // [r]

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
        if (s < Dk) Kc[t * ldk + s] = o[i];
      }
    }
    __syncthreads();
  }

  // ---- Gram matrix C = K~ K~^T / L,  W = I ---------------------------------------------------------
  const float inv_l = 1.0f / (float)L;
  for (int c = tid; c < L * L; c += kBuildThreads) {
    const int i = c / L, j = c - i * L;
    if (j >= i) {
      float s = 0.f;
      for (int d = 0; d < Dk; ++d) s = fmaf(Kc[i * ldk + d], Kc[j * ldk + d], s);
      s *= inv_l;
      C[i * ldc + j] = s;
      C[j * ldc + i] = s;
    }
    W[i * ldc + j] = (i == j) ? 1.f : 0.f;
  }
  __syncthreads();

  // ---- parallel cyclic Jacobi (round-robin pairing), two-sided on C, rotations accumulated in W ----
  const int half = L / 2;
  float prev_off = INFINITY;
  for (int sweep = 0; sweep < kMaxSweeps; ++sweep) {
    // convergence: off-diagonal mass against diagonal mass (every thread computes the same totals)
    float off = 0.f, dia = 0.f;
    for (int c = tid; c < L * L; c += kBuildThreads) {
      const int i = c / L, j = c - i * L;
      const float x = C[i * ldc + j];
      if (i == j) dia = fmaf(x, x, dia); else off = fmaf(x, x, off);
    }
    off = warp_sum(off); dia = warp_sum(dia);
    __syncthreads();
    if (lane == 0) { red[warp] = off; red[NW + warp] = dia; }
    __syncthreads();
    float off_t = 0.f, dia_t = 0.f;
    for (int w = 0; w < NW; ++w) { off_t += red[w]; dia_t += red[NW + w]; }
    // done when the off-diagonal mass is at rounding level, or small and no longer shrinking
    if (off_t <= 1e-13f * dia_t || dia_t == 0.f) break;
    if (off_t <= 1e-10f * dia_t && off_t > 0.5f * prev_off) break;
    prev_off = off_t;

    for (int round = 0; round < L - 1; ++round) {
      if (tid < half) {
        int pi, qi;
        if (tid == 0) { pi = L - 1; qi = round; }
        else { pi = (round + tid) % (L - 1); qi = (round - tid + (L - 1)) % (L - 1); }
        if (pi > qi) { const int t = pi; pi = qi; qi = t; }
        const float app = C[pi * ldc + pi], aqq = C[qi * ldc + qi], apq = C[pi * ldc + qi];
        float cs = 1.f, sn = 0.f;
        if (fabsf(apq) > 1e-30f && fabsf(apq) > 1e-9f * sqrtf(fabsf(app * aqq))) {
          const float theta = (aqq - app) / (2.f * apq);
          const float tt = copysignf(1.f, theta) / (fabsf(theta) + sqrtf(fmaf(theta, theta, 1.f)));
          cs = rsqrtf(fmaf(tt, tt, 1.f));
          sn = tt * cs;
        }
        rot_c[tid] = cs; rot_s[tid] = sn;
      }
      __syncthreads();
      // rows: C <- J^T C
      for (int c = tid; c < half * L; c += kBuildThreads) {
        const int pr = c / L, j = c - pr * L;
        int pi, qi;
        if (pr == 0) { pi = L - 1; qi = round; }
        else { pi = (round + pr) % (L - 1); qi = (round - pr + (L - 1)) % (L - 1); }
        if (pi > qi) { const int t = pi; pi = qi; qi = t; }
        const float cs = rot_c[pr], sn = rot_s[pr];
        const float x = C[pi * ldc + j], y = C[qi * ldc + j];
        C[pi * ldc + j] = cs * x - sn * y;
        C[qi * ldc + j] = sn * x + cs * y;
      }
      __syncthreads();
      // columns: C <- C J,  W <- W J
      for (int c = tid; c < half * L; c += kBuildThreads) {
        const int pr = c / L, j = c - pr * L;
        int pi, qi;
        if (pr == 0) { pi = L - 1; qi = round; }
        else { pi = (round + pr) % (L - 1); qi = (round - pr + (L - 1)) % (L - 1); }
        if (pi > qi) { const int t = pi; pi = qi; qi = t; }
        const float cs = rot_c[pr], sn = rot_s[pr];
        float x = C[j * ldc + pi], y = C[j * ldc + qi];
        C[j * ldc + pi] = cs * x - sn * y;
        C[j * ldc + qi] = sn * x + cs * y;
        x = W[j * ldc + pi]; y = W[j * ldc + qi];
        W[j * ldc + pi] = cs * x - sn * y;
        W[j * ldc + qi] = sn * x + cs * y;
      }
      __syncthreads();
    }
  }
  __syncthreads();

  // ---- top-r eigenvalues (descending, lower index on ties), by warp 0 ------------------------------
  if (tid < L) vec[tid] = C[tid * ldc + tid];
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

  // ---- rotations in fp32 are orthogonal only to rounding: renormalise the chosen eigenvectors ------
  for (int i = warp; i < p.r; i += NW) {
    const int col = top[i];
    float s = 0.f;
    if (col >= 0)
      for (int t = lane; t < L; t += 32) s = fmaf(W[t * ldc + col], W[t * ldc + col], s);
    s = warp_sum(s);
    if (lane == 0) wnorm[i] = (col >= 0 && s > 0.f) ? 1.0f / sqrtf(s) : 0.f;
  }
  __syncthreads();

  // ---- factors xi_i = K~^T w_i / sqrt(L), written over C (its diagonal has been copied out) -----------
  float *xi_s = C;   // [r][Dk]
  const float inv_sqrt_l = 1.0f / sqrtf((float)L);
  for (int c = tid; c < p.r * Dk; c += kBuildThreads) {
    const int i = c / Dk, d = c - i * Dk;
    const int col = top[i];
    float s = 0.f;
    if (col >= 0)
      for (int t = 0; t < L; ++t) s = fmaf(Kc[t * ldk + d], W[t * ldc + col], s);
    xi_s[c] = (col >= 0) ? s * wnorm[i] * inv_sqrt_l : 0.f;
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
}

size_t build_smem_bytes(const Params &p) {
  const int L = p.L, ldk = ((p.D > p.Ds) ? p.D : p.Ds) + 1, ldc = L + 1;
  size_t f = (size_t)L * ldk + 2 * (size_t)L * ldc + L + ((p.D > L) ? p.D : L) + 2 * (kBuildThreads / 32) +
             COBS_MAX_RANK;
  return f * sizeof(float) + (size_t)(COBS_MAX_RANK + 1) * sizeof(int);
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

}  // namespace cobs
