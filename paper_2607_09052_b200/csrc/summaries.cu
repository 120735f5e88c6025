// Step (a): per-block summaries.
//
//   mean   = (1/L) sum_t k_t                                  (Eq. cgf-cumulants)
//   K~     = rows k_t - mean  (times U_Q for the subspace descriptor)
//   C      = K~ K~^T / L      (L x L Gram matrix)             (Method, Cost: Gram trick)
//   (lambda_i, w_i) = eigenpairs of C, lambda descending
//   xi_i   = K~^T w_i / sqrt(L)  = sqrt(lambda_i) u_i         (Eq. lowrank)
// Only the r largest eigenpairs are wanted: C is tridiagonalised by Householder reflections, the r largest
// eigenvalues are located by Sturm counts, their eigenvectors come from inverse iteration and are carried back
// through the reflections (the builder's comment below has the details).  A block whose eigenvectors fail their
// residual check is solved by one-sided (Hestenes) Jacobi instead: pairs of ROWS of K~ are rotated until all rows
// are mutually orthogonal; the product of the rotations is W^T, so the rows end up as K~^T w_i = sqrt(L) xi_i with
// squared norms L lambda_i.
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

// --- Gram matrix and Householder tridiagonalisation in registers -----------------------------------------------
// The 256 threads form a 16 x 16 grid; thread (ty, tx) keeps the elements (ty + 16 a, tx + 16 b) of the symmetric
// matrix, a, b < TL = L / 16, in registers (a cyclic layout: the trailing matrix of every step is spread evenly, and
// whole groups a or b that lie in the finished part are skipped).  Step k: the 16 threads that own row k have left
// its reflector v in shared memory, the threads multiply their tiles by v and reduce over the 16 threads of
// a matrix row (p = beta A v), then apply A <- A - v w^T - w v^T with w = p - (beta v^T p / 2) v.  The threads that
// own row k + 1 publish their rows and form the next reflector.  Two barriers per step.
// Out: dd / ee (diagonal and off-diagonal of T), bet (2 / v^T v, 0 where a row needed no reflector), and the
// reflectors packed row after row in Ct (row k: its L - 1 - k elements right of the diagonal).
__host__ __device__ constexpr int refl_offset(int k, int L) { return k * (L - 1) - k * (k - 1) / 2; }

template <int TL>
__device__ __forceinline__ void gram_tridiag(const float *__restrict__ Kc, int ldk, int Dk4, float *__restrict__ Ct,
                                             float *__restrict__ dd, float *__restrict__ ee, float *__restrict__ bet,
                                             float *__restrict__ xrow /* [2][TL][L] */, float *__restrict__ dgl,
                                             float *__restrict__ pp, float *__restrict__ kpart, int tid, int warp, int lane) {
  constexpr int L = 16 * TL, NW = kBuildThreads / 32;
  const int ty = tid >> 4, tx = tid & 15;
  float A[TL][TL];
#pragma unroll
  for (int a = 0; a < TL; ++a)
#pragma unroll
    for (int b = 0; b < TL; ++b) A[a][b] = 0.f;
  for (int d = 0; d < Dk4; d += 4) {
    float4 ra[TL];
#pragma unroll
    for (int a = 0; a < TL; ++a) ra[a] = *reinterpret_cast<const float4 *>(Kc + (ty + 16 * a) * ldk + d);
#pragma unroll
    for (int b = 0; b < TL; ++b) {
      const float4 rb = *reinterpret_cast<const float4 *>(Kc + (tx + 16 * b) * ldk + d);
#pragma unroll
      for (int a = 0; a < TL; ++a)
        A[a][b] = fmaf(ra[a].w, rb.w, fmaf(ra[a].z, rb.z, fmaf(ra[a].y, rb.y, fmaf(ra[a].x, rb.x, A[a][b]))));
    }
  }
  __syncthreads();                                    // the keys have been read: their place is free for the reflectors
  // The 16 threads that own row `row` publish their TL rows (zeros up to the diagonal, column `row` included), then
  // turn the published row into its reflector v: sigma = |x|^2 over the 16 lanes, alpha = -sign(x0) sqrt(sigma),
  // beta = 1 / (sigma - x0 alpha), v = x with x0 - alpha as its first element.  bet[row] = 0: the row needs no reflector.
  auto publish = [&](int row, float *xn) {
    if (ty != (row & 15)) return;
    const unsigned mask = 0xffffu << (16 * (ty & 1));          // the half-warp of these threads
#pragma unroll
    for (int a = 0; a < TL; ++a)
#pragma unroll
      for (int b = 0; b < TL; ++b) xn[a * L + tx + 16 * b] = (tx + 16 * b > row) ? A[a][b] : 0.f;
    if (row + 2 >= L) return;                                  // the last two rows are only read, not reduced
    __syncwarp(mask);
    float *xr = xn + (row >> 4) * L;
    float sg = 0.f;
#pragma unroll
    for (int b = 0; b < TL; ++b) { const float x = xr[tx + 16 * b]; sg = fmaf(x, x, sg); }
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) sg += __shfl_xor_sync(mask, sg, o);
    const float x0 = xr[row + 1];
    const bool refl = sg - x0 * x0 > 1e-30f + 1e-14f * sg;
    const float alpha = refl ? -copysignf(sqrtf(sg), x0) : x0;
    const float beta = refl ? 1.0f / (sg - x0 * alpha) : 0.f;
    __syncwarp(mask);                                          // everyone has read x0
    if (tx == 0) {
      ee[row] = alpha; bet[row] = beta;
      if (refl) xr[row + 1] = x0 - alpha;
    }
  };
  publish(0, xrow);
  if (ty == tx) {
#pragma unroll
    for (int a = 0; a < TL; ++a) dgl[ty + 16 * a] = A[a][a];
  }
  __syncthreads();
  for (int k = 0; k + 2 < L; ++k) {
    const float *xc = xrow + (k & 1) * TL * L + (k >> 4) * L;      // the reflector of row k
    float *xn = xrow + ((k + 1) & 1) * TL * L;
    const int amin = (k + 1) >> 4;                    // groups below hold finished rows / columns only
    const float beta = bet[k];
    if (beta != 0.f) {                                // (uniform)
      float vr[TL], vc[TL];
#pragma unroll
      for (int a = 0; a < TL; ++a) { vr[a] = xc[ty + 16 * a]; vc[a] = xc[tx + 16 * a]; }
      if (ty == 0) {
#pragma unroll
        for (int b = 0; b < TL; ++b)
          if (tx + 16 * b > k) Ct[refl_offset(k, L) + tx + 16 * b - k - 1] = vc[b];
      }
      float part[TL];
#pragma unroll
      for (int a = 0; a < TL; ++a) {
        part[a] = 0.f;
        if (a >= amin) {                                // (uniform)
          float sp = 0.f;
#pragma unroll
          for (int b = 0; b < TL; ++b) sp = fmaf(A[a][b], vc[b], sp);
#pragma unroll
          for (int o = 8; o > 0; o >>= 1) sp += __shfl_xor_sync(0xffffffffu, sp, o);
          part[a] = (ty + 16 * a > k) ? beta * sp : 0.f;
        }
      }
      float kp = 0.f;                                   // this warp's share of v^T p
#pragma unroll
      for (int a = 0; a < TL; ++a) kp = fmaf(vr[a], part[a], kp);
      kp += __shfl_xor_sync(0xffffffffu, kp, 16);
      if (tx == 0) {
#pragma unroll
        for (int a = 0; a < TL; ++a) pp[ty + 16 * a] = part[a];
      }
      if (lane == 0) kpart[warp] = kp;
      __syncthreads();
      float kk = 0.f;
#pragma unroll
      for (int w = 0; w < NW; ++w) kk += kpart[w];
      kk *= 0.5f * beta;
      float wc[TL];
#pragma unroll
      for (int a = 0; a < TL; ++a) wc[a] = pp[tx + 16 * a] - kk * vc[a];
#pragma unroll
      for (int a = 0; a < TL; ++a) {
        if (a >= amin) {                                // (uniform)
          const float wra = part[a] - kk * vr[a];
#pragma unroll
          for (int b = 0; b < TL; ++b) A[a][b] = fmaf(-wra, vc[b], fmaf(-vr[a], wc[b], A[a][b]));
        }
      }
    } else if (ty == 0) {
#pragma unroll
      for (int b = 0; b < TL; ++b)
        if (tx + 16 * b > k) Ct[refl_offset(k, L) + tx + 16 * b - k - 1] = 0.f;
    }
    publish(k + 1, xn);
    if (ty == tx) {
#pragma unroll
      for (int a = 0; a < TL; ++a) dgl[ty + 16 * a] = A[a][a];
    }
    __syncthreads();
  }
  if (tid < L) dd[tid] = dgl[tid];
  if (tid == 0) { ee[L - 2] = xrow[((L - 2) & 1) * TL * L + ((L - 2) >> 4) * L + L - 1]; ee[L - 1] = 0.f; }   // row L - 2 was the last one published
  __syncthreads();
}

// w = Q z for the eigenvectors z of T (one warp per vector, the vector in registers): the reflectors in reverse order.
template <int TL>
__device__ __forceinline__ void back_transform(float *__restrict__ Z, const float *__restrict__ Ct,
                                               const float *__restrict__ bet, const int *__restrict__ top, int r_eff,
                                               int warp, int lane) {
  constexpr int L = 16 * TL, NZ = (L + 31) / 32, NW = kBuildThreads / 32;
  for (int j = warp; j < r_eff; j += NW) {
    if (top[j] < 0) continue;
    float z[NZ];
#pragma unroll
    for (int i = 0; i < NZ; ++i) z[i] = (lane + 32 * i < L) ? Z[j * L + lane + 32 * i] : 0.f;
#pragma unroll 2
    for (int k = L - 3; k >= 0; --k) {
      const float beta = bet[k];
      const float *vrow = Ct + refl_offset(k, L) - k - 1;
      float v[NZ], dt = 0.f;
#pragma unroll
      for (int i = 0; i < NZ; ++i) {
        const int c = lane + 32 * i;
        v[i] = (c > k && c < L) ? vrow[c] : 0.f;
        dt = fmaf(v[i], z[i], dt);
      }
      dt = beta * warp_sum(dt);
#pragma unroll
      for (int i = 0; i < NZ; ++i) z[i] -= dt * v[i];
    }
#pragma unroll
    for (int i = 0; i < NZ; ++i)
      if (lane + 32 * i < L) Z[j * L + lane + 32 * i] = z[i];
  }
}

// --- builder ---------------------------------------------------------------------------------------
// One CTA per (sequence, KV head, block).  Only the r <= 16 largest eigenpairs of the L x L Gram matrix are wanted
// (Method, "Low-rank covariance compression"; Method, "Cost": Gram trick), so the block is solved the way dense
// symmetric eigen-solvers do it when few pairs are asked for:
//   G = K~ K~^T (fp32)  ->  Householder tridiagonalisation  T = Q^T G Q  ->  the r largest eigenvalues of T by Sturm
//   counts (each warp narrows one eigenvalue 32 ways per step)  ->  their eigenvectors by inverse iteration (one
//   pivoted factorisation of T - lambda I per vector, reused by three solves, Gram-Schmidt between the solves so that
//   vectors of close eigenvalues separate)  ->  w = Q z  ->  xi = K~^T w / sqrt(L).
// About L^3 + r L D operations instead of the ~10 sweeps x L^2 D / 2 of a Jacobi solve.  Every vector's residual
// |T z - lambda z| is checked; a block that fails the check is solved again by the one-sided Jacobi method that was
// this kernel's first form (rotating the rows of K~ until they are mutually orthogonal), which converges always.
// solver = 1 takes the Jacobi route for every block (tests).
// Shared memory: the centred keys Kc [L][ldk] are read by the Gram product only, so the reflectors and the
// factorisation scratch of the inverse iteration take their place; the keys are loaded again (from L2, mostly) for
// the last product.  What outlives that sits behind: small arrays, factor rows, T, the published rows, eigenvectors.
struct BuildSmem {
  int region, nrm, vec, red, top, xi, dd, xrow, lam, Z, total;      // offsets in floats
};
__host__ __device__ inline BuildSmem build_smem_layout(const Params &p) {
  const int L = p.L, D = p.D, NW = kBuildThreads / 32;
  const int keys = L * build_ldk(p) + (p.u_q ? COBS_MAX_RANK * D : 0);          // + K~^T w in the full space (subspace form)
  const int solve = L * (L - 1) / 2 + NW * 5 * L;
  BuildSmem o;
  o.region = (((keys > solve) ? keys : solve) + 3) / 4 * 4;
  o.nrm = o.region;
  o.vec = o.nrm + L;
  o.red = o.vec + ((D > L) ? D : L);
  o.top = o.red + NW;
  o.xi = o.top + 2 * COBS_MAX_RANK;
  o.dd = o.xi + COBS_MAX_RANK * p.Ds;
  o.xrow = o.dd + 6 * L;
  o.lam = o.xrow + 2 * (L / 16) * L;
  o.Z = o.lam + 64;
  o.total = o.Z + COBS_MAX_RANK * L;
  return o;
}

template <int TL>
__global__ void __launch_bounds__(kBuildThreads, (TL == 8) ? 2 : 4) build_kernel(Params p, int block_begin, int block_end, int solver) {
  extern __shared__ __align__(16) float sm[];
  constexpr int L = 16 * TL;
  const int D = p.D, Dk = p.Ds, ldk = build_ldk(p);
  const BuildSmem lay = build_smem_layout(p);
  float *Kc = sm;                        // [L][ldk] centred keys (Jacobi: rotated in place into sqrt(L) xi rows)
  float *nrm = sm + lay.nrm;             // [L] squared row norms (Jacobi)
  float *vec = sm + lay.vec;             // [max(D, L)] the mean (Jacobi: then the eigenvalues)
  float *red = sm + lay.red;             // [kBuildThreads / 32]
  int *top = reinterpret_cast<int *>(sm + lay.top);                    // [16] factor i is kept (>= 0) or null (-1)
  int *flag = top + COBS_MAX_RANK;                                     // [1] a rotation was applied in this sweep
  float *xi_s = sm + lay.xi;             // [r][Dk] the factors

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int NW = kBuildThreads / 32;
  const int n_range = block_end - block_begin;
  const int blk = block_begin + (int)(blockIdx.x % n_range);
  const int u = blockIdx.x / n_range, b_idx = u / p.Hkv, h = u - b_idx * p.Hkv;
  const int T = p.seq_lens[b_idx];
  if (blk >= min(T / L, p.NB)) return;
  const size_t rec = (size_t)u * p.NB + blk;
  const int Dk4 = (Dk + 3) / 4 * 4;
  const float inv_sqrt_l = 1.0f / sqrtf((float)L);
  float meansq = 0.f;

  // Kc <- the block's keys as fp32, minus their mean; first: the mean (fixed summation order) is computed and stored,
  // and the mean squared norm; project: K~ <- K~ U_Q (one warp per row, in place).
  auto load_keys = [&](bool first, bool project) {
#pragma unroll 4
    for (int c = tid; c < L * (D / 8); c += kBuildThreads) {        // 16 bytes (8 keys' elements) per thread and turn
      const int t = c / (D / 8), d8 = c - t * (D / 8);
      const int tok = blk * L + t;
      const int pg = p.page_table[(size_t)b_idx * p.mpp + tok / p.P];
      uint4 w = make_uint4(0u, 0u, 0u, 0u);
      if (pg < 0 || pg >= p.n_pages) report(p.status, COBS_ERR_BOUNDS);
      else w = reinterpret_cast<const uint4 *>(p.k_pages + (((size_t)pg * p.Hkv + h) * p.P + (tok % p.P)) * D)[d8];
      float *dst = Kc + t * ldk + 8 * d8;
      *reinterpret_cast<float4 *>(dst) = make_float4(bf16_lo(w.x), bf16_hi(w.x), bf16_lo(w.y), bf16_hi(w.y));
      *reinterpret_cast<float4 *>(dst + 4) = make_float4(bf16_lo(w.z), bf16_hi(w.z), bf16_lo(w.w), bf16_hi(w.w));
    }
    __syncthreads();
    if (first) {
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
      for (int w = 0; w < NW; ++w) meansq += red[w];
      meansq /= (float)L;
    }
    for (int c = tid; c < L * D; c += kBuildThreads) {
      const int t = c / D, d = c - t * D;
      Kc[t * ldk + d] -= vec[d];
    }
    __syncthreads();
    if (project && p.u_q) {
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
  };
  load_keys(true, true);

  // ---- the tridiagonal route ------------------------------------------------------------------------------------------
  float *Ct = sm;                        // [L (L - 1) / 2] the reflectors, in the keys' place
  float *scr = Ct + L * (L - 1) / 2;     // [NW][5][L] factorisation of T - lambda I, per warp
  float *dd = sm + lay.dd;               // [L] diagonal of T
  float *ee = dd + L;                    // [L] off-diagonal of T (ee[k] joins k and k + 1)
  float *bet = ee + L;                   // [L] 2 / v^T v of reflector k (0: none)
  float *e2 = bet + L;                   // [L] ee^2
  float *dgl = e2 + L, *pp = dgl + L;    // [L] each: the diagonal as the reduction goes; beta A v
  float *xrow = sm + lay.xrow;           // [2][L / 16][L] the rows of the threads that own the row being reduced (two buffers)
  float *lam = sm + lay.lam;             // [16] eigenvalues of G, descending; [16] shifts; [8] bounds; [8] flags; [8] shares of v^T p
  float *Z = sm + lay.Z;                 // [16][L] eigenvectors of T, then of G
  const int r_eff = min(p.r, L);
  int *s_fallback = reinterpret_cast<int *>(lam + 40);
  bool use_jacobi = solver == 1;
  if (!use_jacobi) {
    if (tid == 0) *s_fallback = 0;
    gram_tridiag<TL>(Kc, ldk, Dk4, Ct, dd, ee, bet, xrow, dgl, pp, lam + 48, tid, warp, lane);

    // ---- the r largest eigenvalues of T: Gershgorin bounds, then every warp narrows one eigenvalue 32 ways per step ----
    if (warp == 0) {
      float lo = INFINITY, hi = -INFINITY, em = 0.f;
      for (int i = lane; i < L; i += 32) {
        const float rad = ((i > 0) ? fabsf(ee[i - 1]) : 0.f) + ((i + 1 < L) ? fabsf(ee[i]) : 0.f);
        lo = fminf(lo, dd[i] - rad); hi = fmaxf(hi, dd[i] + rad);
        const float q = ee[i] * ee[i];
        e2[i] = q; em = fmaxf(em, q);
      }
      lo = -warp_max(-lo); hi = warp_max(hi); em = warp_max(em);
      const float tn = fmaxf(fabsf(lo), fabsf(hi));
      if (lane == 0) {
        lam[32] = lo - 2e-6f * tn - 1e-30f; lam[33] = hi + 2e-6f * tn + 1e-30f;
        lam[34] = fmaxf(1e-35f, 1e-14f * em);          // smallest pivot allowed
        lam[35] = tn;
      }
    }
    __syncthreads();
    const float pivmin = lam[34], tnorm = lam[35];
    for (int j = warp; j < r_eff; j += NW) {
      const int target = L - 1 - j;                     // the eigenvalue with exactly `target` eigenvalues below it
      float a = lam[32], b = lam[33];
      for (int it = 0; it < 5; ++it) {
        const float x = a + (b - a) * ((float)(lane + 1) * (1.0f / 33.0f));
        float q = dd[0] - x;
        if (fabsf(q) < pivmin) q = -pivmin;
        int cnt = q < 0.f;
#pragma unroll 8
        for (int i = 1; i < L; ++i) {
          q = dd[i] - x - __fdividef(e2[i - 1], q);
          if (fabsf(q) < pivmin) q = -pivmin;
          cnt += q < 0.f;
        }
        const int n_ok = __popc(__ballot_sync(0xffffffffu, cnt <= target));   // counts grow with x: the lanes below form a prefix
        const float xa = __shfl_sync(0xffffffffu, x, max(n_ok - 1, 0)), xb = __shfl_sync(0xffffffffu, x, min(n_ok, 31));
        if (n_ok > 0) a = xa;
        if (n_ok < 32) b = xb;
      }
      if (lane == 0) lam[j] = 0.5f * (a + b);
    }
    __syncthreads();
    // shifts: equal eigenvalues are moved apart by a few ulps of |T| so that their inverse iterations differ; a direction
    // whose eigenvalue is below the null threshold is not computed
    if (tid == 0) {
      float prev = INFINITY;
      for (int j = 0; j < COBS_MAX_RANK; ++j) {
        float sft = (j < r_eff) ? lam[j] : 0.f;
        if (j < r_eff && prev - sft < 2e-7f * tnorm) sft = prev - 2e-7f * tnorm;
        lam[16 + j] = sft;
        prev = sft;
        top[j] = (j < r_eff && lam[j] / (float)L > 1e-12f * meansq) ? j : -1;
      }
    }
    __syncthreads();

    // ---- eigenvectors of T by inverse iteration ---------------------------------------------------------------------
    // (T - s I) = P L U with row interchanges, by lane 0 of the vector's warp: the reciprocal of U's diagonal, its two
    // upper diagonals, the multipliers, a swap flag per step.  Then three rounds of: solve and scale (every warp its
    // vectors), then Gram-Schmidt in order of descending eigenvalue: the owner of vector i normalises it, the owners of
    // the later vectors take its direction out of theirs.
    {
      float *__restrict__ u1 = scr + warp * 5 * L, *__restrict__ u2 = u1 + L, *__restrict__ mm = u2 + L, *__restrict__ iv = mm + L,
            *__restrict__ sw = iv + L;
      constexpr int NZ = (L + 31) / 32, NV = COBS_MAX_RANK / NW;
      for (int round = 0; round < 3; ++round) {
        float zr[NV][NZ];                                 // this warp's vectors (vector warp + NW n), lane + 32 i
#pragma unroll
        for (int n = 0; n < NV; ++n) {
          const int j = warp + NW * n;
#pragma unroll
          for (int i = 0; i < NZ; ++i) zr[n][i] = 0.f;
          if (j >= r_eff || top[j] < 0) continue;         // (uniform per warp)
          float *__restrict__ z = Z + j * L;
          const float sft = lam[16 + j];
          if (round == 0 || r_eff > NW) {                 // the factorisation survives the rounds unless two vectors share the warp
            if (lane == 0) {
              float a0 = dd[0] - sft, a1 = ee[0];          // the row being reduced: its entries in columns i and i + 1
#pragma unroll 4
              for (int i = 0; i + 1 < L; ++i) {
                const float sub = ee[i], nd = dd[i + 1] - sft, ne = ee[i + 1];   // the next row: columns i, i + 1, i + 2
                const bool swp = fabsf(sub) > fabsf(a0);    // interchange: the next row becomes the pivot row
                float p0 = swp ? sub : a0;
                const float p1 = swp ? nd : a1, p2 = swp ? ne : 0.f;
                if (fabsf(p0) < pivmin) p0 = copysignf(pivmin, p0);
                const float inv = __fdividef(1.0f, p0), mlt = (swp ? a0 : sub) * inv;   // (a rounding error here only moves the shift)
                u1[i] = p1; u2[i] = p2; iv[i] = inv; mm[i] = mlt; sw[i] = swp ? 1.f : 0.f;
                a0 = (swp ? a1 : nd) - mlt * p1;
                a1 = (swp ? 0.f : ne) - mlt * p2;
              }
              if (fabsf(a0) < pivmin) a0 = copysignf(pivmin, a0);
              iv[L - 1] = __fdividef(1.0f, a0); u1[L - 1] = 0.f; u2[L - 1] = 0.f;
            }
            __syncwarp();
          }
          if (round == 0)                                  // a fixed start vector with a component in every direction
            for (int i = lane; i < L; i += 32) z[i] = (float)((i * 40503u + j * 9973u + 12345u) & 1023u) * (1.0f / 512.0f) - 1.0f;
          __syncwarp();
          if (lane == 0) {
            float zi = z[0];
#pragma unroll 4
            for (int i = 0; i + 1 < L; ++i) {             // the right-hand side through P and L
              const float zn = z[i + 1], mlt = mm[i];
              const bool swp = sw[i] != 0.f;
              z[i] = swp ? zn : zi;
              zi = swp ? zi - mlt * zn : zn - mlt * zi;
            }
            float x1 = zi * iv[L - 1], x2 = 0.f;           // back substitution through U's three diagonals
            z[L - 1] = x1;
#pragma unroll 4
            for (int i = L - 2; i >= 0; --i) {
              const float x = (z[i] - u1[i] * x1 - u2[i] * x2) * iv[i];
              z[i] = x; x2 = x1; x1 = x;
            }
          }
          __syncwarp();
          float mx = 0.f;
#pragma unroll
          for (int i = 0; i < NZ; ++i) {
            zr[n][i] = (lane + 32 * i < L) ? z[lane + 32 * i] : 0.f;
            mx = fmaxf(mx, fabsf(zr[n][i]));
          }
          mx = warp_max(mx);
          const float sc = (mx > 0.f && mx < INFINITY) ? 1.0f / mx : 0.f;
#pragma unroll
          for (int i = 0; i < NZ; ++i) zr[n][i] *= sc;
        }
        for (int i = 0; i < r_eff; ++i) {
          if (top[i] < 0) continue;                        // (uniform)
#pragma unroll
          for (int n = 0; n < NV; ++n) {
            if (warp + NW * n != i) continue;
            float n2 = 0.f;
#pragma unroll
            for (int c = 0; c < NZ; ++c) n2 = fmaf(zr[n][c], zr[n][c], n2);
            n2 = warp_sum(n2);
            const float sc = (n2 > 0.f) ? rsqrtf(n2) : 0.f;
#pragma unroll
            for (int c = 0; c < NZ; ++c) {
              zr[n][c] *= sc;
              if (lane + 32 * c < L) Z[i * L + lane + 32 * c] = zr[n][c];
            }
          }
          __syncthreads();
#pragma unroll
          for (int n = 0; n < NV; ++n) {
            const int j = warp + NW * n;
            if (j <= i || j >= r_eff || top[j] < 0) continue;
            float y[NZ], dt = 0.f;
#pragma unroll
            for (int c = 0; c < NZ; ++c) {
              y[c] = (lane + 32 * c < L) ? Z[i * L + lane + 32 * c] : 0.f;
              dt = fmaf(zr[n][c], y[c], dt);
            }
            dt = warp_sum(dt);
#pragma unroll
            for (int c = 0; c < NZ; ++c) zr[n][c] -= dt * y[c];
          }
        }
        __syncthreads();
      }
    }
    // ---- check |T z - lambda z| (and that z is a unit vector); a failure sends the block to the Jacobi solver ----------
    for (int j = warp; j < r_eff; j += NW) {
      if (top[j] < 0) continue;
      const float *z = Z + j * L;
      float rmax = 0.f, n2 = 0.f;
      for (int i = lane; i < L; i += 32) {
        const float tz = dd[i] * z[i] + ((i > 0) ? ee[i - 1] * z[i - 1] : 0.f) + ((i + 1 < L) ? ee[i] * z[i + 1] : 0.f);
        rmax = fmaxf(rmax, fabsf(tz - lam[j] * z[i]));
        n2 = fmaf(z[i], z[i], n2);
      }
      rmax = warp_max(rmax); n2 = warp_sum(n2);
      if (lane == 0 && !(rmax <= 2e-5f * fmaxf(lam[0], 0.f) && fabsf(n2 - 1.f) < 1e-3f)) *s_fallback = 1;
    }
    __syncthreads();
    use_jacobi = *s_fallback != 0;
    if (!use_jacobi) {
      back_transform<TL>(Z, Ct, bet, top, r_eff, warp, lane);      // w = Q z
      __syncthreads();
      // ---- factors xi_i = K~^T w_i / sqrt(L); with a subspace, U_Q^T [(K - mean)^T w_i] / sqrt(L) ------------------------
      load_keys(false, false);
      float *yv = p.u_q ? Kc + L * ldk : xi_s;            // [r][D]
      for (int c = tid; c < p.r * D; c += kBuildThreads) {
        const int i = c / D, d = c - i * D;
        float acc = 0.f;
        if (i < r_eff && top[i] >= 0) {
          const float *z = Z + i * L;
#pragma unroll 8
          for (int t = 0; t < L; ++t) acc = fmaf(Kc[t * ldk + d], z[t], acc);
        }
        yv[c] = acc * inv_sqrt_l;
      }
      if (tid < COBS_MAX_RANK && tid >= r_eff) top[tid] = -1;
      __syncthreads();
      if (p.u_q) {
        const float *uq = p.u_q + (size_t)h * D * Dk;
        for (int c = tid; c < p.r * Dk; c += kBuildThreads) {
          const int i = c / Dk, sidx = c - i * Dk;
          float acc = 0.f;
          if (i < r_eff && top[i] >= 0)
            for (int d = 0; d < D; ++d) acc = fmaf(uq[(size_t)d * Dk + sidx], yv[i * D + d], acc);
          xi_s[c] = acc;
        }
        __syncthreads();
      }
    } else {
      load_keys(false, true);                              // the Jacobi route starts from the (projected) centred keys
    }
  }
  if (use_jacobi) {
  // ---- one-sided Jacobi on the rows of K~ (round-robin pairing: L / 2 disjoint pairs per round) --------
  // A half-warp owns a pair: lane l (of 16) holds columns 4 l .. 4 l + 3 and 64 + 4 l .. 64 + 4 l + 3 of both rows.
  // Pair slot s of round R joins rows (R + s) mod (L - 1) and (R - s) mod (L - 1); slot 0 joins row L - 1 and row R.
  constexpr int half = L / 2;
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
  for (int c = tid; c < p.r * Dk; c += kBuildThreads) {
    const int i = c / Dk, d = c - i * Dk;
    const int col = top[i];
    xi_s[c] = (col >= 0) ? Kc[col * ldk + d] * inv_sqrt_l : 0.f;
  }
  __syncthreads();
  }

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

size_t build_smem_bytes(const Params &p) { return (size_t)build_smem_layout(p).total * sizeof(float); }

template <int TL>
static cudaError_t launch_build_tl(const Params &p, int block_begin, int block_end, int solver, cudaStream_t stream) {
  const size_t smem = build_smem_bytes(p);
  cudaError_t e = cudaFuncSetAttribute(build_kernel<TL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  const long long n_cta = (long long)p.B * p.Hkv * (block_end - block_begin);
  build_kernel<TL><<<(unsigned)n_cta, kBuildThreads, smem, stream>>>(p, block_begin, block_end, solver);
  count_launch();
  return cudaGetLastError();
}

// COBS_BUILD_SOLVER=jacobi (read at every call) sends every block down the Jacobi route; the default is the
// tridiagonal route with Jacobi as its fallback.
cudaError_t launch_build(const Params &p, int block_begin, int block_end, cudaStream_t stream) {
  if (block_end - block_begin <= 0) return cudaSuccess;
  const char *v = getenv("COBS_BUILD_SOLVER");
  const int solver = (v && strcmp(v, "jacobi") == 0) ? 1 : 0;
  switch (p.L) {
    case 16: return launch_build_tl<1>(p, block_begin, block_end, solver, stream);
    case 32: return launch_build_tl<2>(p, block_begin, block_end, solver, stream);
    case 64: return launch_build_tl<4>(p, block_begin, block_end, solver, stream);
    default: return launch_build_tl<8>(p, block_begin, block_end, solver, stream);
  }
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
