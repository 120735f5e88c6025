// Steps (b) and (c): second-order block scores from the stored summaries, GQA group score, top-k.
//
//   e[g][b]  = ln L + q'_g . mean_b + 1/2 sum_i (xi_{b,i} . q~_g)^2      (Eq. trunc with Eq. gram)
//              [+ 1/6 sum_i c_{b,i} (xi_{b,i} . q'_g)^3 when skew scalars are given: Appendix, Cheap diagonal skew]
//   score[b] = sum_g exp(e[g][b] - logsumexp_b' e[g][b'])                (Eq. gqa-secondorder)
//   selection: k largest scores among the candidate blocks, lower index on ties, ascending output.
#include "common.cuh"

namespace cobs {

// ------------------------------------------------------------------------------------------------
// Query preparation shared by the scoring kernels: q' = q / sqrt(D) and q~ = U_Q^T q' (or q').
// qs: [G][D], qt: [G][Ds_pad] (zero padded), both in shared memory.
// ------------------------------------------------------------------------------------------------
template <int G>
__device__ void prepare_query(const Params &p, int b_idx, int h, float *qs, float *qt) {
  const float inv_sqrt_d = 1.0f / sqrtf((float)p.D);
  for (int i = threadIdx.x; i < G * p.D; i += blockDim.x) {
    int g = i / p.D, d = i - g * p.D;
    qs[i] = __bfloat162float(p.q[((size_t)b_idx * p.Hq + h * G + g) * p.D + d]) * inv_sqrt_d;
  }
  __syncthreads();
  for (int i = threadIdx.x; i < G * p.Ds_pad; i += blockDim.x) {
    int g = i / p.Ds_pad, s = i - g * p.Ds_pad;
    float v = 0.f;
    if (s < p.Ds) {
      if (p.u_q) {
        const float *u = p.u_q + (size_t)h * p.D * p.Ds + s;
        for (int d = 0; d < p.D; ++d) v = fmaf(u[(size_t)d * p.Ds], qs[g * p.D + d], v);
      } else {
        v = qs[g * p.D + s];
      }
    }
    qt[i] = v;
  }
  __syncthreads();
}

// ------------------------------------------------------------------------------------------------
// Generic scoring kernel (any summary dtype, any Ds): one warp per block record, lanes stride the
// row, fp32 FMA, warp-shuffle reduction per (row, head).
// grid = (ceil(NB / blocks_per_cta), B * Hkv), block = 256 threads.
// ------------------------------------------------------------------------------------------------
template <int G, int DT>
__global__ void __launch_bounds__(256) score_generic_kernel(Params p, int blocks_per_cta) {
  extern __shared__ float smem[];
  float *qs = smem;                 // [G][D]
  float *qt = smem + G * p.D;       // [G][Ds_pad]
  const int u = blockIdx.y, b_idx = u / p.Hkv, h = u - b_idx * p.Hkv;
  int T = p.seq_lens[b_idx];
  int n_sum = min(T / p.L, p.NB);
  const int first = blockIdx.x * blocks_per_cta;
  if (first >= n_sum) return;
  prepare_query<G>(p, b_idx, h, qs, qt);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
  const int last = min(first + blocks_per_cta, n_sum);
  const float ln_l = logf((float)p.L);
  for (int b = first + warp; b < last; b += n_warps) {
    const size_t rec = (size_t)u * p.NB + b;
    float acc[G];
#pragma unroll
    for (int g = 0; g < G; ++g) acc[g] = 0.f;
    // first-order term: q' . mean
    for (int j = lane; j < p.D; j += 32) {
      float m = (DT == COBS_SUMM_FP32) ? ((const float *)p.mean)[rec * p.D + j]
                                       : __bfloat162float(((const __nv_bfloat16 *)p.mean)[rec * p.D + j]);
#pragma unroll
      for (int g = 0; g < G; ++g) acc[g] = fmaf(m, qs[g * p.D + j], acc[g]);
    }
    float first_order[G], second[G];
#pragma unroll
    for (int g = 0; g < G; ++g) { first_order[g] = warp_sum(acc[g]); second[g] = 0.f; }
    // curvature term from the r stored factors
    for (int i = 0; i < p.r; ++i) {
#pragma unroll
      for (int g = 0; g < G; ++g) acc[g] = 0.f;
      float sc = 1.0f;
      if (DT == COBS_SUMM_FP4_E2M1) {
        sc = (p.scale_dtype == COBS_SCALE_FP16) ? __half2float(((const __half *)p.scale)[rec * p.r + i])
                                                : ((const float *)p.scale)[rec * p.r + i];
      }
      for (int j = lane; j < p.Ds; j += 32) {
        float x;
        if (DT == COBS_SUMM_FP32) {
          x = ((const float *)p.xi)[(rec * p.r + i) * p.Ds + j];
        } else if (DT == COBS_SUMM_BF16) {
          x = __bfloat162float(((const __nv_bfloat16 *)p.xi)[(rec * p.r + i) * p.Ds + j]);
        } else {
          uint32_t byte = ((const uint8_t *)p.xi)[(rec * p.r + i) * (size_t)(p.Ds_pad / 2) + (j >> 1)];
          x = e2m1_value((j & 1) ? (byte >> 4) : (byte & 15u));
        }
#pragma unroll
        for (int g = 0; g < G; ++g) acc[g] = fmaf(x, qt[g * p.Ds_pad + j], acc[g]);
      }
      const float c6 = p.skew ? p.skew[rec * p.r + i] * (1.0f / 3.0f) : 0.f;   // (c / 6) / (1 / 2): folded into `second`
#pragma unroll
      for (int g = 0; g < G; ++g) {
        float d = warp_sum(acc[g]) * sc;
        second[g] = fmaf(d * d, fmaf(c6, d, 1.0f), second[g]);                 // d^2 + (c / 3) d^3
      }
    }
    if (lane < G) {
      float v = 0.f;
#pragma unroll
      for (int g = 0; g < G; ++g)
        if (lane == g) v = ln_l + first_order[g] + 0.5f * second[g];
      p.e[((size_t)u * G + lane) * p.NB + b] = v;
    }
  }
}

// ------------------------------------------------------------------------------------------------
// Group score + top-k, one CTA per (sequence, KV head).
// ------------------------------------------------------------------------------------------------
constexpr int kSelThreads = 512;
constexpr int kSelWarps = kSelThreads / 32;

// Exclusive prefix sum of one int per thread over the CTA (fixed order); *total gets the sum.
__device__ __forceinline__ int block_exclusive_scan(int v, int *warp_tot, int *total) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  __syncthreads();
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  int base = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < kSelWarps; ++w) {
    const int t = warp_tot[w];
    if (w < warp) base += t;
    tot += t;
  }
  *total = tot;
  return base + inc - v;
}

__global__ void __launch_bounds__(kSelThreads) select_kernel(Params p) {
  extern __shared__ float score[];                 // [NB]
  __shared__ float red_m[kSelWarps], red_s[kSelWarps];
  __shared__ float lse[8];
  __shared__ int hist[256];
  __shared__ int warp_tot[kSelWarps];
  __shared__ uint32_t s_prefix;
  __shared__ int s_need;

  const int u = blockIdx.x, b_idx = u / p.Hkv, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int T = p.seq_lens[b_idx];
  const int n_sum = min(T / p.L, p.NB);
  const int n_cand = min(window_start(T, p.window, p.L) / p.L, n_sum);
  const int G = p.G;

  // log-sum-exp of each head's estimates over every summarised block: one pass of (max, sum) pairs
  for (int g = 0; g < G; ++g) {
    const float *e = p.e + ((size_t)u * G + g) * p.NB;
    float mx = -INFINITY, sm = 0.f;
    for (int b = tid; b < n_sum; b += kSelThreads) {
      const float x = e[b];
      if (x > mx) { sm = sm * expf(mx - x) + 1.0f; mx = x; }
      else sm += expf(x - mx);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float om = __shfl_xor_sync(0xffffffffu, mx, o), os = __shfl_xor_sync(0xffffffffu, sm, o);
      const float nm = fmaxf(mx, om);
      sm = (nm == -INFINITY) ? 0.f : sm * expf(mx - nm) + os * expf(om - nm);
      mx = nm;
    }
    if (lane == 0) { red_m[warp] = mx; red_s[warp] = sm; }
    __syncthreads();
    if (tid == 0) {
      float M = -INFINITY;
      for (int w = 0; w < kSelWarps; ++w) M = fmaxf(M, red_m[w]);
      float S = 0.f;
      for (int w = 0; w < kSelWarps; ++w) S += (red_m[w] == -INFINITY) ? 0.f : red_s[w] * expf(red_m[w] - M);
      lse[g] = M + logf(S);
    }
    __syncthreads();
  }
  for (int b = tid; b < n_sum; b += kSelThreads) {
    float s = 0.f;
    for (int g = 0; g < G; ++g) s += expf(p.e[((size_t)u * G + g) * p.NB + b] - lse[g]);
    score[b] = s;
    if (p.scores) p.scores[(size_t)u * p.NB + b] = s;
  }
  __syncthreads();

  int32_t *out = p.sel_idx + (size_t)u * p.topk;
  const int k = min(p.topk, n_cand);
  if (tid == 0) p.sel_cnt[u] = k;
  for (int i = k + tid; i < p.topk; i += kSelThreads) out[i] = -1;
  if (k == 0) return;
  if (k == n_cand) {
    for (int i = tid; i < k; i += kSelThreads) out[i] = i;
    return;
  }

  // radix select of the k-th largest key (scores are >= 0, so their bit patterns order like integers)
  if (tid == 0) { s_prefix = 0u; s_need = k; }
  uint32_t mask = 0u;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = tid; i < 256; i += kSelThreads) hist[i] = 0;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    for (int b = tid; b < n_cand; b += kSelThreads) {
      const uint32_t key = __float_as_uint(score[b]);
      if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1);
    }
    __syncthreads();
    if (warp == 0) {
      // lane l owns bins 255 - 8 l ... 248 - 8 l (descending); find the bin where the running count reaches `need`
      const int need = s_need;
      int mine = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) mine += hist[255 - 8 * lane - j];
      int inc = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
      }
      const int before = inc - mine;
      if (before < need && inc >= need) {          // exactly one lane
        int cum = before, bin = 255 - 8 * lane;
        for (int j = 0; j < 8; ++j, --bin) {
          if (cum + hist[bin] >= need) break;
          cum += hist[bin];
        }
        s_need = need - cum;
        s_prefix = prefix | ((uint32_t)bin << shift);
      }
    }
    mask |= 255u << shift;
    __syncthreads();
  }
  const uint32_t theta = s_prefix;   // key of the k-th largest score
  const int need_eq = s_need;        // how many blocks with exactly that key to keep (lowest indices)

  // ordered compaction: each thread owns a contiguous index range
  const int per = (n_cand + kSelThreads - 1) / kSelThreads;
  const int lo = min(tid * per, n_cand), hi = min(lo + per, n_cand);
  int n_eq = 0;
  for (int b = lo; b < hi; ++b) n_eq += (__float_as_uint(score[b]) == theta);
  int total;
  const int eq_base = block_exclusive_scan(n_eq, warp_tot, &total);
  int eq_rank = eq_base, n_keep = 0;
  for (int b = lo; b < hi; ++b) {
    const uint32_t key = __float_as_uint(score[b]);
    if (key > theta) ++n_keep;
    else if (key == theta) { if (eq_rank < need_eq) ++n_keep; ++eq_rank; }
  }
  int pos = block_exclusive_scan(n_keep, warp_tot, &total);
  eq_rank = eq_base;
  for (int b = lo; b < hi; ++b) {
    const uint32_t key = __float_as_uint(score[b]);
    bool keep = false;
    if (key > theta) keep = true;
    else if (key == theta) { keep = eq_rank < need_eq; ++eq_rank; }
    if (keep && pos < k) out[pos++] = b;
  }
}

// ------------------------------------------------------------------------------------------------
// host launchers
// ------------------------------------------------------------------------------------------------
template <int G>
static cudaError_t launch_score_g(const Params &p, cudaStream_t stream) {
  const int blocks_per_cta = 32;
  dim3 grid((p.NB + blocks_per_cta - 1) / blocks_per_cta, p.B * p.Hkv);
  size_t smem = (size_t)G * (p.D + p.Ds_pad) * sizeof(float);
  switch (p.summ_dtype) {
    case COBS_SUMM_FP32: score_generic_kernel<G, COBS_SUMM_FP32><<<grid, 256, smem, stream>>>(p, blocks_per_cta); break;
    case COBS_SUMM_BF16: score_generic_kernel<G, COBS_SUMM_BF16><<<grid, 256, smem, stream>>>(p, blocks_per_cta); break;
    default: score_generic_kernel<G, COBS_SUMM_FP4_E2M1><<<grid, 256, smem, stream>>>(p, blocks_per_cta); break;
  }
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_score(const Params &p, cudaStream_t stream) {
  switch (p.G) {
    case 1: return launch_score_g<1>(p, stream);
    case 2: return launch_score_g<2>(p, stream);
    case 4: return launch_score_g<4>(p, stream);
    default: return launch_score_g<8>(p, stream);
  }
}

cudaError_t launch_select(const Params &p, cudaStream_t stream) {
  size_t smem = (size_t)p.NB * sizeof(float);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  select_kernel<<<p.B * p.Hkv, kSelThreads, smem, stream>>>(p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace cobs
