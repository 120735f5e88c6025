// Step (d): softmax attention over the selected blocks plus the local window (one softmax over
// their union, i.e. the kept blocks renormalised among themselves, Eq. oracle-true), computed as
// split-KV partials with an online softmax and merged by a combine kernel.
#include "common.cuh"

namespace cobs {

constexpr int kAttThreads = 128;

__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gmem_src) {
  uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(d), "l"(gmem_src));
}
__device__ __forceinline__ void cp_async_wait_all() {
  asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;\n" ::: "memory");
}

// One CTA walks a contiguous range of the unit's items (selected blocks first, ascending, then the
// window blocks).  K and V tiles of one block are staged in shared memory; K rows are stored with
// their 16-byte chunks XOR-swizzled by the row index so that a lane-per-token read is conflict free.
template <int G, int D>
__global__ void __launch_bounds__(kAttThreads) attend_kernel(Params p) {
  constexpr int CH = D / 8;                      // 16-byte chunks per row
  constexpr int GROUPS = kAttThreads / (D / 2);  // head groups in the P.V phase
  constexpr int HPT = (G + GROUPS - 1) / GROUPS; // heads per thread in the P.V phase
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int L = p.L;
  uint4 *Ks = reinterpret_cast<uint4 *>(smem_raw);                    // [L][CH]
  uint4 *Vs = Ks + L * CH;                                            // [L][CH]
  float *qs = reinterpret_cast<float *>(Vs + L * CH);                 // [G][D]
  float *sc = qs + G * D;                                             // [G][L]
  float *st_m = sc + G * L, *st_l = st_m + G, *st_c = st_l + G;       // [G] each
  int *pages = reinterpret_cast<int *>(st_c + G);                     // [L / P]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int u = blockIdx.y, split = blockIdx.x, b_idx = u / p.Hkv, h = u - b_idx * p.Hkv;
  const int T = p.seq_lens[b_idx];
  const int ws = window_start(T, p.window, L);
  const int n_cand = ws / L;
  const int n_win = (T - ws + L - 1) / L;
  const int n_sel = min(min(p.sel_cnt[u], p.topk), n_cand);
  const int n_items = n_sel + n_win;
  const int per = (n_items + p.n_splits - 1) / p.n_splits;
  const int i0 = min(split * per, n_items), i1 = min(i0 + per, n_items);

  const float inv_sqrt_d = 1.0f / sqrtf((float)D);
  for (int i = tid; i < G * D; i += kAttThreads)
    qs[i] = __bfloat162float(p.q[((size_t)b_idx * p.Hq + h * G) * D + i]) * inv_sqrt_d;
  if (tid < G) { st_m[tid] = -INFINITY; st_l[tid] = 0.f; }
  float acc[HPT][2];
#pragma unroll
  for (int j = 0; j < HPT; ++j) acc[j][0] = acc[j][1] = 0.f;
  const int dp = tid % (D / 2), hg = tid / (D / 2);
  __syncthreads();

  for (int it = i0; it < i1; ++it) {
    int blk;
    if (it < n_sel) {
      blk = p.sel_idx[(size_t)u * p.topk + it];
      if (blk < 0 || blk >= n_cand) {            // not a candidate block: skip it, tell the host
        if (tid == 0) report(p.status, COBS_ERR_BOUNDS);
        continue;
      }
    } else {
      blk = n_cand + (it - n_sel);
    }
    const int tok0 = blk * L;
    const int n_valid = min(L, T - tok0);
    const int n_pg = (n_valid + p.P - 1) / p.P;
    if (tid < n_pg) {
      int pg = p.page_table[(size_t)b_idx * p.mpp + tok0 / p.P + tid];
      if (pg < 0 || pg >= p.n_pages) { report(p.status, COBS_ERR_BOUNDS); pg = -1; }
      pages[tid] = pg;
    }
    __syncthreads();
    for (int c = tid; c < n_valid * CH; c += kAttThreads) {
      const int t = c / CH, col = c - t * CH;
      const int pg = pages[t / p.P];
      if (pg >= 0) {
        const size_t off = (((size_t)pg * p.Hkv + h) * p.P + (t % p.P)) * D + col * 8;
        cp_async16(&Ks[t * CH + (col ^ (t & 7))], p.k_pages + off);
        cp_async16(&Vs[t * CH + col], p.v_pages + off);
      } else {
        Ks[t * CH + (col ^ (t & 7))] = make_uint4(0, 0, 0, 0);
        Vs[t * CH + col] = make_uint4(0, 0, 0, 0);
      }
    }
    cp_async_wait_all();
    __syncthreads();

    // logits: one (token, head) dot product per work item
    for (int w = tid; w < L * G; w += kAttThreads) {
      const int t = w % L, g = w / L;
      if (t < n_valid) {
        const float *qg = qs + g * D;
        float s = 0.f;
#pragma unroll
        for (int c = 0; c < CH; ++c) {
          const uint4 kv = Ks[t * CH + (c ^ (t & 7))];
          const float4 qa = *reinterpret_cast<const float4 *>(qg + c * 8);
          const float4 qb = *reinterpret_cast<const float4 *>(qg + c * 8 + 4);
          s = fmaf(bf16_lo(kv.x), qa.x, s); s = fmaf(bf16_hi(kv.x), qa.y, s);
          s = fmaf(bf16_lo(kv.y), qa.z, s); s = fmaf(bf16_hi(kv.y), qa.w, s);
          s = fmaf(bf16_lo(kv.z), qb.x, s); s = fmaf(bf16_hi(kv.z), qb.y, s);
          s = fmaf(bf16_lo(kv.w), qb.z, s); s = fmaf(bf16_hi(kv.w), qb.w, s);
        }
        sc[g * L + t] = s;
      }
    }
    __syncthreads();

    // online softmax statistics, one warp per head
    for (int g = warp; g < G; g += kAttThreads / 32) {
      float mx = -INFINITY;
      for (int t = lane; t < n_valid; t += 32) mx = fmaxf(mx, sc[g * L + t]);
      mx = warp_max(mx);
      const float m_old = st_m[g], m_new = fmaxf(m_old, mx);
      float sum = 0.f;
      for (int t = lane; t < n_valid; t += 32) {
        const float pv = __expf(sc[g * L + t] - m_new);
        sc[g * L + t] = pv;
        sum += pv;
      }
      sum = warp_sum(sum);
      if (lane == 0) {
        const float corr = (m_old == -INFINITY) ? 0.f : __expf(m_old - m_new);
        st_c[g] = corr;
        st_m[g] = m_new;
        st_l[g] = st_l[g] * corr + sum;
      }
    }
    __syncthreads();

    // P.V: each thread owns two output dims of HPT heads
    const uint32_t *Vw = reinterpret_cast<const uint32_t *>(Vs);
#pragma unroll
    for (int j = 0; j < HPT; ++j) {
      const int g = hg + j * GROUPS;
      if (g < G) {
        const float corr = st_c[g];
        float a0 = acc[j][0] * corr, a1 = acc[j][1] * corr;
        const float *pg = sc + g * L;
        for (int t = 0; t < n_valid; ++t) {
          const uint32_t vv = Vw[t * (D / 2) + dp];
          const float pt = pg[t];
          a0 = fmaf(pt, bf16_lo(vv), a0);
          a1 = fmaf(pt, bf16_hi(vv), a1);
        }
        acc[j][0] = a0; acc[j][1] = a1;
      }
    }
    __syncthreads();
  }

  // partial record: [G][D + 2] = acc[D], running max, running sum
  float *part = p.partial + ((size_t)u * p.n_splits + split) * G * (D + 2);
#pragma unroll
  for (int j = 0; j < HPT; ++j) {
    const int g = hg + j * GROUPS;
    if (g < G) {
      part[g * (D + 2) + 2 * dp] = acc[j][0];
      part[g * (D + 2) + 2 * dp + 1] = acc[j][1];
    }
  }
  if (tid < G) {
    part[tid * (D + 2) + D] = st_m[tid];
    part[tid * (D + 2) + D + 1] = st_l[tid];
  }
}

// Merge of the split partials: o = sum_s e^{m_s - M} acc_s / sum_s e^{m_s - M} l_s.
// grid = B * Hq, block = D threads.
__global__ void combine_kernel(Params p) {
  const int bh = blockIdx.x, b_idx = bh / p.Hq, hq = bh - b_idx * p.Hq;
  const int h = hq / p.G, g = hq - h * p.G, u = b_idx * p.Hkv + h, d = threadIdx.x, D = p.D;
  const float *base = p.partial + ((size_t)u * p.n_splits * p.G + g) * (D + 2);
  const size_t stride = (size_t)p.G * (D + 2);
  float M = -INFINITY;
  for (int s = 0; s < p.n_splits; ++s) M = fmaxf(M, base[s * stride + D]);
  float den = 0.f, num = 0.f;
  for (int s = 0; s < p.n_splits; ++s) {
    const float m = base[s * stride + D];
    const float w = (m == -INFINITY) ? 0.f : __expf(m - M);
    den = fmaf(w, base[s * stride + D + 1], den);
    num = fmaf(w, base[s * stride + d], num);
  }
  p.out[(size_t)bh * D + d] = num / den;
  if (p.lse && d == 0) p.lse[bh] = M + logf(den);
}

template <int G, int D>
static cudaError_t launch_attend_gd(const Params &p, cudaStream_t stream) {
  size_t smem = (size_t)2 * p.L * D * 2 + (size_t)(G * D + G * p.L + 3 * G) * sizeof(float) +
                (size_t)(p.L / p.P + 1) * sizeof(int);
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(attend_kernel<G, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  dim3 grid(p.n_splits, p.B * p.Hkv);
  attend_kernel<G, D><<<grid, kAttThreads, smem, stream>>>(p);
  count_launch();
  return cudaGetLastError();
}

template <int G>
static cudaError_t launch_attend_g(const Params &p, cudaStream_t stream) {
  return p.D == 64 ? launch_attend_gd<G, 64>(p, stream) : launch_attend_gd<G, 128>(p, stream);
}

cudaError_t launch_attend(const Params &p, cudaStream_t stream) {
  cudaError_t e;
  switch (p.G) {
    case 1: e = launch_attend_g<1>(p, stream); break;
    case 2: e = launch_attend_g<2>(p, stream); break;
    case 4: e = launch_attend_g<4>(p, stream); break;
    default: e = launch_attend_g<8>(p, stream); break;
  }
  if (e != cudaSuccess) return e;
  combine_kernel<<<p.B * p.Hq, p.D, 0, stream>>>(p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace cobs
