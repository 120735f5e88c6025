// Step (d): softmax attention over the selected blocks plus the local window (one softmax over
// their union, i.e. the kept blocks renormalised among themselves, Eq. oracle-true), computed as
// split-KV partials with an online softmax and merged by a combine kernel.
//
// Kernel shape.  Decode attention for one KV head is G query rows against a stream of K/V rows: 2 G
// flop per byte, HBM-bound, so the kernel is built around keeping many bytes in flight per SM and few
// instructions per byte:
//   * a CTA of 4 warps walks a contiguous slice of one (sequence, KV head) unit's block list (selected
//     blocks ascending, then the window blocks); each WARP works alone on 16-token groups of that
//     slice with its own online-softmax state (no CTA barrier in the loop), merged once at the end;
//   * S^T = q K^T on mma.sync m16n8k16 (bf16 x bf16 -> fp32): the G query heads are the 16 M-rows
//     (zero padded), 8 tokens are the N-columns; K fragments come straight from global memory with
//     16-byte loads (the contraction index is permuted so that a thread's fragment is contiguous in
//     memory, and the query fragments are permuted the same way);
//   * the S accumulators are, as they sit in registers, the A fragments of P V; P is split into a
//     bf16 high and low part (two mma per tile) so that rounding P costs 2^-17, not 2^-9;
//   * V goes global -> shared by cp.async into a 3-stage per-warp ring (XOR-swizzled 16-byte chunks)
//     and is read with ldmatrix.trans as the B fragments of P V.
#include "common.cuh"

namespace cobs {

constexpr int kAttWarps = 4;
constexpr int kAttThreads = kAttWarps * 32;
constexpr int kVStages = 3;
constexpr int kMaxGroupsPerCta = 1024;     // 16-token groups a CTA can index (shared-memory table)

__device__ __forceinline__ void cp_async16_zfill(uint32_t smem_dst, const void *gmem_src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(smem_dst), "l"(gmem_src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

__device__ __forceinline__ void mma_bf16_16816(float &c0, float &c1, float &c2, float &c3, uint32_t a0, uint32_t a1,
                                               uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c0), "+f"(c1), "+f"(c2), "+f"(c3)
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ uint4 ldg_nc(const uint4 *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t *>(&v);
}

// grid = (n_splits, B * Hkv), block = 128 threads.
template <int D>
__global__ void __launch_bounds__(kAttThreads, 3) attend_kernel(Params p) {
  constexpr int CH = D / 8;              // 16-byte chunks per row
  constexpr int KS = D / 16;             // k-steps of q K^T
  constexpr int NT = D / 8;              // 8-wide dim tiles of the output
  constexpr int STAGE_BYTES = 16 * D * 2;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char *vring = smem_raw;                                               // [warps][stages][16][D] bf16
  uint32_t *goff = reinterpret_cast<uint32_t *>(vring + kAttWarps * kVStages * STAGE_BYTES);   // [groups] 16-B units
  int *gtok = reinterpret_cast<int *>(goff + kMaxGroupsPerCta);                   // [groups] first token
  float *mrg = reinterpret_cast<float *>(vring);                                 // reused at the end: [warps][8][D + 2]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gid = lane >> 2, tig = lane & 3;
  const int u = blockIdx.y, split = blockIdx.x, b_idx = u / p.Hkv, h = u - b_idx * p.Hkv;
  const int G = p.G, L = p.L, P = p.P;
  const int T = p.seq_lens[b_idx];
  const int ws = window_start(T, p.window, L);
  const int n_cand = ws / L;
  const int n_win = (T - ws + L - 1) / L;
  const int n_sel = min(min(p.sel_cnt[u], p.topk), n_cand);
  const int n_items = n_sel + n_win;
  const int per = (n_items + p.n_splits - 1) / p.n_splits;
  const int i0 = min(split * per, n_items), i1 = min(i0 + per, n_items);
  const int gpb = L / 16;                 // groups per block
  int n_groups = (i1 - i0) * gpb;
  if (n_groups > kMaxGroupsPerCta) n_groups = kMaxGroupsPerCta;   // cannot happen for supported shapes

  // ---- table of this CTA's 16-token groups: global offset of the group's first K/V row, first token ----
  for (int g = tid; g < n_groups; g += kAttThreads) {
    const int it = i0 + g / gpb, sub = g - (g / gpb) * gpb;
    int blk;
    bool ok = true;
    if (it < n_sel) {
      blk = p.sel_idx[(size_t)u * p.topk + it];
      if (blk < 0 || blk >= n_cand) { ok = false; report(p.status, COBS_ERR_BOUNDS); }
    } else {
      blk = n_cand + (it - n_sel);
    }
    const int tok0 = blk * L + sub * 16;
    int first = -1;
    uint32_t off = 0;
    if (ok && tok0 < T) {
      const int pg = p.page_table[(size_t)b_idx * p.mpp + tok0 / P];
      if (pg < 0 || pg >= p.n_pages) report(p.status, COBS_ERR_BOUNDS);
      else { first = tok0; off = (uint32_t)(((((size_t)pg * p.Hkv + h) * P + (tok0 % P)) * D) / 8); }
    }
    goff[g] = off;
    gtok[g] = first;                       // -1: nothing to read for this group
  }

  // ---- query fragments (A operand of q K^T): rows = heads (zero padded), k permuted like K's -----------
  uint32_t qa[KS][2];
  {
    const __nv_bfloat16 *qg = p.q + ((size_t)b_idx * p.Hq + h * G) * D;
#pragma unroll
    for (int m = 0; m < KS / 2; ++m) {
      uint4 v = make_uint4(0, 0, 0, 0);
      if (gid < G) v = *reinterpret_cast<const uint4 *>(qg + gid * D + (tig + 4 * m) * 8);
      qa[2 * m][0] = v.x; qa[2 * m][1] = v.y; qa[2 * m + 1][0] = v.z; qa[2 * m + 1][1] = v.w;
    }
  }
  __syncthreads();

  const uint4 *kbase = reinterpret_cast<const uint4 *>(p.k_pages);
  const uint4 *vbase = reinterpret_cast<const uint4 *>(p.v_pages);
  const uint32_t vring_s = (uint32_t)__cvta_generic_to_shared(vring) + warp * (kVStages * STAGE_BYTES);
  const float sl2 = (1.0f / sqrtf((float)D)) * 1.4426950408889634f;    // logits in the log2 domain

  float o[NT][2];
#pragma unroll
  for (int n = 0; n < NT; ++n) o[n][0] = o[n][1] = 0.f;
  float m_run = -INFINITY, l_run = 0.f, z2 = 0.f, z3 = 0.f;

  // issue the V copy of group g into ring stage `st` (always commits, so that group counting is uniform)
  auto issue_v = [&](int g, int st) {
    if (g < n_groups) {
      const int first = gtok[g];
      if (first >= 0) {
        const int nv = min(16, T - first);
        const uint4 *src = vbase + goff[g];
#pragma unroll
        for (int j = 0; j < (16 * CH) / 32; ++j) {
          const int i = lane + 32 * j, t = i / CH, c = i - t * CH;
          cp_async16_zfill(vring_s + st * STAGE_BYTES + t * (D * 2) + ((c ^ (t & 7)) << 4), src + i, t < nv ? 16 : 0);
        }
      }
    }
    cp_async_commit();
  };
  auto load_k = [&](int g, uint4 (&kr)[2][KS / 2]) {
    if (g < n_groups && gtok[g] >= 0) {
      const uint4 *src = kbase + goff[g];
#pragma unroll
      for (int m = 0; m < KS / 2; ++m) {
        kr[0][m] = ldg_nc(src + gid * CH + tig + 4 * m);
        kr[1][m] = ldg_nc(src + (gid + 8) * CH + tig + 4 * m);
      }
    }
  };

  uint4 kcur[2][KS / 2], knext[2][KS / 2];
#pragma unroll
  for (int a = 0; a < 2; ++a)
#pragma unroll
    for (int m = 0; m < KS / 2; ++m) kcur[a][m] = knext[a][m] = make_uint4(0, 0, 0, 0);

  // prologue: V of the first two groups of this warp, K of the first
  issue_v(warp, 0);
  issue_v(warp + kAttWarps, 1);
  load_k(warp, kcur);

  int st = 0;
  for (int g = warp; g < n_groups; g += kAttWarps) {
    issue_v(g + 2 * kAttWarps, (st + 2) % kVStages);
    load_k(g + kAttWarps, knext);
    const int first = gtok[g];
    if (first >= 0) {
      const int nv = min(16, T - first);
      // ---- S^T = q K^T for tokens 0-7 (s0) and 8-15 (s1) of the group ---------------------------------
      float s0[2] = {0.f, 0.f}, s1[2] = {0.f, 0.f};
#pragma unroll
      for (int m = 0; m < KS / 2; ++m) {
        mma_bf16_16816(s0[0], s0[1], z2, z3, qa[2 * m][0], 0u, qa[2 * m][1], 0u, kcur[0][m].x, kcur[0][m].y);
        mma_bf16_16816(s0[0], s0[1], z2, z3, qa[2 * m + 1][0], 0u, qa[2 * m + 1][1], 0u, kcur[0][m].z, kcur[0][m].w);
        mma_bf16_16816(s1[0], s1[1], z2, z3, qa[2 * m][0], 0u, qa[2 * m][1], 0u, kcur[1][m].x, kcur[1][m].y);
        mma_bf16_16816(s1[0], s1[1], z2, z3, qa[2 * m + 1][0], 0u, qa[2 * m + 1][1], 0u, kcur[1][m].z, kcur[1][m].w);
      }
      // this thread: head gid, tokens 2 tig, 2 tig + 1 (s0) and 2 tig + 8, 2 tig + 9 (s1)
      float t0 = (2 * tig < nv) ? s0[0] * sl2 : -INFINITY;
      float t1 = (2 * tig + 1 < nv) ? s0[1] * sl2 : -INFINITY;
      float t2 = (2 * tig + 8 < nv) ? s1[0] * sl2 : -INFINITY;
      float t3 = (2 * tig + 9 < nv) ? s1[1] * sl2 : -INFINITY;
      float mx = fmaxf(fmaxf(t0, t1), fmaxf(t2, t3));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float m_new = fmaxf(m_run, mx);
      const float corr = exp2f(m_run - m_new);
      m_run = m_new;
      const float p0 = exp2f(t0 - m_new), p1 = exp2f(t1 - m_new), p2 = exp2f(t2 - m_new), p3 = exp2f(t3 - m_new);
      l_run = l_run * corr + ((p0 + p1) + (p2 + p3));
#pragma unroll
      for (int n = 0; n < NT; ++n) { o[n][0] *= corr; o[n][1] *= corr; }
      // P = hi + lo, both bf16
      const uint32_t a0h = pack_bf16(p0, p1), a2h = pack_bf16(p2, p3);
      const float h0 = bf16_lo(a0h), h1 = bf16_hi(a0h), h2 = bf16_lo(a2h), h3 = bf16_hi(a2h);
      const uint32_t a0l = pack_bf16(p0 - h0, p1 - h1), a2l = pack_bf16(p2 - h2, p3 - h3);

      // ---- O += P V, V fragments by ldmatrix.trans from this warp's ring stage ----------------------------
      cp_async_wait<2>();                  // the copy of group g has landed (two younger copies may be in flight)
      __syncwarp();
      const uint32_t vs = vring_s + st * STAGE_BYTES;
      // lane -> row address of matrix (lane / 8): tokens (lane / 8 % 2) * 8 + lane % 8, chunk 2 np + lane / 16
      const int lt = ((lane >> 3) & 1) * 8 + (lane & 7), lc = lane >> 4;
#pragma unroll
      for (int np = 0; np < NT / 2; ++np) {
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4_trans(b0, b1, b2, b3, vs + lt * (D * 2) + (((2 * np + lc) ^ (lt & 7)) << 4));
        mma_bf16_16816(o[2 * np][0], o[2 * np][1], z2, z3, a0h, 0u, a2h, 0u, b0, b1);
        mma_bf16_16816(o[2 * np][0], o[2 * np][1], z2, z3, a0l, 0u, a2l, 0u, b0, b1);
        mma_bf16_16816(o[2 * np + 1][0], o[2 * np + 1][1], z2, z3, a0h, 0u, a2h, 0u, b2, b3);
        mma_bf16_16816(o[2 * np + 1][0], o[2 * np + 1][1], z2, z3, a0l, 0u, a2l, 0u, b2, b3);
      }
      __syncwarp();                        // every lane is done reading the stage before it is refilled
    }
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int m = 0; m < KS / 2; ++m) kcur[a][m] = knext[a][m];
    st = (st + 1) % kVStages;
  }
  cp_async_wait<0>();

  // ---- merge the four warps' states, write the split's partial: [G][D + 2] = acc, running max, sum -------
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
  __syncthreads();                         // everyone is done with the V ring; reuse it
  if (gid < G) {
    float *dst = mrg + ((size_t)warp * 8 + gid) * (D + 2);
#pragma unroll
    for (int n = 0; n < NT; ++n) { dst[8 * n + 2 * tig] = o[n][0]; dst[8 * n + 2 * tig + 1] = o[n][1]; }
    if (tig == 0) { dst[D] = m_run; dst[D + 1] = l_run; }
  }
  __syncthreads();
  float *part = p.partial + ((size_t)u * p.n_splits + split) * G * (D + 2);
  const float ln2 = 0.6931471805599453f;
  for (int i = tid; i < G * D; i += kAttThreads) {
    const int g = i / D, d = i - g * D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kAttWarps; ++w) M = fmaxf(M, mrg[((size_t)w * 8 + g) * (D + 2) + D]);
    float acc = 0.f, l = 0.f;
#pragma unroll
    for (int w = 0; w < kAttWarps; ++w) {
      const float *src = mrg + ((size_t)w * 8 + g) * (D + 2);
      const float wgt = (src[D] == -INFINITY) ? 0.f : exp2f(src[D] - M);
      acc = fmaf(wgt, src[d], acc);
      l = fmaf(wgt, src[D + 1], l);
    }
    part[g * (D + 2) + d] = acc;
    if (d == 0) {
      part[g * (D + 2) + D] = M * ln2;     // back to natural-log units
      part[g * (D + 2) + D + 1] = l;
    }
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

template <int D>
static cudaError_t launch_attend_d(const Params &p, cudaStream_t stream) {
  const size_t ring = (size_t)kAttWarps * kVStages * 16 * D * 2;
  const size_t merge = (size_t)kAttWarps * 8 * (D + 2) * sizeof(float);
  const size_t smem = (ring > merge ? ring : merge) + (size_t)kMaxGroupsPerCta * 8;
  cudaError_t e = cudaFuncSetAttribute(attend_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid(p.n_splits, p.B * p.Hkv);
  attend_kernel<D><<<grid, kAttThreads, smem, stream>>>(p);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_attend(const Params &p, cudaStream_t stream) {
  cudaError_t e = p.D == 64 ? launch_attend_d<64>(p, stream) : launch_attend_d<128>(p, stream);
  if (e != cudaSuccess) return e;
  combine_kernel<<<p.B * p.Hq, p.D, 0, stream>>>(p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace cobs
