// The exact-mass selector (the paper's oracle sparse attention, OSA): the log attention mass of every full block
// for every query head by direct summation over the block's keys,
//
//   e[g][b] = ln sum_{t in b} exp(q'_g . k_t)                                   (Eq. bg-defs)
//
// which then goes through the same group score and top-k as the estimates do (Eq. prop-gqa).  It reads every key
// (the work the estimator exists to avoid), so it is a quality reference, not part of the decode step.
//
// One warp per (sequence, KV head, block): the block's keys pass 16 tokens at a time through a two-stage cp.async
// ring of the warp (XOR-swizzled 16-byte chunks, read back with ldmatrix); logits by mma.sync m16n8k16 with the
// heads as rows (zero padded to 16) and 8 tokens as columns; a running (max, sum) per head in registers.
#include "common.cuh"

namespace cobs {

namespace {

constexpr int kEWarps = 8;

__device__ __forceinline__ void cpa16(uint32_t dst, const void *src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src));
}
__device__ __forceinline__ void cpa_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cpa_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldsm_x4(uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float &c0, float &c1, float &c2, float &c3, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c0), "+f"(c1), "+f"(c2), "+f"(c3) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

}  // namespace

template <int D>
__global__ void __launch_bounds__(kEWarps * 32) exact_mass_kernel(Params p) {
  constexpr int CH = D / 8, KS = D / 16, ROWB = D * 2, STAGE = 16 * ROWB, NCP = (16 * CH) / 32;
  extern __shared__ __align__(128) unsigned char esm[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gid = lane >> 2, tig = lane & 3;
  const uint32_t ring = (uint32_t)__cvta_generic_to_shared(esm + warp * 2 * STAGE);
  const int G = p.G, L = p.L, P = p.P, NB = p.NB, gpb = L / 16;
  const long long items = (long long)p.B * p.Hkv * NB;
  const float sl = 1.0f / sqrtf((float)D);
  uint32_t cdst[NCP];
#pragma unroll
  for (int j = 0; j < NCP; ++j) {
    const int i = lane + 32 * j, t = i / CH, c = i - t * CH;
    cdst[j] = t * ROWB + ((c ^ (t & 7)) << 4);
  }
  const int kt = ((lane >> 4) & 1) * 8 + (lane & 7), kc = (lane >> 3) & 1;
  const uint4 *kbase = reinterpret_cast<const uint4 *>(p.k_pages) + lane;
  int cur_u = -1;
  uint32_t qa[KS][2];
  for (long long it = (long long)blockIdx.x * kEWarps + warp; it < items; it += (long long)gridDim.x * kEWarps) {
    const int u = (int)(it / NB), blk = (int)(it - (long long)u * NB);
    const int b_idx = u / p.Hkv, h = u - b_idx * p.Hkv;
    const int T = p.seq_lens[b_idx];
    if (blk >= min(T / L, NB)) continue;         // only full blocks have a mass here, as only they have summaries
    if (u != cur_u) {
      cur_u = u;
      const uint32_t *qg = reinterpret_cast<const uint32_t *>(p.q + ((size_t)b_idx * p.Hq + h * G + gid) * D);
#pragma unroll
      for (int s = 0; s < KS; ++s) {
        qa[s][0] = (gid < G) ? qg[8 * s + tig] : 0u;
        qa[s][1] = (gid < G) ? qg[8 * s + 4 + tig] : 0u;
      }
    }
    auto issue = [&](int g, int st) {
      if (g < gpb) {
        const int tok0 = blk * L + g * 16;
        const int pslot = tok0 / P;                 // < mpp for every full block (mpp * P >= NB * L); checked all the same
        const int pg = (pslot < p.mpp) ? p.page_table[(size_t)b_idx * p.mpp + pslot] : -1;
        if (pg < 0 || pg >= p.n_pages) report(p.status, COBS_ERR_BOUNDS);
        else {
          const uint4 *ks = kbase + ((((size_t)pg * p.Hkv + h) * P + (tok0 % P)) * D) / 8;
#pragma unroll
          for (int j = 0; j < NCP; ++j) cpa16(ring + st * STAGE + cdst[j], ks + 32 * j);
        }
      }
      cpa_commit();
    };
    float m_run = -1e30f, l_run = 0.f, z2 = 0.f, z3 = 0.f;
    issue(0, 0);
    for (int g = 0; g < gpb; ++g) {
      issue(g + 1, (g + 1) & 1);
      cpa_wait<1>();
      __syncwarp();
      const uint32_t sb = ring + (g & 1) * STAGE;
      float s00 = 0.f, s01 = 0.f, s10 = 0.f, s11 = 0.f;
#pragma unroll
      for (int s = 0; s < KS; ++s) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4(b0, b1, b2, b3, sb + kt * ROWB + (((2 * s + kc) ^ (kt & 7)) << 4));
        mma_bf16(s00, s01, z2, z3, qa[s][0], 0u, qa[s][1], 0u, b0, b1);
        mma_bf16(s10, s11, z2, z3, qa[s][0], 0u, qa[s][1], 0u, b2, b3);
      }
      // row gid = head, this lane's four tokens of the group; running max and sum in natural-log units
      const float x0 = s00 * sl, x1 = s01 * sl, x2 = s10 * sl, x3 = s11 * sl;
      const float mx = fmaxf(fmaxf(x0, x1), fmaxf(x2, x3));
      const float m_new = fmaxf(m_run, mx);
      l_run = l_run * __expf(m_run - m_new) + __expf(x0 - m_new) + __expf(x1 - m_new) + __expf(x2 - m_new) + __expf(x3 - m_new);
      m_run = m_new;
      __syncwarp();
    }
    cpa_wait<0>();
    // the four lanes of a head hold different tokens: merge their (max, sum) pairs
#pragma unroll
    for (int o = 1; o <= 2; o <<= 1) {
      const float om = __shfl_xor_sync(0xffffffffu, m_run, o), ol = __shfl_xor_sync(0xffffffffu, l_run, o);
      const float nm = fmaxf(m_run, om);
      l_run = l_run * __expf(m_run - nm) + ol * __expf(om - nm);
      m_run = nm;
    }
    if (gid < G && tig == 0) p.e[((size_t)u * G + gid) * NB + blk] = m_run + logf(l_run);
  }
}

cudaError_t launch_exact_mass(const Params &p, cudaStream_t stream) {
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  const size_t smem = (size_t)kEWarps * 2 * 16 * p.D * 2;
  const long long items = (long long)p.B * p.Hkv * p.NB;
  long long grid = (items + kEWarps - 1) / kEWarps;
  if (grid > 4LL * sms) grid = 4LL * sms;
  if (grid < 1) grid = 1;
  if (p.D == 128) {
    if ((e = cudaFuncSetAttribute(exact_mass_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    exact_mass_kernel<128><<<(unsigned)grid, kEWarps * 32, smem, stream>>>(p);
  } else {
    if ((e = cudaFuncSetAttribute(exact_mass_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    exact_mass_kernel<64><<<(unsigned)grid, kEWarps * 32, smem, stream>>>(p);
  }
  count_launch();
  return cudaGetLastError();
}

}  // namespace cobs
