// The decode step as ONE persistent kernel: block scoring, top-k selection, block-sparse attention
// and the split-KV merge (steps (b), (c), (d)).
//
// Why one kernel.  A step moves a few hundred MiB; at HBM speed that is tens of microseconds, so
// every kernel boundary (launch, ramp-up, tail, the idle time while a single CTA per unit selects)
// costs a visible fraction of the step.  Here the grid is one CTA per SM, fully resident (cooperative
// launch), with two kinds of warps:
//
//   streaming warps (8 per CTA), each with its own slice of shared memory:
//     phase S  score 16-block chunks of summaries: the units are scored in waves, and inside a wave every
//              warp takes one contiguous range of chunks; per chunk it leaves t = exp(e - chunk max) per
//              block and head, the chunk's (max, sum) pair, and counts the chunk on its unit;
//     phase A  attend over (unit, slice) items drawn from one global counter in unit order; a warp whose
//              slice holds selected blocks waits (bounded) for that unit's selection, slices that hold only
//              window blocks never wait; the warp that finishes the last slice of a unit merges the
//              partials and writes the output;
//   a selection team (4 warps per CTA) that selects unit u (team of CTA u mod grid) as soon as all its
//     chunks are counted, while the streaming warps carry on with the next wave.
//
// Data movement.  Every stream a warp consumes goes global -> shared into a ring that belongs to that warp
// alone (no CTA barrier anywhere in the loops).  Scoring: a chunk is three contiguous pieces of the summary
// arrays, fetched by three bulk copies (cp.async.bulk, completion on an mbarrier) issued by one lane, two
// stages.  Attention: K and V of a 16-token group share a stage of a three-stage cp.async ring (XOR-swizzled
// 16-byte chunks, read back with ldmatrix / ldmatrix.trans).
//
// Arithmetic.  mma.sync m16n8k16 with fp32 accumulation throughout:
//   scoring   rows = 16 block means, or factor i of 16 blocks; columns = the G query heads.  A thread
//             owns two blocks (rows gid, gid + 8), so all results of a block land in one thread.
//             bf16 operands multiply the raw bf16 query (exact products); FP4 codes become f16 by
//             the hardware conversion and multiply the query scaled by a per-head power of two
//             (exact in f16), or an f16 high + low split of the fp32 subspace query.
//   attention S^T = q K^T with the heads as rows (zero padded to 16) and 8 tokens as columns; the S
//             accumulators are the A fragments of P V as they sit in registers; P = bf16 high + low.
// An opt-in variant runs phase S of the main configuration on tcgen05 (further down).
//
// Cross-warp hand-offs go through global counters in the workspace (release: write, __threadfence,
// atomicAdd; acquire: volatile read, __threadfence, .cg loads).  Every wait is bounded; on expiry the
// kernel records COBS_ERR_TIMEOUT, skips the dependent work and returns.  The counters come in two sets
// that alternate launches take turns on (ctl_begin), so a workspace needs zeroing only once
// (cobs_reset_status) and nothing is cleaned up when the kernel ends.
#include <cuda.h>
#include <cuda_fp8.h>

#include <cstdlib>
#include <cstring>
#include <mutex>
#include <type_traits>

#include "common.cuh"

namespace cobs {

constexpr int kFWarps = 8;                                   // streaming warps per CTA (score, then attend)
constexpr int kSelWarps = 4;                                 // selection team of the CTA
constexpr int kSelThreads = kSelWarps * 32;
constexpr int kLenCache = 256;                               // sequence lengths cached in shared memory
constexpr int kFThreads = (kFWarps + kSelWarps) * 32;        // one CTA per SM
constexpr int kScoreStageBytes = 14080;                      // means + factor rows + scales of a 16-block chunk
constexpr int kAttStages = 3;
constexpr int kAttStageBytes = 2 * 16 * 128 * 2;             // K + V of one 16-token group, D = 128
// The hand-off counters exist twice.  A launch works on the set named by bit 31 of the epoch word; the low bits of
// that word count the CTAs that have begun.  The CTA that begins last (every other CTA then holds its set number) turns
// the word over for the next launch and clears the other set, which the previous launch left dirty (as far as that
// launch's unit count reached: the word after the epoch word keeps it, so a workspace may serve calls of different
// shapes).  Nothing has to be cleaned up when the kernel ends, and a launch that gave up half-way does not poison
// the next one.  Status block, in ints: 0 status, 1 epoch, 2 / 3 item and barrier words of set 0, 4 extent, 5 / 6
// item and barrier words of set 1.
__shared__ int s_ctl[4];          // offset of this launch's per-unit counters, of its item / barrier words; "begun last"; extent
#define CTL_UNIT(ptr) ((ptr) + s_ctl[0])
#define CTL_MISC(ptr) ((ptr) + s_ctl[1])
__device__ __forceinline__ void ctl_begin(const Params &p) {          // thread 0 of every CTA, before the CTA's first barrier
  const unsigned old = atomicAdd(reinterpret_cast<unsigned *>(p.ctl_epoch), 1u);
  const int set = (int)(old >> 31);
  s_ctl[0] = set * p.ctl_set_stride;
  s_ctl[1] = set * 3;
  s_ctl[2] = (old & 0x7fffffffu) == gridDim.x - 1;
}
__device__ __forceinline__ void ctl_turn(const Params &p) {           // the whole CTA that began last, after that barrier
  const int other_u = s_ctl[0] ? 0 : p.ctl_set_stride, other_m = s_ctl[1] ? 0 : 3;
  if (threadIdx.x == 0) {
    s_ctl[3] = min(*reinterpret_cast<const volatile int *>(p.ctl_epoch + 3), p.ctl_set_stride);   // ints of the other set its last launch used
    atomicAdd(reinterpret_cast<unsigned *>(p.ctl_epoch), 0x80000000u - gridDim.x);     // flips bit 31, zeroes the count
    p.ctl_item[other_m] = 0;
    p.ctl_bar[other_m] = 0;
  }
  __syncthreads();
  const int ext = s_ctl[3];
  for (int i = threadIdx.x; i < ext; i += blockDim.x) p.ctl_score[other_u + i] = 0;     // score, ready, att: contiguous
  if (threadIdx.x == 0) p.ctl_epoch[3] = 3 * p.B * p.Hkv;             // what this launch will leave behind in its set
}

constexpr int kTableEntries = 256;                           // 16-token groups per attention item
constexpr int kRingBytes = (2 * kScoreStageBytes > kAttStages * kAttStageBytes + kTableEntries * 8)
                               ? 2 * kScoreStageBytes : kAttStages * kAttStageBytes + kTableEntries * 8;
constexpr int kWarpSmemBytes = kRingBytes;                   // 28160
constexpr int kFusedSmemBytes = kFWarps * kWarpSmemBytes;    // 225280: one CTA per SM
constexpr long long kSpinLimit = 4000000;                    // x ~100 ns: bounded wait on another warp

enum { PH_SCORE = 1, PH_ATTEND = 2 };
constexpr int kWaves = 4;                                    // the units are scored in this many waves
constexpr int kScoreRowGroup = 4;                            // FP4 factor rows decoded and multiplied together

// Phase timing (the build with -DCOBS_TIMING, `python -m paper_2607_09052_b200.build --timing`, which makes
// libcobs_timing.so; read by `bench.py --phase-times`): every streaming warp records the global timer at its phase
// boundaries and accumulates clock cycles per category inside the phases; the selection teams record when a unit
// was complete and when its selection was published.  The production library carries none of this.
#ifdef COBS_TIMING
__device__ unsigned long long g_dbg_times[4][4096];   // [start | scoring done | attention start | attention done][warp]
__device__ unsigned long long g_dbg_acc[8][4096];     // accumulated clock cycles by category: attention [warp], scoring
                                                      // [1200 + warp]; selection stamps (ns) [3000 + unit]
__device__ __forceinline__ unsigned long long gtime() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
#define COBS_STAMP(k) do { if (lane == 0 && wg < 4096) g_dbg_times[k][wg] = gtime(); } while (0)
#define COBS_SEL_STAMP(k) do { if (tid == 0 && u < 1024) g_dbg_acc[k][3000 + u] = gtime(); } while (0)
#define COBS_ACC_DECL long long acc_t[8] = {0,0,0,0,0,0,0,0}; long long acc_last = clock64()
#define COBS_ACC(k) do { long long now_ = clock64(); acc_t[k] += now_ - acc_last; acc_last = now_; } while (0)
#define COBS_ACC_FLUSH(id) do { if ((threadIdx.x & 31) == 0 && (id) < 4096) { for (int k_ = 0; k_ < 8; ++k_) g_dbg_acc[k_][id] += acc_t[k_]; } } while (0)
#else
#define COBS_ACC_DECL do { } while (0)
#define COBS_ACC(k) do { } while (0)
#define COBS_ACC_FLUSH(id) do { } while (0)
#define COBS_STAMP(k) do { } while (0)
#define COBS_SEL_STAMP(k) do { } while (0)
#endif


// ---------------------------------------------------------------------------------------------------
// small PTX helpers
// ---------------------------------------------------------------------------------------------------
// The summaries and the selected K / V are read exactly once per step: their copies carry an L2 evict-first policy,
// so that they do not push the step's small shared state (block scores, chunk pairs, selections, split partials,
// flags: written by one warp, read by another a few microseconds later) out of L2 and into the HBM queues.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void cpa16(uint32_t dst, const void *src, uint64_t pol) {
  asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "l"(pol));
}
__device__ __forceinline__ void cpa16z(uint32_t dst, const void *src, int bytes, uint64_t pol) {
  asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2, %3;\n" ::"r"(dst), "l"(src), "r"(bytes), "l"(pol));
}
__device__ __forceinline__ void cpa4(uint32_t dst, const void *src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;\n" ::"r"(dst), "l"(src));
}
__device__ __forceinline__ void cpa_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cpa_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];\n" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}
__device__ __forceinline__ float lds_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ void mma16816_bf16(float &c0, float &c1, float &c2, float &c3, uint32_t a0, uint32_t a1,
                                              uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c0), "+f"(c1), "+f"(c2), "+f"(c3)
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma16816_f16(float &c0, float &c1, float &c2, float &c3, uint32_t a0, uint32_t a1,
                                             uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c0), "+f"(c1), "+f"(c2), "+f"(c3)
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void ldsm_x4(uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// Eight E2M1 codes -> four f16x2 (code 2 i in the low half of h[i], code 2 i + 1 in the high half).
__device__ __forceinline__ void e2m1x8_to_f16(uint32_t w, uint32_t (&h)[4]) {
  asm("{\n .reg .b8 b0, b1, b2, b3;\n mov.b32 {b0, b1, b2, b3}, %4;\n cvt.rn.f16x2.e2m1x2 %0, b0;\n"
      " cvt.rn.f16x2.e2m1x2 %1, b1;\n cvt.rn.f16x2.e2m1x2 %2, b2;\n cvt.rn.f16x2.e2m1x2 %3, b3;\n}\n"
      : "=r"(h[0]), "=r"(h[1]), "=r"(h[2]), "=r"(h[3]) : "r"(w));
}
__device__ __forceinline__ uint32_t f16x2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t *>(&h);
}
__device__ __forceinline__ uint32_t bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];\n" : "=r"(v) : "r"(addr));
  return v;
}
// ---- mbarrier + bulk copy (global -> shared, completion counted in bytes on an mbarrier) -----------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar, uint64_t pol) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;\n"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(pol) : "memory");
}
// Wait for the phase with the given parity to complete.  Bounded; false on expiry.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (int it = 0; it < 20000000; ++it) {
    uint32_t done;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    if (done) return true;
  }
  return false;
}
__device__ __forceinline__ int ld_volatile(const int *p) { return *reinterpret_cast<const volatile int *>(p); }

// Wait until *flag != 0 (set by another warp of the grid).  Bounded; false on expiry.
__device__ __forceinline__ bool wait_flag(const int *flag) {
  for (long long it = 0; it < kSpinLimit; ++it) {
    if (ld_volatile(flag) != 0) return true;
    __nanosleep(100);
  }
  return false;
}

// ---------------------------------------------------------------------------------------------------
// Selection.  Every CTA has a team of four warps that does nothing but select: unit u is selected by the team
// of CTA u mod gridDim.x as soon as all chunks of the unit are scored, while the CTA's streaming warps carry on
// scoring later units (the selection is a chain of short dependent steps; it runs in issue slots the streaming
// warps leave idle).  Scoring left, per block, t = exp(e - chunk max) and, per chunk, (max, sum of t):
//   lse_g   = log-sum-exp over the chunks of head g
//   score_b = sum_g t[g][b] * exp(chunk max[g] - lse_g)          (= sum_g exp(e[g][b] - lse_g))
// then the k largest scores among the candidate blocks, lower index on ties, ascending output.
// ---------------------------------------------------------------------------------------------------
__device__ __forceinline__ void team_sync() { asm volatile("bar.sync 1, %0;\n" ::"n"(kSelThreads) : "memory"); }

// Selection of one unit of at most 128 * BPT summarised blocks (BPT = 4, 8 or 16): thread t of the CTA's selection
// team owns blocks BPT t ... BPT t + BPT - 1 (a part of chunk BPT t / 16, or all of chunk t), so that with few
// blocks all four warps still hold keys and every loop over a thread's keys is short.  The global loads (the chunk
// pairs, the maxima of this thread's own chunk parts, its t values of the first heads) are issued before the first
// use: one round trip.  Needs NB % 4 == 0.
// PPC: (max, sum) pairs per 16-block chunk and head left by the scoring path (1, or 4 = one per four blocks).
template <int PPC, int BPT>
__device__ void select_unit(const Params &p, int u, int n_sum, int n_cand, int tid, int part) {
  static_assert(BPT == 4 || BPT == 8 || BPT == 16, "blocks per thread");
  static_assert(kSelWarps == 4, "one 16-byte read takes the four warps' words");
  constexpr int NQ = BPT / 4;                    // groups of four blocks of a thread
  constexpr int GB = (BPT == 16) ? 4 : 8;        // heads whose t values are in registers at a time
  constexpr int CW = (BPT == 4) ? 1 : 2;         // words the three counts of a bisection round are packed in
  __shared__ float s_m[8][kSelWarps], s_s[8][kSelWarps];
  __shared__ __align__(16) uint32_t s_cnt[2][2][kSelWarps];
  __shared__ int s_scan[kSelWarps];
  const int warp = tid >> 5, lane = tid & 31;
  const int G = p.G, NB = p.NB, cpu = (NB + 15) / 16, n_chunks = (n_sum + 15) / 16;
  const int b0 = tid * BPT, c_own = b0 >> 4, part0 = (b0 & 15) >> 2;
  const bool mine = b0 < n_sum, loader = tid < n_chunks;
  const float2 *pp = reinterpret_cast<const float2 *>(p.lse_part) + (size_t)u * G * cpu * PPC;
  const float *tu = p.e + (size_t)u * G * NB + b0;
  // ---- loads -------------------------------------------------------------------------------------------------
  float2 pr[8];                                  // (max, sum) of chunk `tid`, per head (threads below n_chunks)
  float own_m[8][NQ];                            // max of the chunk part each of this thread's groups lies in
  float4 x[GB][NQ];
  float sc[BPT];
  uint32_t keys[BPT];
#pragma unroll
  for (int j = 0; j < BPT; ++j) { sc[j] = 0.f; keys[j] = 0u; }
  // part < 0: the selection proper.  part = 0 .. 3: a rehearsal of one quarter of this code by one warp alone (no
  // barrier, nothing written), see select_team.
  const bool real = part < 0, dry = !real;
  auto load_t = [&](int g0) {
#pragma unroll
    for (int g = 0; g < GB; ++g)
#pragma unroll
      for (int q = 0; q < NQ; ++q)
        x[g][q] = (g0 + g < G && b0 + 4 * q < n_sum) ? __ldcg(reinterpret_cast<const float4 *>(tu + (size_t)(g0 + g) * NB) + q)
                                                     : make_float4(0.f, 0.f, 0.f, 0.f);
  };
#pragma unroll
  for (int g = 0; g < 8; ++g) {
    pr[g] = make_float2(-INFINITY, 0.f);
#pragma unroll
    for (int q = 0; q < NQ; ++q) own_m[g][q] = -INFINITY;
  }
#pragma unroll
  for (int g = 0; g < GB; ++g)
#pragma unroll
    for (int q = 0; q < NQ; ++q) x[g][q] = make_float4(0.f, 0.f, 0.f, 0.f);
  if (real || part == 0) {
#pragma unroll
  for (int g = 0; g < 8; ++g) {
    if (g < G) {
      if (PPC == 1) {
        if (loader) pr[g] = __ldcg(pp + (size_t)g * cpu + tid);
        if (mine) {
          const float m = (BPT == 16) ? pr[g].x : __ldcg(pp + (size_t)g * cpu + c_own).x;
#pragma unroll
          for (int q = 0; q < NQ; ++q) own_m[g][q] = m;
        }
      } else {
        float2 part[PPC];
#pragma unroll
        for (int j = 0; j < PPC; ++j) part[j] = make_float2(-INFINITY, 0.f);
        if (loader) {
#pragma unroll
          for (int j = 0; j < PPC; j += 2) {
            const float4 v = __ldcg(reinterpret_cast<const float4 *>(pp + ((size_t)g * cpu + tid) * PPC + j));
            part[j] = make_float2(v.x, v.y);
            part[j + (PPC > 1 ? 1 : 0)] = make_float2(v.z, v.w);
          }
          float m = -INFINITY;
#pragma unroll
          for (int j = 0; j < PPC; ++j) m = fmaxf(m, part[j].x);
          float sum = 0.f;
#pragma unroll
          for (int j = 0; j < PPC; ++j) sum += (part[j].x == -INFINITY) ? 0.f : part[j].y * __expf(part[j].x - m);
          pr[g] = make_float2(m, sum);
        }
        if (mine) {
#pragma unroll
          for (int q = 0; q < NQ; ++q)
            own_m[g][q] = (BPT == 16) ? part[q < PPC ? q : 0].x : __ldcg(pp + ((size_t)g * cpu + c_own) * PPC + part0 + q).x;
        }
      }
    }
  }
  load_t(0);
  // ---- log-sum-exp per head: warp maximum by an integer reduction on the order-preserving bit pattern ----------
#pragma unroll
  for (int g = 0; g < 8; ++g) {
    if (g < G) {
      int im = __float_as_int(pr[g].x);
      im ^= (im >> 31) & 0x7fffffff;
      im = __reduce_max_sync(0xffffffffu, im);
      im ^= (im >> 31) & 0x7fffffff;
      const float M = __int_as_float(im);
      float sum = (pr[g].x == -INFINITY) ? 0.f : pr[g].y * __expf(pr[g].x - M);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      if (lane == 0) { s_m[g][warp] = M; s_s[g][warp] = sum; }
    }
  }
  }
  COBS_SEL_STAMP(2);
  if (real) team_sync();
  // ---- scores of this thread's blocks: score_b = sum_g t[g][b] * exp(part max[g] - lse_g) -----------------------
  if (real || part == 1) {
#pragma unroll
  for (int g0 = 0; g0 < 8; g0 += GB) {
    if (g0 < G) {
      if (g0 > 0) load_t(g0);
#pragma unroll
      for (int gg = 0; gg < GB; ++gg) {
        const int g = g0 + gg;
        if (g < G) {
          float M = -INFINITY;
#pragma unroll
          for (int q = 0; q < kSelWarps; ++q) M = fmaxf(M, s_m[g][q]);
          float S = 0.f;
#pragma unroll
          for (int q = 0; q < kSelWarps; ++q) S += (s_m[g][q] == -INFINITY) ? 0.f : s_s[g][q] * __expf(s_m[g][q] - M);
          const float lse = M + __logf(S);              // fast forms: a few instructions instead of dozens (this code runs cold)
#pragma unroll
          for (int q = 0; q < NQ; ++q) {
            const float wq = (own_m[g][q] != -INFINITY) ? __expf(own_m[g][q] - lse) : 0.f;
            sc[4 * q + 0] = fmaf(x[gg][q].x, wq, sc[4 * q + 0]); sc[4 * q + 1] = fmaf(x[gg][q].y, wq, sc[4 * q + 1]);
            sc[4 * q + 2] = fmaf(x[gg][q].z, wq, sc[4 * q + 2]); sc[4 * q + 3] = fmaf(x[gg][q].w, wq, sc[4 * q + 3]);
          }
        }
      }
    }
  }
#pragma unroll
  for (int j = 0; j < BPT; ++j) {
    const int b = b0 + j;
    if (b >= n_sum) sc[j] = 0.f;                 // beyond the summarised blocks nothing was written
    if (p.scores && b < n_sum && !dry) p.scores[(size_t)u * NB + b] = sc[j];
    keys[j] = (b < n_cand) ? __float_as_uint(sc[j]) : 0u;
  }
  }
  COBS_SEL_STAMP(3);
  // ---- top-k ------------------------------------------------------------------------------------------------
  int32_t *out = p.sel_idx + (size_t)u * p.topk;
  const int k = min(p.topk, n_cand);
  uint32_t theta = 0u;
  if (real) {
    if (tid == 0) p.sel_cnt[u] = k;
    for (int i = k + tid; i < p.topk; i += kSelThreads) out[i] = -1;
    if (k == n_cand) {
      for (int i = tid; i < k; i += kSelThreads) out[i] = i;
      return;
    }
  }
  if (real || part == 2) {
  // k-th largest key by bisection on its bits (scores are >= 0, so their bit patterns order like integers):
  // theta = the largest T with #(key >= T) >= k.  Bit 30 alone, then two bits per round: three trial values, whose
  // counts travel packed as unsigned fields (11, 11 and 10 bits of one word while a team holds at most 512 keys - no
  // field can reach its width - else 16 bits each in two words): per round one or two warp reductions, one shared
  // store per warp, one barrier, one 16-byte read per word.
  constexpr int SH = (CW == 1) ? 11 : 16, SH2 = (CW == 1) ? 22 : 0;
  static_assert(CW == 2 || kSelThreads * BPT < (1 << 10), "a packed count would overflow its field");
  int par = 0;
  auto cta_sum = [&](uint32_t c0, uint32_t c1, uint32_t &n0, uint32_t &n1) {
    c0 = __reduce_add_sync(0xffffffffu, c0);
    if (CW == 2) c1 = __reduce_add_sync(0xffffffffu, c1);
    if (lane == 0) { s_cnt[par][0][warp] = c0; if (CW == 2) s_cnt[par][1][warp] = c1; }
    if (real) team_sync();
    const uint4 v = *reinterpret_cast<const uint4 *>(&s_cnt[par][0][0]);
    n0 = v.x + v.y + v.z + v.w;
    n1 = 0;
    if (CW == 2) {
      const uint4 w = *reinterpret_cast<const uint4 *>(&s_cnt[par][1][0]);
      n1 = w.x + w.y + w.z + w.w;
    }
    par ^= 1;
  };
  {
    const uint32_t t = 1u << 30;
    uint32_t c = 0, n0, n1;
#pragma unroll
    for (int j = 0; j < BPT; ++j) c += (keys[j] >= t);
    cta_sum(c, 0u, n0, n1);
    if (n0 >= (uint32_t)k) theta = t;
  }
  for (int bit = 29; bit >= 1; bit -= 2) {
    const uint32_t ta = theta | (3u << (bit - 1)), tb = theta | (2u << (bit - 1)), tc = theta | (1u << (bit - 1));
    uint32_t c0 = 0, c1 = 0, n0, n1;
#pragma unroll
    for (int j = 0; j < BPT; ++j) {
      c0 += (keys[j] >= ta ? 1u : 0u) + (keys[j] >= tb ? (1u << SH) : 0u);
      if (CW == 1) c0 += (keys[j] >= tc ? (1u << SH2) : 0u);
      else c1 += (keys[j] >= tc ? 1u : 0u);
    }
    cta_sum(c0, c1, n0, n1);
    const uint32_t ku = (uint32_t)k;
    const uint32_t na = n0 & ((1u << SH) - 1), nb = (n0 >> SH) & ((1u << SH) - 1), nc = (CW == 1) ? (n0 >> SH2) : n1;
    if (na >= ku) theta = ta; else if (nb >= ku) theta = tb; else if (nc >= ku) theta = tc;
  }
  }
  COBS_SEL_STAMP(4);
  if (real || part == 3) {
  // keep every key above theta and the lowest-index `need_eq` keys equal to it, in index order: one scan of the
  // packed (above, equal) counts gives both the totals and this thread's position
  int v = 0;
#pragma unroll
  for (int j = 0; j < BPT; ++j)
    if (b0 + j < n_cand) v += (keys[j] > theta ? (1 << 16) : 0) + (keys[j] == theta ? 1 : 0);
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) s_scan[warp] = inc;
  if (real) team_sync();
  int base = 0, total = 0;
#pragma unroll
  for (int q = 0; q < kSelWarps; ++q) { const int t = s_scan[q]; total += t; base += (q < warp) ? t : 0; }
  const int need_eq = max(k - (total >> 16), 0);
  const int excl = base + inc - v;
  int eq_rank = excl & 0xffff;
  int pos = (excl >> 16) + min(eq_rank, need_eq);
#pragma unroll
  for (int j = 0; j < BPT; ++j) {
    if (b0 + j < n_cand) {
      bool keep = false;
      if (keys[j] > theta) keep = true;
      else if (keys[j] == theta) { keep = eq_rank < need_eq; ++eq_rank; }
      if (keep && pos >= 0 && pos < k && !dry) out[pos++] = b0 + j;
    }
  }
  }
  COBS_SEL_STAMP(5);
}

// count_mult: how often the scoring path counts a chunk on its unit; empty_need: the count a unit without
// summarised blocks reaches.
template <int PPC>
__device__ void select_team(const Params &p, const int *seq_lens, int tid, int count_mult, int empty_need) {
  __shared__ int s_ok;
  const int units = p.B * p.Hkv;
  // The first pass over the first unit is a rehearsal: the same code on whatever the workspace holds, nothing written,
  // run while the unit is still being scored, each of the team's four warps taking one quarter of it.  The
  // selection is executed once or twice per CTA and launch, so its instructions are never in the SM's instruction
  // cache when it is needed, and after other work has swept L2 they come from HBM, one dependent miss after
  // another (measured: 16 us for a selection that takes 5 us once its code is near); rehearsed in four parallel
  // pieces, the real pass finds them close by.
  bool rehearsal = true;
  for (int u = blockIdx.x; u < units;) {
    const int T = seq_lens[u / p.Hkv];
    const int n_sum = min(T / p.L, p.NB);
    const int n_cand = min(window_start(T, p.window, p.L) / p.L, n_sum);
    const int n_chunks = (n_sum + 15) / 16;
    if (!rehearsal) {
      if (tid == 0) {
        int ok = 0;
        for (long long it = 0; it < kSpinLimit; ++it) {
          if (ld_volatile(CTL_UNIT(p.ctl_score) + u) >= (n_chunks > 0 ? n_chunks * count_mult : empty_need)) { ok = 1; break; }
          __nanosleep(200);
        }
        if (!ok) report(p.status, COBS_ERR_TIMEOUT);
        s_ok = ok;
      }
      team_sync();
      const int ok = s_ok;
      team_sync();
      if (!ok) { u += gridDim.x; continue; }     // never scored: leave the unit unselected (its attention times out too)
      __threadfence();
      COBS_SEL_STAMP(0);
    }
    const int part = rehearsal ? (tid >> 5) : -1;
    if (n_sum <= kSelThreads * 4) select_unit<PPC, 4>(p, u, n_sum, n_cand, tid, part);
    else if (n_sum <= kSelThreads * 8) select_unit<PPC, 8>(p, u, n_sum, n_cand, tid, part);
    else select_unit<PPC, 16>(p, u, n_sum, n_cand, tid, part);
    team_sync();
    if (rehearsal) { rehearsal = false; continue; }
    __threadfence();
    team_sync();
    if (tid == 0) atomicExch(CTL_UNIT(p.ctl_ready) + u, 1);
    COBS_SEL_STAMP(1);
    u += gridDim.x;
  }
}

// Curvature term of a 16-block chunk whose packed E2M1 rows are full width (128 codes: one 16-byte read per thread and
// row) and whose rank R is a multiple of four: no clamps or row tests, four rows (four independent accumulator chains) at
// a time, the four scales of a block read in one go.  xa / xb: this thread's 16 bytes of row 0 of blocks 2 gid and
// 2 gid + 1 (rows 64 bytes apart); sp: the scales of block 2 gid (those of block 2 gid + 1 follow them).
// Adds sum_i (scale_i * (xi_i . q))^2 per block and head; the query's per-head factor is applied by the caller.
template <int R, bool SCALE_F32>
__device__ __forceinline__ void fp4_rows_full_width(uint32_t xa, uint32_t xb, uint32_t sp, const uint32_t (&bq)[8][2], float &sA0,
                                                    float &sA1, float &sB0, float &sB1) {
  static_assert(R % 4 == 0, "whole groups of four rows");
#pragma unroll 1                                 // rolled: half the code at rank 8 (instruction fetch is a visible stall of this kernel)
  for (int i0 = 0; i0 < R; i0 += 4) {
    uint4 wa[4], wb[4];
    float d[4][4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      wa[k] = lds128(xa + (i0 + k) * 64);
      wb[k] = lds128(xb + (i0 + k) * 64);
      d[k][0] = d[k][1] = d[k][2] = d[k][3] = 0.f;
    }
    float sa[4], sb[4];
    if (SCALE_F32) {
      const uint4 a = lds128(sp + i0 * 4), b = lds128(sp + R * 4 + i0 * 4);
      sa[0] = __uint_as_float(a.x); sa[1] = __uint_as_float(a.y); sa[2] = __uint_as_float(a.z); sa[3] = __uint_as_float(a.w);
      sb[0] = __uint_as_float(b.x); sb[1] = __uint_as_float(b.y); sb[2] = __uint_as_float(b.z); sb[3] = __uint_as_float(b.w);
    } else {
      const uint2 a = lds64(sp + i0 * 2), b = lds64(sp + R * 2 + i0 * 2);
      const float2 a0 = __half22float2(*reinterpret_cast<const __half2 *>(&a.x)), a1 = __half22float2(*reinterpret_cast<const __half2 *>(&a.y));
      const float2 b0 = __half22float2(*reinterpret_cast<const __half2 *>(&b.x)), b1 = __half22float2(*reinterpret_cast<const __half2 *>(&b.y));
      sa[0] = a0.x; sa[1] = a0.y; sa[2] = a1.x; sa[3] = a1.y;
      sb[0] = b0.x; sb[1] = b0.y; sb[2] = b1.x; sb[3] = b1.y;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        uint32_t ha[4], hb[4];
        e2m1x8_to_f16(j == 0 ? wa[k].x : j == 1 ? wa[k].y : j == 2 ? wa[k].z : wa[k].w, ha);
        e2m1x8_to_f16(j == 0 ? wb[k].x : j == 1 ? wb[k].y : j == 2 ? wb[k].z : wb[k].w, hb);
        mma16816_f16(d[k][0], d[k][1], d[k][2], d[k][3], ha[0], hb[0], ha[1], hb[1], bq[2 * j][0], bq[2 * j][1]);
        mma16816_f16(d[k][0], d[k][1], d[k][2], d[k][3], ha[2], hb[2], ha[3], hb[3], bq[2 * j + 1][0], bq[2 * j + 1][1]);
      }
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float d0 = d[k][0] * sa[k], d1 = d[k][1] * sa[k], d2 = d[k][2] * sb[k], d3 = d[k][3] * sb[k];
      sA0 = fmaf(d0, d0, sA0); sA1 = fmaf(d1, d1, sA1); sB0 = fmaf(d2, d2, sB0); sB1 = fmaf(d3, d3, sB1);
    }
  }
}

// ---------------------------------------------------------------------------------------------------
// phase S: scoring (+ selection by the warp that completes a unit)
// DT: COBS_SUMM_BF16 | COBS_SUMM_FP4_E2M1.  WPT: 32-bit words of codes per thread per FP4 row
// (Ds_pad / 32).  NT: f16 terms of the query (1: full space, 2: fp32 subspace query).
// ---------------------------------------------------------------------------------------------------
// Returns false when a wait for this warp's own copies ran out (COBS_ERR_TIMEOUT is recorded): copies may then still
// be on their way into the warp's ring, so the caller must not reuse it.
template <int DT, int D, int WPT, int NT>
__device__ bool score_phase(const Params &p, const int *seq_lens, unsigned char *wsm, uint64_t *bars, int wg, int n_wg,
                            int lane) {
  constexpr bool FP4 = (DT == COBS_SUMM_FP4_E2M1);
  constexpr int MCH = D / 32;                 // 16-byte chunks of a bf16 row per thread
  constexpr int KSM = D / 16;                 // k-steps of a bf16 row
  constexpr int KSQ = FP4 ? WPT * 2 : 1;      // k-steps of an FP4 row
  // stage layout: [16 block means, row stride MROW][16 blocks x rows of factors, block stride XS][scales]
  // The +32 bytes of padding per row / block put the rows of neighbouring quads in different bank halves.
  constexpr int MROW = D * 2 + 32;
  constexpr int MEAN_BYTES = 16 * MROW;
  constexpr int ROWB = FP4 ? WPT * 16 : D * 2;                 // bytes of one factor row
  constexpr int ROWS_CAP = (kScoreStageBytes - 16 * 32) / (16 * ROWB);
  constexpr int ROWS_MAX = ROWS_CAP < COBS_MAX_RANK ? ROWS_CAP : COBS_MAX_RANK;   // rows a batch can hold at most
  static_assert((kScoreStageBytes - MEAN_BYTES - 16 * 32 - 16 * COBS_MAX_RANK * 4) / (16 * ROWB) >= 1, "stage too small");
  const int gid = lane >> 2, tig = lane & 3;
  const int G = p.G, r = p.r, NB = p.NB, L = p.L;
  const int units = p.B * p.Hkv;
  const int cpu = (NB + 15) / 16;             // chunks per unit
  const int scale_sz = (p.scale_dtype == COBS_SCALE_FP16) ? 2 : 4;
  const int scale_bytes = FP4 ? 16 * r * scale_sz : 0;        // scales of a chunk, at the end of the stage
  // Common case: means, all r factor rows and scales of the 16 blocks fit one stage.  Then a chunk is three
  // contiguous pieces of the summary arrays and is fetched by three bulk copies in memory layout (`single`).
  // Otherwise the factor rows go in batches, each block copied on its own to a padded position.
  const bool single = 16 * D * 2 + 16 * r * ROWB + scale_bytes <= kScoreStageBytes && r <= ROWS_MAX;
  const int ROWS0 = single ? r : min(ROWS_MAX, (kScoreStageBytes - MEAN_BYTES - 16 * 32 - scale_bytes) / (16 * ROWB));
  const int ROWSN = min(ROWS_MAX, (kScoreStageBytes - 16 * 32 - scale_bytes) / (16 * ROWB));
  const int mrow = single ? D * 2 : MROW;                                  // row stride of the mean area
  const int mean_bytes = 16 * mrow;
  const int XS0 = single ? r * ROWB : ROWS0 * ROWB + 32, XSN = ROWSN * ROWB + 32;   // block stride of the factor area
  const int n_batches = (r <= ROWS0) ? 1 : 1 + (r - ROWS0 + ROWSN - 1) / ROWSN;
  const uint32_t ring = (uint32_t)__cvta_generic_to_shared(wsm);
  const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(bars);
  const float inv_sqrt_d = 1.0f / sqrtf((float)D);
  const float ln_l = (float)(31 - __clz(L)) * 0.6931471805599453f;      // L is a power of two

  // Work order.  The units are scored in kWaves waves (first half, second half); within a wave every streaming
  // warp takes one contiguous range of the wave's chunks (mostly one unit: its query fragments are built once, and
  // its finished chunks are counted once).  The selection teams pick up a wave's units while the next wave is being
  // scored - or, for the last wave, while the first wave's units are being attended.
  // A position is (unit, chunk-in-unit, blocks of the unit); 32-bit arithmetic throughout.
  auto unit_blocks = [&](int u) -> int { return min(seq_lens[u / p.Hkv] / L, NB); };
  // waves only when there is enough work to keep every warp busy in each of them: with fewer chunks than warps a
  // wave would serialise chunks on a few warps while the rest idle
  const int n_waves = max(1, min(min(kWaves, units / 2), (units * cpu) / n_wg));
  int wave = 0, c_end = 0;
  auto wave_range = [&](int w, int &cb, int &ce) {          // this warp's chunk range [cb, ce) in wave w
    const int u0 = (units * w) / n_waves, u1 = (units * (w + 1)) / n_waves;
    const int tot = (u1 - u0) * cpu;                       // the host refuses configurations where this overflows
    // ceil-sized ranges: at the benchmark's size this leaves the last 20 CTAs without scoring work; they start on the
    // attention of the first selected units while the others still score.  Equal shares for every warp end the
    // scoring 5 us earlier and the step 4 us later (measured, several forms): the warps then reach the attention
    // phase together, before most selections are published, and move through it in lockstep.
    const int per = (tot + n_wg - 1) / n_wg;
    cb = u0 * cpu + min(wg * per, tot);
    ce = u0 * cpu + min(wg * per + per, tot);
  };
  // first position at or after (u, ck) that holds work, moving on to the next wave's range when this one is
  // exhausted; u = units when there is nothing left.  Chunk 0 of a unit without summarised blocks counts as work:
  // its warp counts it, so that the selection sees the unit as scored.
  auto seek = [&](int &u, int &ck, int &n_sum) {
    for (;;) {
      while (u < units && u * cpu + ck < c_end) {
        if (ck * 16 < n_sum || ck == 0) return;
        ++u; ck = 0;                           // rest of this unit has no summaries
        if (u < units) n_sum = unit_blocks(u);
      }
      if (++wave >= n_waves) { u = units; return; }
      int cb;
      wave_range(wave, cb, c_end);
      u = cb / cpu; ck = cb - u * cpu;
      if (u < units) n_sum = unit_blocks(u);
    }
  };

  COBS_ACC_DECL;
  const uint64_t pol = l2_evict_first_policy();
  // ---- bulk copies of (chunk c, batch b) into stage st; completion is counted on the stage's mbarrier ----
  // lanes 0-15 copy the factor rows of block `lane`, lanes 16-31 the mean of block `lane - 16`, lane 0 the scales
  auto issue = [&](int u, int ck, int n_sum, int b, int st) {
    if (u >= units) return;
    if (ck * 16 >= n_sum) return;
    const int nblk = min(16, NB - ck * 16);
    const size_t rec0 = (size_t)u * NB + ck * 16;
    const int row0 = (b == 0) ? 0 : ROWS0 + (b - 1) * ROWSN;
    const int rows = min(r - row0, (b == 0) ? ROWS0 : ROWSN);
    const uint32_t sbase = ring + st * kScoreStageBytes;
    const uint32_t xoff = (b == 0) ? mean_bytes : 0;
    const uint32_t xs = (b == 0) ? XS0 : XSN;
    const uint32_t soff = kScoreStageBytes - scale_bytes;
    const bool scales_bulk = FP4 && nblk == 16 && r > 0;
    const uint32_t bar = bar0 + st * 8;
    if (lane == 0) {
      uint32_t tx = (uint32_t)nblk * (uint32_t)(rows > 0 ? rows * ROWB : 0);
      if (b == 0) tx += (uint32_t)nblk * (D * 2);
      if (scales_bulk) tx += (uint32_t)(16 * r * scale_sz);
      mbar_expect_tx(bar, tx);
      if (single) {                            // the whole chunk: three contiguous pieces, one lane issues them
        bulk_g2s(sbase, (const char *)p.mean + rec0 * (size_t)(D * 2), nblk * D * 2, bar, pol);
        if (rows > 0) bulk_g2s(sbase + xoff, (const char *)p.xi + rec0 * r * (size_t)ROWB, nblk * r * ROWB, bar, pol);
        if (scales_bulk) bulk_g2s(sbase + soff, (const char *)p.scale + rec0 * (size_t)(r * scale_sz), 16 * r * scale_sz, bar, pol);
      }
    }
    COBS_ACC(5);
    if (single) {
      if (FP4 && r > 0 && !scales_bulk) {      // ragged last chunk of the array: plain loads, 4 bytes at a time
        const char *ssrc = (const char *)p.scale + rec0 * (size_t)(r * scale_sz);
        for (int w = lane * 4; w < nblk * r * scale_sz; w += 128)
          *reinterpret_cast<uint32_t *>(wsm + st * kScoreStageBytes + soff + w) = *reinterpret_cast<const uint32_t *>(ssrc + w);
      }
      return;
    }
    __syncwarp();
    if (lane < 16) {
      if (lane < nblk && rows > 0)
        bulk_g2s(sbase + xoff + lane * xs, (const char *)p.xi + ((rec0 + lane) * r + row0) * (size_t)ROWB, rows * ROWB, bar, pol);
    } else if (b == 0 && lane - 16 < nblk) {
      bulk_g2s(sbase + (lane - 16) * mrow, (const char *)p.mean + (rec0 + lane - 16) * (size_t)(D * 2), D * 2, bar, pol);
    }
    if (FP4 && r > 0) {
      const char *ssrc = (const char *)p.scale + rec0 * (size_t)(r * scale_sz);
      if (scales_bulk) {
        if (lane == 2) bulk_g2s(sbase + soff, ssrc, 16 * r * scale_sz, bar, pol);
      } else {                                // ragged last chunk of the array: plain loads, 4 bytes at a time
        for (int w = lane * 4; w < nblk * r * scale_sz; w += 128)
          *reinterpret_cast<uint32_t *>(wsm + st * kScoreStageBytes + soff + w) = *reinterpret_cast<const uint32_t *>(ssrc + w);
      }
    }
  };

  int cu, cck, cn = 0;                                        // current position and its unit's block count
  {
    int cb;
    wave_range(0, cb, c_end);
    cu = cb / cpu; cck = cb - cu * cpu;
    if (cu < units) cn = unit_blocks(cu);
    seek(cu, cck, cn);
  }
  int cur_b = 0, st = 0;
  uint32_t phase_bits = 0;                  // bit st = parity to wait for on stage st
  int pend_u = -1, pend_n = 0;              // chunks finished but not yet counted (counted once per unit run)
  issue(cu, cck, cn, 0, 0);
  // per-chunk state
  uint32_t bm[KSM][2];
  uint32_t bq[FP4 ? NT : 1][KSQ][2];
  float m0 = 0.f, m1 = 0.f;
  float fA0 = 0.f, fA1 = 0.f, fB0 = 0.f, fB1 = 0.f, sA0 = 0.f, sA1 = 0.f, sB0 = 0.f, sB1 = 0.f;
  int cur_u = -1;
  bool alive = true;

  while (cu < units && alive) {
    COBS_ACC(0);
    // ---- prefetch the next batch of this warp --------------------------------------------------------
    int nu = cu, nck = cck, nn = cn, nxt_b = cur_b + 1;
    if (nxt_b >= n_batches) {
      nxt_b = 0;
      if (++nck >= cpu) { ++nu; nck = 0; if (nu < units) nn = unit_blocks(nu); }
      seek(nu, nck, nn);
    }
    COBS_ACC(6);
    issue(nu, nck, nn, nxt_b, st ^ 1);
    COBS_ACC(1);

    const int u = cu, ck = cck, n_sum = cn;
    const uint32_t sbase = ring + st * kScoreStageBytes;
    if (ck * 16 < n_sum) {
      if (!mbar_wait(bar0 + st * 8, (phase_bits >> st) & 1u)) {     // bounded: the copies never landed
        if (lane == 0) report(p.status, COBS_ERR_TIMEOUT);
        alive = false;
        break;
      }
      phase_bits ^= 1u << st;
      __syncwarp();
      COBS_ACC(2);
        if (cur_b == 0) {
        if (u != cur_u) {
          cur_u = u;
          const int b_idx = u / p.Hkv, h = u - b_idx * p.Hkv;      // a division: once per unit, not per chunk
          // ---- query fragments of this unit ------------------------------------------------------------
          const __nv_bfloat16 *qg = p.q + ((size_t)b_idx * p.Hq + h * G) * D;
#pragma unroll
          for (int m = 0; m < KSM / 2; ++m) {
            uint4 v = make_uint4(0, 0, 0, 0);
            if (gid < G) v = *reinterpret_cast<const uint4 *>(qg + gid * D + (tig + 4 * m) * 8);
            bm[2 * m][0] = v.x; bm[2 * m][1] = v.y; bm[2 * m + 1][0] = v.z; bm[2 * m + 1][1] = v.w;
          }
          if (FP4) {
            // this thread's WPT * 8 query elements of head gid: the raw bf16 query (full space; the
            // 1/sqrt(D) factor is applied to the tile result) or the prepared fp32 q~ (subspace)
            float e[WPT][8];
            float mx = 0.f;
#pragma unroll
            for (int j = 0; j < WPT; ++j) {
              if (p.qtilde) {
                const float4 *src = reinterpret_cast<const float4 *>(
                    p.qtilde + ((size_t)b_idx * p.Hq + h * G + gid) * p.Ds_pad + tig * (WPT * 8) + j * 8);
                float4 lo = make_float4(0.f, 0.f, 0.f, 0.f), hi = lo;
                if (gid < G) { lo = __ldcg(src); hi = __ldcg(src + 1); }
                e[j][0] = lo.x; e[j][1] = lo.y; e[j][2] = lo.z; e[j][3] = lo.w;
                e[j][4] = hi.x; e[j][5] = hi.y; e[j][6] = hi.z; e[j][7] = hi.w;
              } else {
                uint4 v = make_uint4(0, 0, 0, 0);
                if (gid < G) v = *reinterpret_cast<const uint4 *>(qg + gid * D + tig * (WPT * 8) + j * 8);
                e[j][0] = bf16_lo(v.x); e[j][1] = bf16_hi(v.x); e[j][2] = bf16_lo(v.y); e[j][3] = bf16_hi(v.y);
                e[j][4] = bf16_lo(v.z); e[j][5] = bf16_hi(v.z); e[j][6] = bf16_lo(v.w); e[j][7] = bf16_hi(v.w);
              }
#pragma unroll
              for (int n = 0; n < 8; ++n) mx = fmaxf(mx, fabsf(e[j][n]));
            }
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            // mx in [2^(ex-1), 2^ex), from its exponent field (clamped: an all-zero or absurdly large query keeps
            // the powers of two below in range)
            const int ex = (int)(__float_as_uint(fminf(fmaxf(mx, 1e-30f), 1e30f)) >> 23) - 126;
            const float inv_s = __uint_as_float((uint32_t)(128 - ex) << 23);       // 2^(1-ex): brings max |q| into [1, 2)
            const float mult = __uint_as_float((uint32_t)(126 + ex) << 23) * (p.qtilde ? 1.0f : inv_sqrt_d);
#pragma unroll
            for (int j = 0; j < WPT; ++j) {
#pragma unroll
              for (int t = 0; t < NT; ++t) {
                float hi[8];
#pragma unroll
                for (int n = 0; n < 8; ++n) {
                  const float x = (t == 0) ? e[j][n] * inv_s : e[j][n];
                  hi[n] = __half2float(__float2half_rn(x));
                  e[j][n] = x - hi[n];
                }
                bq[t][2 * j][0] = f16x2(hi[0], hi[1]); bq[t][2 * j][1] = f16x2(hi[2], hi[3]);
                bq[t][2 * j + 1][0] = f16x2(hi[4], hi[5]); bq[t][2 * j + 1][1] = f16x2(hi[6], hi[7]);
              }
            }
            // result columns 2 tig, 2 tig + 1 are heads whose factor sits in the lanes gid = 2 tig, 2 tig + 1
            m0 = __shfl_sync(0xffffffffu, mult, (2 * tig) * 4);
            m1 = __shfl_sync(0xffffffffu, mult, (2 * tig + 1) * 4);
          }
        }
            // ---- first-order term: block means against the raw bf16 query ------------------------------------
        float c0 = 0.f, c1 = 0.f, c2 = 0.f, c3 = 0.f, e0 = 0.f, e1 = 0.f, e2 = 0.f, e3 = 0.f;   // two chains
        const uint32_t ma = sbase + (2 * gid) * mrow + tig * 16, mb = ma + mrow;
#pragma unroll
        for (int m = 0; m < MCH; ++m) {
          const uint4 va = lds128(ma + m * 64), vb = lds128(mb + m * 64);
          mma16816_bf16(c0, c1, c2, c3, va.x, vb.x, va.y, vb.y, bm[2 * m][0], bm[2 * m][1]);
          mma16816_bf16(e0, e1, e2, e3, va.z, vb.z, va.w, vb.w, bm[2 * m + 1][0], bm[2 * m + 1][1]);
        }
        fA0 = (c0 + e0) * inv_sqrt_d; fA1 = (c1 + e1) * inv_sqrt_d;
        fB0 = (c2 + e2) * inv_sqrt_d; fB1 = (c3 + e3) * inv_sqrt_d;
        sA0 = sA1 = sB0 = sB1 = 0.f;
      }
      // ---- curvature term: rows of this batch ----------------------------------------------------------
      const int row0 = (cur_b == 0) ? 0 : ROWS0 + (cur_b - 1) * ROWSN;
      const int rows = min(r - row0, (cur_b == 0) ? ROWS0 : ROWSN);
      const uint32_t xs = (cur_b == 0) ? XS0 : XSN;
      const uint32_t xa = sbase + ((cur_b == 0) ? mean_bytes : 0) + (2 * gid) * xs + tig * (FP4 ? WPT * 4 : 16), xb = xa + xs;
      bool rows_done = false;
      if constexpr (FP4 && WPT == 4 && NT == 1) {
        // the benchmark's descriptors (full key space, rank 4 or 8, the whole chunk in one stage): straight-line code
        if (single && (r == 8 || r == 4)) {
          const uint32_t spa = sbase + (kScoreStageBytes - scale_bytes) + (2 * gid) * r * scale_sz;
          if (r == 8) {
            if (scale_sz == 4) fp4_rows_full_width<8, true>(xa, xb, spa, bq[0], sA0, sA1, sB0, sB1);
            else fp4_rows_full_width<8, false>(xa, xb, spa, bq[0], sA0, sA1, sB0, sB1);
          } else {
            if (scale_sz == 4) fp4_rows_full_width<4, true>(xa, xb, spa, bq[0], sA0, sA1, sB0, sB1);
            else fp4_rows_full_width<4, false>(xa, xb, spa, bq[0], sA0, sA1, sB0, sB1);
          }
          rows_done = true;
        }
      }
      if (rows_done) {
      } else if (FP4) {
        // RG factor rows at a time: RG independent accumulator chains keep the tensor pipe busy
        constexpr int RG = kScoreRowGroup;
        const unsigned char *sp = wsm + st * kScoreStageBytes + (kScoreStageBytes - scale_bytes) + (2 * gid) * r * scale_sz;
#pragma unroll 1
        for (int i0 = 0; i0 < ROWS_MAX; i0 += RG) {
          if (i0 < rows) {
            float d[RG][4];
            uint32_t wa[RG][4], wb[RG][4];
#pragma unroll
            for (int k = 0; k < RG; ++k) {
              // neighbouring quads walk the group's rows in a rotated order (their rows then sit in different
              // bank halves); a row past the end of the batch is read from the last row and weighted by zero
              const int i = min(i0 + ((k + gid) & (RG - 1)), rows - 1);
              if (WPT == 4) {
                const uint4 a = lds128(xa + i * ROWB), bb = lds128(xb + i * ROWB);
                wa[k][0] = a.x; wa[k][1] = a.y; wa[k][2] = a.z; wa[k][3] = a.w;
                wb[k][0] = bb.x; wb[k][1] = bb.y; wb[k][2] = bb.z; wb[k][3] = bb.w;
              } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  wa[k][j] = (j < WPT) ? lds_u32(xa + i * ROWB + j * 4) : 0u;
                  wb[k][j] = (j < WPT) ? lds_u32(xb + i * ROWB + j * 4) : 0u;
                }
              }
              d[k][0] = d[k][1] = d[k][2] = d[k][3] = 0.f;
            }
#pragma unroll
            for (int j = 0; j < WPT; ++j) {
#pragma unroll
              for (int k = 0; k < RG; ++k) {
                uint32_t ha[4], hb[4];
                e2m1x8_to_f16(wa[k][j], ha);
                e2m1x8_to_f16(wb[k][j], hb);
#pragma unroll
                for (int t = 0; t < NT; ++t) {
                  mma16816_f16(d[k][0], d[k][1], d[k][2], d[k][3], ha[0], hb[0], ha[1], hb[1], bq[t][2 * j][0], bq[t][2 * j][1]);
                  mma16816_f16(d[k][0], d[k][1], d[k][2], d[k][3], ha[2], hb[2], ha[3], hb[3], bq[t][2 * j + 1][0],
                               bq[t][2 * j + 1][1]);
                }
              }
            }
            // scales of this lane's rows of the group (clamped like the rows themselves; a row past the end weighs
            // zero).  The per-head query factors m0, m1 are applied once per chunk, to the sums of squares.
            auto accumulate = [&](auto f32) {
#pragma unroll
              for (int k = 0; k < RG; ++k) {
                const int io = i0 + ((k + gid) & (RG - 1));
                const int ri = row0 + min(io, rows - 1);
                float sa, sb;
                if (decltype(f32)::value) {
                  sa = reinterpret_cast<const float *>(sp)[ri];
                  sb = reinterpret_cast<const float *>(sp)[r + ri];
                } else {
                  sa = __half2float(reinterpret_cast<const __half *>(sp)[ri]);
                  sb = __half2float(reinterpret_cast<const __half *>(sp)[r + ri]);
                }
                if (io >= rows) { sa = 0.f; sb = 0.f; }
                const float d0 = d[k][0] * sa, d1 = d[k][1] * sa, d2 = d[k][2] * sb, d3 = d[k][3] * sb;
                sA0 = fmaf(d0, d0, sA0); sA1 = fmaf(d1, d1, sA1); sB0 = fmaf(d2, d2, sB0); sB1 = fmaf(d3, d3, sB1);
              }
            };
            if (scale_sz == 4) accumulate(std::true_type{}); else accumulate(std::false_type{});
          }
        }
      } else {
#pragma unroll
        for (int i = 0; i < ROWS_MAX; ++i) {
          if (i < rows) {
            float d0 = 0.f, d1 = 0.f, d2 = 0.f, d3 = 0.f;
#pragma unroll
            for (int m = 0; m < MCH; ++m) {
              const uint4 va = lds128(xa + i * ROWB + m * 64), vb = lds128(xb + i * ROWB + m * 64);
              mma16816_bf16(d0, d1, d2, d3, va.x, vb.x, va.y, vb.y, bm[2 * m][0], bm[2 * m][1]);
              mma16816_bf16(d0, d1, d2, d3, va.z, vb.z, va.w, vb.w, bm[2 * m + 1][0], bm[2 * m + 1][1]);
            }
            d0 *= inv_sqrt_d; d1 *= inv_sqrt_d; d2 *= inv_sqrt_d; d3 *= inv_sqrt_d;
            sA0 = fmaf(d0, d0, sA0); sA1 = fmaf(d1, d1, sA1); sB0 = fmaf(d2, d2, sB0); sB1 = fmaf(d3, d3, sB1);
          }
        }
      }
    }

    COBS_ACC(3);
    // ---- end of a chunk: publish t = exp(e - chunk max) per block and the chunk's (max, sum of t) per head ----
    if (cur_b == n_batches - 1) {
      if (pend_u != u && pend_n > 0) {       // moving on to another unit: count the finished one's chunks
        __threadfence();
        __syncwarp();
        if (lane == 0) atomicAdd(CTL_UNIT(p.ctl_score) + pend_u, pend_n);
        pend_n = 0;
        COBS_ACC(7);
      }
      pend_u = u;
      if (ck * 16 < n_sum) {
        const int bA = ck * 16 + 2 * gid, bB = bA + 1, g0 = 2 * tig, g1 = g0 + 1;
        // 1/2 of the sums of squared projections; for FP4 the squares still lack the query's per-head factor
        const float h0 = FP4 ? 0.5f * m0 * m0 : 0.5f, h1 = FP4 ? 0.5f * m1 * m1 : 0.5f;
        const float eA0 = (bA < n_sum) ? ln_l + fA0 + h0 * sA0 : -INFINITY;
        const float eB0 = (bB < n_sum) ? ln_l + fB0 + h0 * sB0 : -INFINITY;
        const float eA1 = (bA < n_sum) ? ln_l + fA1 + h1 * sA1 : -INFINITY;
        const float eB1 = (bB < n_sum) ? ln_l + fB1 + h1 * sB1 : -INFINITY;
        // max over the chunk's 16 blocks (over gid), per head
        float mx0 = fmaxf(eA0, eB0), mx1 = fmaxf(eA1, eB1);
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {
          mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, o));
          mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, o));
        }
        const float tA0 = __expf(eA0 - mx0), tB0 = __expf(eB0 - mx0), tA1 = __expf(eA1 - mx1), tB1 = __expf(eB1 - mx1);
        float *e0 = p.e + ((size_t)u * G + g0) * NB, *e1 = p.e + ((size_t)u * G + g1) * NB;
        // blocks bA (even) and bA + 1 are neighbours in memory: one 8-byte store when both exist
        if (bB < n_sum) {
          if (g0 < G) __stcg(reinterpret_cast<float2 *>(e0 + bA), make_float2(tA0, tB0));
          if (g1 < G) __stcg(reinterpret_cast<float2 *>(e1 + bA), make_float2(tA1, tB1));
        } else if (bA < n_sum) {
          if (g0 < G) __stcg(e0 + bA, tA0);
          if (g1 < G) __stcg(e1 + bA, tA1);
        }
        float sm0 = tA0 + tB0, sm1 = tA1 + tB1;
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {
          sm0 += __shfl_xor_sync(0xffffffffu, sm0, o);
          sm1 += __shfl_xor_sync(0xffffffffu, sm1, o);
        }
        if (gid == 0) {
          if (g0 < G) __stcg(reinterpret_cast<float2 *>(p.lse_part) + ((size_t)u * G + g0) * cpu + ck, make_float2(mx0, sm0));
          if (g1 < G) __stcg(reinterpret_cast<float2 *>(p.lse_part) + ((size_t)u * G + g1) * cpu + ck, make_float2(mx1, sm1));
        }
      }
      ++pend_n;
    }
    __syncwarp();                           // all lanes are done with stage st before it is refilled
    COBS_ACC(4);
    cu = nu; cck = nck; cn = nn; cur_b = nxt_b; st ^= 1;
  }
  if (pend_n > 0) {
    __threadfence();
    __syncwarp();
    if (lane == 0) atomicAdd(CTL_UNIT(p.ctl_score) + pend_u, pend_n);
  }
  COBS_ACC(0);
  COBS_ACC_FLUSH(1200 + wg);
  return alive;
}

// ---------------------------------------------------------------------------------------------------
// phase A: attention over (unit, split) items + merge
// ---------------------------------------------------------------------------------------------------
template <int D>
__device__ void attend_phase(const Params &p, const int *seq_lens, unsigned char *wsm, int wg, int n_wg, int lane,
                             bool wait_select) {
  constexpr int CH = D / 8;                   // 16-byte chunks per row
  constexpr int KS = D / 16;
  constexpr int NTL = D / 8;                  // 8-wide output tiles
  constexpr int ROWB = D * 2;
  constexpr int VOFF = 16 * ROWB;             // V half of a stage
  constexpr int STAGE = 2 * VOFF;
  constexpr int NCP = (16 * CH) / 32;         // cp.async per lane per operand per stage
  const int gid = lane >> 2, tig = lane & 3;
  const int G = p.G, L = p.L, P = p.P, units = p.B * p.Hkv, n_splits = p.n_splits;
  const int lgL = 31 - __clz(L), lgP = 31 - __clz(P), lgg = lgL - 4;      // L and P are powers of two: shifts, not divisions
  const int gpb = L >> 4;
  const uint32_t ring = (uint32_t)__cvta_generic_to_shared(wsm);
  uint32_t *goff = reinterpret_cast<uint32_t *>(wsm + kAttStages * kAttStageBytes);
  int *gtok = reinterpret_cast<int *>(goff + kTableEntries);
  const float sl2 = (1.0f / sqrtf((float)D)) * 1.4426950408889634f;
  const uint4 *kbase = reinterpret_cast<const uint4 *>(p.k_pages) + lane;
  const uint4 *vbase = reinterpret_cast<const uint4 *>(p.v_pages) + lane;

  // lane-constant shared-memory offsets
  uint32_t cdst[NCP];                          // destination of this lane's j-th 16-byte copy (swizzled)
#pragma unroll
  for (int j = 0; j < NCP; ++j) {
    const int i = lane + 32 * j, t = i / CH, c = i - t * CH;
    cdst[j] = t * ROWB + ((c ^ (t & 7)) << 4);
  }
  // ldmatrix row addresses.  K (not transposed): matrices (tokens 0-7, chunk 2s), (0-7, 2s+1), (8-15, 2s), (8-15, 2s+1)
  const int kt = ((lane >> 4) & 1) * 8 + (lane & 7), kc = (lane >> 3) & 1;
  // V (transposed): matrices (tokens 0-7, chunk 2np), (8-15, 2np), (0-7, 2np+1), (8-15, 2np+1)
  const int vt = ((lane >> 3) & 1) * 8 + (lane & 7), vc = lane >> 4;

  // items are handed out in unit order from a global counter: a warp that arrives late simply takes fewer
  const int n_items = units * n_splits;
  const uint64_t pol = l2_evict_first_policy();
  COBS_ACC_DECL;

  // Closing an item = making its partial visible, counting it, and merging the unit if it was the last slice.
  // (Drawing the next item before this one is closed was measured and is slower: a warp that turns out to be the
  // last of its unit then holds an item back for the length of a merge.)
  auto close_item = [&](int u) {
    __threadfence();
    __syncwarp();
    int last = 0;
    if (lane == 0) last = (atomicAdd(CTL_UNIT(p.ctl_att) + u, 1) + 1 == n_splits);
    last = __shfl_sync(0xffffffffu, last, 0);
    COBS_ACC(5);
    if (!last) return;
    // ---- merge the unit's partials: o = sum_s e^{m_s - M} acc_s / sum_s e^{m_s - M} l_s -------------------
    // A slice is [G][D] accumulators followed by [G] (max, sum) pairs.  Few round trips: all pairs at once, then the
    // accumulators of four slices and up to four heads at a time; the weights sit in the (now idle) copy ring.
    __threadfence();
    const int b_idx = u / p.Hkv, h = u - b_idx * p.Hkv;
    const int SL = G * (D + 2), np = n_splits * G;
    const float *pu = p.partial + (size_t)u * n_splits * SL;
    float *sm_w = reinterpret_cast<float *>(wsm);            // [n_splits][G] maxima, then weights
    float *sm_l = sm_w + kMaxSplits * 8;        // [n_splits][G] sums
    float *sm_M = sm_l + kMaxSplits * 8;        // [8] maxima, [8] denominators, [8] their reciprocals
    for (int base = 0; base < np; base += 128) {
      float2 pv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int t = base + lane + 32 * i, sidx = t / G, g = t - sidx * G;
        pv[i] = (t < np) ? __ldcg(reinterpret_cast<const float2 *>(pu + (size_t)sidx * SL + G * D + 2 * g)) : make_float2(-INFINITY, 0.f);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int t = base + lane + 32 * i;
        if (t < np) { sm_w[t] = pv[i].x; sm_l[t] = pv[i].y; }
      }
    }
    __syncwarp();
    {
      const int g = lane & 7, sub = lane >> 3;
      float mx = -INFINITY;
      if (g < G) for (int sidx = sub; sidx < n_splits; sidx += 4) mx = fmaxf(mx, sm_w[sidx * G + g]);
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
      float dn = 0.f;
      if (g < G) for (int sidx = sub; sidx < n_splits; sidx += 4) {
        const float m = sm_w[sidx * G + g];
        const float w = (m == -INFINITY) ? 0.f : __expf(m - mx);
        dn = fmaf(w, sm_l[sidx * G + g], dn);
        sm_w[sidx * G + g] = w;
      }
      dn += __shfl_xor_sync(0xffffffffu, dn, 8);
      dn += __shfl_xor_sync(0xffffffffu, dn, 16);
      if (sub == 0 && g < G) { sm_M[g] = mx; sm_M[8 + g] = dn; sm_M[16 + g] = 1.0f / dn; }
    }
    __syncwarp();
    constexpr int KV = 4 * D / 64;                           // float2 per lane for four heads
    for (int gq = 0; gq < G; gq += 4) {
      const int nv2 = min(4, G - gq) * (D / 2);              // float2 in this group of heads
      float2 acc[KV];
#pragma unroll
      for (int k = 0; k < KV; ++k) acc[k] = make_float2(0.f, 0.f);
      for (int s0 = 0; s0 < n_splits; s0 += 4) {
        float2 x[4][KV];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float2 *ps = reinterpret_cast<const float2 *>(pu + (size_t)min(s0 + q, n_splits - 1) * SL + gq * D);
#pragma unroll
          for (int k = 0; k < KV; ++k) x[q][k] = (lane + 32 * k < nv2) ? __ldcg(ps + lane + 32 * k) : make_float2(0.f, 0.f);
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          if (s0 + q < n_splits) {
#pragma unroll
            for (int k = 0; k < KV; ++k) {
              const int idx = lane + 32 * k;
              const float w = (idx < nv2) ? sm_w[(s0 + q) * G + gq + idx / (D / 2)] : 0.f;
              acc[k].x = fmaf(w, x[q][k].x, acc[k].x);
              acc[k].y = fmaf(w, x[q][k].y, acc[k].y);
            }
          }
        }
      }
#pragma unroll
      for (int k = 0; k < KV; ++k) {
        const int idx = lane + 32 * k;
        if (idx < nv2) {
          const int head = gq + idx / (D / 2), col = (idx - (idx / (D / 2)) * (D / 2)) * 2;
          const float inv = sm_M[16 + head];            // one division per head; the rows are scaled by its result
          const size_t bh = (size_t)b_idx * p.Hq + h * G + head;
          *reinterpret_cast<float2 *>(p.out + bh * D + col) = make_float2(acc[k].x * inv, acc[k].y * inv);
        }
      }
      if (p.lse && lane < min(4, G - gq)) {
        const int head = gq + lane;
        p.lse[(size_t)b_idx * p.Hq + h * G + head] = sm_M[head] + __logf(sm_M[8 + head]);
      }
    }
    __syncwarp();
  };

  int item = 0;
  if (lane == 0) item = atomicAdd(CTL_MISC(p.ctl_item), 1);
  item = __shfl_sync(0xffffffffu, item, 0);
  for (;;) {
    COBS_ACC(0);
    if (item >= n_items) break;
    const int u = item / n_splits, split = item - u * n_splits;
    const int b_idx = u / p.Hkv, h = u - b_idx * p.Hkv;
    const int T = seq_lens[b_idx];
    const int ws = window_start(T, p.window, L);
    const int n_cand = ws >> lgL;
    const int n_win = (T - ws + L - 1) >> lgL;
    int n_sel = min(p.topk, n_cand);
    const int n_groups_u = (n_sel + n_win) * gpb;
    // slices of equal size to within one group (ceil-sized slices would leave the last slice of a unit nearly empty
    // and make every other one longer)
    const int g0 = (split * n_groups_u) / n_splits, g1 = ((split + 1) * n_groups_u) / n_splits;
    int n_groups = min(g1 - g0, kTableEntries);
    // ---- query fragments: rows = heads (zero padded to 16), natural k order.
    // Loaded first: the loads fly while the warp waits for the unit's selection and builds its group table.
    uint32_t qa[KS][2];
    {
      const uint32_t *qg = reinterpret_cast<const uint32_t *>(p.q + ((size_t)b_idx * p.Hq + h * G + gid) * D);
#pragma unroll
      for (int s = 0; s < KS; ++s) {
        qa[s][0] = (gid < G) ? qg[8 * s + tig] : 0u;
        qa[s][1] = (gid < G) ? qg[8 * s + 4 + tig] : 0u;
      }
    }
    bool ok = true;
    COBS_ACC(1);
    if (g0 < n_sel * gpb && n_groups > 0) {
      if (wait_select) {
        ok = wait_flag(CTL_UNIT(p.ctl_ready) + u);
        if (!ok && lane == 0) report(p.status, COBS_ERR_TIMEOUT);
        __threadfence();
      } else {
        n_sel = min(n_sel, min(__ldcg(p.sel_cnt + u), p.topk));
      }
    }
    COBS_ACC(2);
    // ---- table of this item's groups -----------------------------------------------------------------
    __syncwarp();
    for (int g = lane; g < n_groups; g += 32) {
      const int gg = g0 + g, it = gg >> lgg, sub = gg - (it << lgg);
      int blk;
      bool good = ok;
      if (it < min(p.topk, n_cand)) {          // a selected-block slot
        blk = (it < n_sel && ok) ? __ldcg(p.sel_idx + (size_t)u * p.topk + it) : -1;
        if (it < n_sel && ok && (blk < 0 || blk >= n_cand)) { good = false; report(p.status, COBS_ERR_BOUNDS); }
        if (blk < 0) good = false;
      } else {
        blk = n_cand + (it - min(p.topk, n_cand));
      }
      const int tok0 = blk * L + sub * 16;
      int first = -1;
      uint32_t off = 0;
      if (good && tok0 < T) {
        const int pslot = tok0 >> lgP;                                // a length beyond the page-table row is not followed
        const int pg = (pslot < p.mpp) ? p.page_table[(size_t)b_idx * p.mpp + pslot] : -1;
        if (pg < 0 || pg >= p.n_pages) report(p.status, COBS_ERR_BOUNDS);
        else { first = tok0; off = (uint32_t)(((((size_t)pg * p.Hkv + h) * P + (tok0 & (P - 1))) * D) / 8); }
      }
      goff[g] = off;
      gtok[g] = first;
    }
    __syncwarp();

    float o[NTL][2];
#pragma unroll
    for (int n = 0; n < NTL; ++n) o[n][0] = o[n][1] = 0.f;
    float m_run = -1e30f, l_run = 0.f, z2 = 0.f, z3 = 0.f;

    auto issue = [&](int g, int st) {
      if (g < n_groups) {
        const int first = gtok[g];
        if (first >= 0) {
          const uint32_t off = goff[g];
          const uint4 *ks = kbase + off, *vs = vbase + off;
          const uint32_t dst = ring + st * STAGE;
          const int nv = T - first;
          if (nv >= 16) {
#pragma unroll
            for (int j = 0; j < NCP; ++j) { cpa16(dst + cdst[j], ks + 32 * j, pol); cpa16(dst + VOFF + cdst[j], vs + 32 * j, pol); }
          } else {                             // ragged tail: rows past the end of the sequence are zero filled
#pragma unroll
            for (int j = 0; j < NCP; ++j) {
              const int bytes = ((lane + 32 * j) / CH < nv) ? 16 : 0;
              cpa16z(dst + cdst[j], ks + 32 * j, bytes, pol);
              cpa16z(dst + VOFF + cdst[j], vs + 32 * j, bytes, pol);
            }
          }
        }
      }
      cpa_commit();
    };

    COBS_ACC(3);
    issue(0, 0);
    issue(1, 1);
    int st = 0, st2 = 2;
    for (int g = 0; g < n_groups; ++g) {
      issue(g + 2, st2);
      cpa_wait<2>();
      __syncwarp();
      const int first = gtok[g];
      if (first >= 0) {
        const uint32_t sb = ring + st * STAGE;
        // ---- S^T = q K^T: s0 tokens 0-7, s1 tokens 8-15 --------------------------------------------------
        float s00 = 0.f, s01 = 0.f, s10 = 0.f, s11 = 0.f;
#pragma unroll
        for (int s = 0; s < KS; ++s) {
          uint32_t b0, b1, b2, b3;
          ldsm_x4(b0, b1, b2, b3, sb + kt * ROWB + (((2 * s + kc) ^ (kt & 7)) << 4));
          mma16816_bf16(s00, s01, z2, z3, qa[s][0], 0u, qa[s][1], 0u, b0, b1);
          mma16816_bf16(s10, s11, z2, z3, qa[s][0], 0u, qa[s][1], 0u, b2, b3);
        }
        const int nv = T - first;
        if (nv < 16) {                         // tokens past the end take no weight
          if (2 * tig >= nv) s00 = -1e30f;
          if (2 * tig + 1 >= nv) s01 = -1e30f;
          if (2 * tig + 8 >= nv) s10 = -1e30f;
          if (2 * tig + 9 >= nv) s11 = -1e30f;
        }
        float mx = fmaxf(fmaxf(s00, s01), fmaxf(s10, s11));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        if (__any_sync(0xffffffffu, mx > m_run)) {       // rescale only when some head's running max moved
          const float m_new = fmaxf(m_run, mx);
          const float corr = ex2((m_run - m_new) * sl2);
          m_run = m_new;
          l_run *= corr;
#pragma unroll
          for (int n = 0; n < NTL; ++n) { o[n][0] *= corr; o[n][1] *= corr; }
        }
        const float mb = m_run * sl2;
        const float p0 = ex2(fmaf(s00, sl2, -mb)), p1 = ex2(fmaf(s01, sl2, -mb));
        const float p2 = ex2(fmaf(s10, sl2, -mb)), p3 = ex2(fmaf(s11, sl2, -mb));
        l_run += (p0 + p1) + (p2 + p3);
        const uint32_t a0h = bf16x2(p0, p1), a2h = bf16x2(p2, p3);
        const uint32_t a0l = bf16x2(p0 - bf16_lo(a0h), p1 - bf16_hi(a0h));
        const uint32_t a2l = bf16x2(p2 - bf16_lo(a2h), p3 - bf16_hi(a2h));
        // ---- O += P V ---------------------------------------------------------------------------------------
#pragma unroll
        for (int np = 0; np < NTL / 2; ++np) {
          uint32_t b0, b1, b2, b3;
          ldsm_x4_t(b0, b1, b2, b3, sb + VOFF + vt * ROWB + (((2 * np + vc) ^ (vt & 7)) << 4));
          mma16816_bf16(o[2 * np][0], o[2 * np][1], z2, z3, a0h, 0u, a2h, 0u, b0, b1);
          mma16816_bf16(o[2 * np + 1][0], o[2 * np + 1][1], z2, z3, a0h, 0u, a2h, 0u, b2, b3);
          mma16816_bf16(o[2 * np][0], o[2 * np][1], z2, z3, a0l, 0u, a2l, 0u, b0, b1);
          mma16816_bf16(o[2 * np + 1][0], o[2 * np + 1][1], z2, z3, a0l, 0u, a2l, 0u, b2, b3);
        }
      }
      __syncwarp();                            // all lanes are done with the stage before it is refilled
      st = (st == kAttStages - 1) ? 0 : st + 1;
      st2 = (st2 == kAttStages - 1) ? 0 : st2 + 1;
    }
    cpa_wait<0>();
    COBS_ACC(4);

    // ---- this warp's partial: [G][D] acc, then [G] (running max in natural log units, running sum) ---------
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    float *part = p.partial + ((size_t)u * n_splits + split) * G * (D + 2);
    if (gid < G) {
      float *dst = part + gid * D;
#pragma unroll
      for (int n = 0; n < NTL; ++n) __stcg(reinterpret_cast<float2 *>(dst + 8 * n + 2 * tig), make_float2(o[n][0], o[n][1]));
      if (tig == 0)
        __stcg(reinterpret_cast<float2 *>(part + G * D + 2 * gid),
               make_float2((l_run > 0.f) ? m_run * (sl2 * 0.6931471805599453f) : -INFINITY, l_run));
    }
    close_item(u);
    COBS_ACC(7);
    int next_item = 0;
    if (lane == 0) next_item = atomicAdd(CTL_MISC(p.ctl_item), 1);
    item = __shfl_sync(0xffffffffu, next_item, 0);
    COBS_ACC(6);
  }
  COBS_ACC_FLUSH(wg);
}

// ---------------------------------------------------------------------------------------------------
// phase S on the 5th-generation tensor cores (tcgen05), for the main configuration: packed E2M1 factors in
// the full key space, D = 128, r = 8.
//
// A 16-block chunk is ONE matrix product: the chunk's 16 x 8 = 128 factor rows (M = 128, K = 128) against the G
// query heads.  The factor rows are fetched by a tiled TMA copy whose element type makes the copy engine unpack
// the 4-bit codes into the 8-bit containers `tcgen05.mma.kind::f8f6f4` reads (128-byte swizzled rows in shared
// memory), so no thread ever touches a code.  The query cannot be FP4: it enters as TWO E4M3 terms per head
// (high part + remainder of the bf16 query scaled by a power of two: together exact for every element within
// 2^-10 of the head's largest), columns h and 8 + h of a 16-column operand.  The accumulator (128 lanes x 16
// fp32 columns) lives in tensor memory, four buffers deep.
//
// Roles inside the CTA (one CTA per SM): warp 12 = producer (TMA / bulk copies of factor rows, means, scales; builds
// the query operand when the unit changes), warp 13 = MMA issuer (one thread), warps 0-3 and 4-7 = two epilogue
// sets taking alternate chunks (warp w reads the TMEM lanes 32 (w mod 4) ..., i.e. blocks 4 (w mod 4) ... of the
// chunk), warps 8-11 = the selection team as before.  All hand-offs are mbarriers with bounded waits.
// ---------------------------------------------------------------------------------------------------
constexpr int kUBlocks = 32;                                  // blocks per pipeline stage: two 128-row products
constexpr int kUStages = 4;                                   // stages per CTA (two groups of kUAccBufs)
constexpr int kUStageBytes = 43008;                           // 32768 unpacked factor rows + 8192 means + 1024 scales + header, padded to 1 KiB
constexpr int kUMeanOff = 32768, kUScaleOff = 40960, kUHdrOff = 41984;
constexpr int kUTiles = 10;                                   // query operands (one per unit the CTA meets)
constexpr int kUTileBytes = 2048;
constexpr int kUTilesOff = kUStages * kUStageBytes;           // 172032
constexpr int kUFacOff = kUTilesOff + kUTiles * kUTileBytes;  // [tile][8] head factors
constexpr int kUSmemBytes = kFusedSmemBytes + 1024;           // + slack to align the base to 1 KiB
static_assert(kUFacOff + kUTiles * 32 <= kFusedSmemBytes, "tcgen05 scoring layout exceeds the CTA's shared memory");
constexpr int kUThreads = (kFWarps + kSelWarps + 2) * 32;     // + producer warp + MMA warp
constexpr int kUAccCols = 32, kUAccBufs = 2;                  // tensor memory: 2 buffers x (2 products x 16 columns)
constexpr int kUWaitLimit = 200000;                           // bounded mbarrier waits (try_wait iterations)
constexpr int kUMaxWaves = 8;
static_assert(kWaves <= kUMaxWaves, "wave table too small");
static_assert(kUStages == 2 * kUAccBufs, "a producer step and an issuer step cover the same kUAccBufs list positions");
// mbarrier indices
constexpr int kBFull = 0, kBEmpty = kBFull + kUStages, kBTFull = kBEmpty + kUStages, kBTEmpty = kBTFull + kUAccBufs,
              kBTiles = kBTEmpty + kUAccBufs, kBCount = kBTiles + 1;

// The CTA's stage list: wave by wave, a contiguous range of each wave's 32-block pieces.  Position n of the list
// goes through pipeline slot n mod kUStages and accumulator n mod kUAccBufs whether or not it holds summarised
// blocks (an empty position passes as a bubble), so every role can address the list at random.  The units the
// ranges touch are numbered in list order: that number is the unit's query-operand tile.
struct UmmaList {
  int n_waves, total, cpu, n_tiles;
  int len[kUMaxWaves], start[kUMaxWaves], tile0[kUMaxWaves];
};
__host__ __device__ inline void umma_list_make(UmmaList &l, int units, int NB, int grid, int bid) {
  l.cpu = NB / kUBlocks;
  l.n_waves = (units >= 2 * kWaves) ? kWaves : 1;
  l.total = 0;
  l.n_tiles = 0;
  for (int w = 0; w < l.n_waves; ++w) {
    const int u0 = (units * w) / l.n_waves, u1 = (units * (w + 1)) / l.n_waves;
    const int tot = (u1 - u0) * l.cpu, per = (tot + grid - 1) / grid;
    const int c = (bid * per < tot) ? bid * per : tot, c_end = (bid * per + per < tot) ? bid * per + per : tot;
    l.start[w] = u0 * l.cpu + c;
    l.len[w] = c_end - c;
    l.total += c_end - c;
    l.tile0[w] = l.n_tiles;
    if (c_end > c) l.n_tiles += (l.start[w] + l.len[w] - 1) / l.cpu - l.start[w] / l.cpu + 1;
  }
}

__device__ __forceinline__ bool mbar_wait_lim(uint32_t bar, uint32_t parity) {
  for (int it = 0; it < kUWaitLimit; ++it) {
    uint32_t done;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    if (done) return true;
  }
  return false;
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
// K-major operand, 128-byte swizzled rows, 8-row groups 1024 bytes apart (shared-memory matrix descriptor)
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (uint64_t(1) << 16) | (uint64_t(1024 >> 4) << 32) | (uint64_t(1) << 46) |
         (uint64_t(2) << 61);
}
// D fp32, A = E2M1, B = E4M3, both K-major, M = 128, N = 16
constexpr uint32_t kUInstrDesc = (1u << 4) | (5u << 7) | (0u << 10) | ((16u >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ void umma_abort(const Params &p, volatile int *abort_flag, int lane) {
  if (lane == 0) { report(p.status, COBS_ERR_TIMEOUT); *abort_flag = 1; }
}

// Query operand of one unit, built by one warp: rows h (high E4M3 term) and 8 + h (remainder) of a 16 x 128
// operand, 128-byte swizzled, plus the head factors (power of two that was divided out, times 1/sqrt(D)).
__device__ void umma_build_tile(const Params &p, unsigned char *fsm, int t, int u, int lane) {
  unsigned char *tile = fsm + kUTilesOff + t * kUTileBytes;
#pragma unroll
  for (int j = 0; j < 4; ++j) reinterpret_cast<uint4 *>(tile)[lane * 4 + j] = make_uint4(0, 0, 0, 0);
  __syncwarp();
  const int G = p.G, b_idx = u / p.Hkv, h = u - b_idx * p.Hkv;
  const float inv_sqrt_d = 1.0f / sqrtf(128.0f);
  uint2 raws[8];                                            // all heads' loads in flight together
#pragma unroll
  for (int g = 0; g < 8; ++g)
    raws[g] = (g < G) ? *reinterpret_cast<const uint2 *>(p.q + ((size_t)b_idx * p.Hq + h * G + g) * 128 + 4 * lane) : make_uint2(0, 0);
#pragma unroll
  for (int g = 0; g < 8; ++g) {
    if (g >= G) break;
    const uint2 raw = raws[g];
    const float x0 = bf16_lo(raw.x), x1 = bf16_hi(raw.x), x2 = bf16_lo(raw.y), x3 = bf16_hi(raw.y);
    const float mx = warp_max(fmaxf(fmaxf(fabsf(x0), fabsf(x1)), fmaxf(fabsf(x2), fabsf(x3))));
    int ex = 0;
    if (mx > 0.f) frexpf(mx, &ex);
    const float sc = ldexpf(1.0f, 8 - ex);                   // largest |q| of the head lands in [128, 256)
    const float y0 = x0 * sc, y1 = x1 * sc, y2 = x2 * sc, y3 = x3 * sc;
    const __nv_fp8x2_storage_t h01 = __nv_cvt_float2_to_fp8x2(make_float2(y0, y1), __NV_SATFINITE, __NV_E4M3);
    const __nv_fp8x2_storage_t h23 = __nv_cvt_float2_to_fp8x2(make_float2(y2, y3), __NV_SATFINITE, __NV_E4M3);
    const __half2_raw b01 = __nv_cvt_fp8x2_to_halfraw2(h01, __NV_E4M3), b23 = __nv_cvt_fp8x2_to_halfraw2(h23, __NV_E4M3);
    const float2 f01 = __half22float2(*reinterpret_cast<const __half2 *>(&b01));
    const float2 f23 = __half22float2(*reinterpret_cast<const __half2 *>(&b23));
    const __nv_fp8x2_storage_t l01 = __nv_cvt_float2_to_fp8x2(make_float2(y0 - f01.x, y1 - f01.y), __NV_SATFINITE, __NV_E4M3);
    const __nv_fp8x2_storage_t l23 = __nv_cvt_float2_to_fp8x2(make_float2(y2 - f23.x, y3 - f23.y), __NV_SATFINITE, __NV_E4M3);
    const uint32_t hi4 = (uint32_t)h01 | ((uint32_t)h23 << 16), lo4 = (uint32_t)l01 | ((uint32_t)l23 << 16);
    const int kb = 4 * lane;                                // byte (= element) position in the row
    const int nh = g, nl = 8 + g;
    *reinterpret_cast<uint32_t *>(tile + (nh >> 3) * 1024 + (nh & 7) * 128 + (((kb >> 4) ^ (nh & 7)) << 4) + (kb & 15)) = hi4;
    *reinterpret_cast<uint32_t *>(tile + (nl >> 3) * 1024 + (nl & 7) * 128 + (((kb >> 4) ^ (nl & 7)) << 4) + (kb & 15)) = lo4;
    if (lane == 0) reinterpret_cast<float *>(fsm + kUFacOff)[t * 8 + g] = ldexpf(1.0f, ex - 8) * inv_sqrt_d;
  }
}

// All query operands of the CTA's list, built by the selection team's warps before they have anything to select.
__device__ void umma_build_tiles(const Params &p, const UmmaList &l, unsigned char *fsm, uint32_t bars, int team_warp, int lane) {
  for (int w = 0; w < l.n_waves; ++w) {
    if (l.len[w] <= 0) continue;
    const int uf = l.start[w] / l.cpu, ul = (l.start[w] + l.len[w] - 1) / l.cpu;
    for (int u = uf + team_warp; u <= ul; u += kSelWarps) umma_build_tile(p, fsm, l.tile0[w] + (u - uf), u, lane);
  }
  fence_proxy_async();
  __syncwarp();
  if (lane == 0) mbar_arrive(bars + kBTiles * 8);
}

// Producer warp.  Step k of the warp issues the list positions kUAccBufs k ... together: lane a does the
// arithmetic of position kUAccBufs k + a and writes the slot's 16-byte header {unit, 32-block piece, summarised
// blocks, flags | tile} for the other roles; lane 0 then issues the copies (their operands are warp-uniform):
// 256 factor rows (tensor copy, unpacked by the copy engine), 32 means, 32 x 8 scales.
__device__ void umma_producer(const Params &p, const int *seq_lens, const UmmaList &l, unsigned char *fsm, uint32_t bars,
                              const CUtensorMap *tmap, int lane, volatile int *abort_flag) {
  const int NB = p.NB, cpu = l.cpu;
  const int scale_sz = (p.scale_dtype == COBS_SCALE_FP16) ? 2 : 4;
  const uint32_t scale_bytes = kUBlocks * 8 * scale_sz;
  const uint32_t sm = (uint32_t)__cvta_generic_to_shared(fsm);
  int w = 0, o = lane;
  COBS_ACC_DECL;
  for (int k = 0;; ++k) {
    while (w < l.n_waves && o >= l.len[w]) { o -= l.len[w]; ++w; }
    const int slot = (lane & (kUAccBufs - 1)) + kUAccBufs * (k & 1);
    const bool has = lane < kUAccBufs && w < l.n_waves;
    if (!__any_sync(0xffffffffu, has) || *abort_flag) break;
    int u = 0, ck = 0, n_sum = 0, tile = 0;
    bool valid = false;
    if (has) {
      const int c = l.start[w] + o;
      u = c / cpu; ck = c - u * cpu;
      n_sum = min(seq_lens[u / p.Hkv] / p.L, NB);
      valid = ck * kUBlocks < n_sum;
      tile = l.tile0[w] + (u - l.start[w] / cpu);
    }
    COBS_ACC(0);
    bool ok = true;
    if (has && k > 1) ok = mbar_wait_lim(bars + (kBEmpty + slot) * 8, ((k >> 1) - 1) & 1);
    if (!__all_sync(0xffffffffu, ok)) { umma_abort(p, abort_flag, lane); break; }
    COBS_ACC(1);
    if (has) *reinterpret_cast<int4 *>(fsm + slot * kUStageBytes + kUHdrOff) = make_int4(u, ck, n_sum, (valid ? 1 : 0) | (tile << 8));
    __syncwarp();
    const unsigned hm = __ballot_sync(0xffffffffu, has), vm = __ballot_sync(0xffffffffu, valid);
    const uint32_t rec0 = (uint32_t)(u * NB + ck * kUBlocks);    // < 2^28 (checked on the host)
    COBS_ACC(2);
#pragma unroll
    for (int sl = 0; sl < kUAccBufs; ++sl) {
      const uint32_t rec = __shfl_sync(0xffffffffu, rec0, sl);
      if (lane == 0 && ((hm >> sl) & 1u)) {
        const int slot_s = sl + kUAccBufs * (k & 1);
        const uint32_t st = sm + slot_s * kUStageBytes, bar = bars + (kBFull + slot_s) * 8;
        if ((vm >> sl) & 1u) {
          mbar_expect_tx(bar, (uint32_t)(kUBlocks * 8 * 64) + (uint32_t)(kUBlocks * 256) + scale_bytes);
          asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n"
                       ::"r"(st), "l"(tmap), "r"(0), "r"((int)(rec * 8u)), "r"(bar) : "memory");
          bulk_g2s(st + kUMeanOff, (const char *)p.mean + (size_t)rec * 256, (uint32_t)(kUBlocks * 256), bar);
          bulk_g2s(st + kUScaleOff, (const char *)p.scale + (size_t)rec * (8 * scale_sz), scale_bytes, bar);
        } else {
          mbar_arrive(bar);                       // a bubble: nothing to copy
        }
      }
    }
    COBS_ACC(3);
    o += kUAccBufs;
  }
  COBS_ACC_FLUSH((int)blockIdx.x);
}

// MMA issuer warp.  Lane a < kUAccBufs waits for and decodes the list positions a, a + kUAccBufs, ... (accumulator
// buffer a); lane 0 issues: two 128 x 16 x 128 products (four K steps each) per stage, then one commit that hands
// the accumulators to the epilogue.  A bubble passes its barrier on by hand.
__device__ void umma_issuer(const Params &p, const UmmaList &l, unsigned char *fsm, uint32_t bars, uint32_t tmem, int lane,
                            volatile int *abort_flag) {
  const uint64_t desc0 = umma_desc((uint32_t)__cvta_generic_to_shared(fsm));   // the whole region lies below 2^18
  int n = lane;
  COBS_ACC_DECL;
  if (!mbar_wait_lim(bars + kBTiles * 8, 0)) { umma_abort(p, abort_flag, lane); return; }
  for (int k = 0;; ++k) {
    const int slot = (lane & (kUAccBufs - 1)) + kUAccBufs * (k & 1), fpar = (k >> 1) & 1;
    const bool has = lane < kUAccBufs && n < l.total;
    if (!__any_sync(0xffffffffu, has) || *abort_flag) break;
    bool ok = true;
    int4 hdr = make_int4(0, 0, 0, 0);
    COBS_ACC(0);
    if (has) {
      ok = mbar_wait_lim(bars + (kBFull + slot) * 8, fpar);
      hdr = *reinterpret_cast<const int4 *>(fsm + slot * kUStageBytes + kUHdrOff);
    }
    COBS_ACC(1);
    const bool valid = has && (hdr.w & 1);
    const int tile = (hdr.w >> 8) & 0xff;
    if (has && ok && k > 0) ok = mbar_wait_lim(bars + (kBTEmpty + lane) * 8, (k - 1) & 1);
    COBS_ACC(2);
    if (!__all_sync(0xffffffffu, ok)) { umma_abort(p, abort_flag, lane); break; }
    tc_fence_after();
    const unsigned hm = __ballot_sync(0xffffffffu, has), vm = __ballot_sync(0xffffffffu, valid);
#pragma unroll
    for (int a = 0; a < kUAccBufs; ++a) {
      const int tile_a = __shfl_sync(0xffffffffu, tile, a);
      if (lane == 0 && ((hm >> a) & 1u)) {
        const int slot_a = a + kUAccBufs * (k & 1);
        const uint32_t bar_t = bars + (kBTFull + a) * 8;
        if ((vm >> a) & 1u) {
          const uint64_t db0 = desc0 + (uint64_t)((kUTilesOff + tile_a * kUTileBytes) >> 4);
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const uint64_t da0 = desc0 + (uint64_t)((slot_a * kUStageBytes + half * 16384) >> 4);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              const uint64_t da = da0 + 2 * ks, db = db0 + 2 * ks;   // 32 bytes along K per step
              const uint32_t accum = ks > 0;
              asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n}\n"
                           ::"r"(tmem + a * kUAccCols + half * 16), "l"(da), "l"(db), "r"(kUInstrDesc), "r"(accum) : "memory");
            }
          }
          tc_commit(bar_t);
        } else {
          mbar_arrive(bar_t);
        }
      }
    }
    COBS_ACC(3);
    n += kUAccBufs;
  }
  COBS_ACC_FLUSH(200 + (int)blockIdx.x);
}

// Epilogue warp (streaming warps 0-7; set = warp / 4 takes the list positions of its parity, warp mod 4 = TMEM lane
// quarter): lane (bl, i) = (lane / 8, lane % 8) holds, for each half of the stage, accumulator row (block
// 16 half + 4 q + bl, factor i).  Leaves per block t = exp(e - max over the warp's four blocks of a half) and that
// (max, sum) pair, i.e. four pairs per 16-block chunk and head; each warp counts a 16-block chunk on the unit
// once, so a unit is complete at 4 x its chunks.
__device__ void umma_epilogue(const Params &p, const UmmaList &l, unsigned char *fsm, uint32_t bars, uint32_t tmem, int warp,
                              int lane, volatile int *abort_flag) {
  const int set = warp >> 2, q = warp & 3;
  const int gid = lane >> 2, tig = lane & 3;      // mma.sync fragment coordinates (mean term)
  const int bl = lane >> 3, i = lane & 7;
  const int G = p.G, NB = p.NB, cpu16 = NB / 16;
  const bool scale_f16 = p.scale_dtype == COBS_SCALE_FP16;
  const float inv_sqrt_d = 1.0f / sqrtf(128.0f), ln_l = logf((float)p.L);
  int my_u = -1, pend_u = -1, pend_n = 0;
  uint32_t bm[8][2];
  float fac2 = 0.f;
#pragma unroll
  for (int m = 0; m < 8; ++m) bm[m][0] = bm[m][1] = 0u;
  auto flush = [&]() {
    if (pend_n > 0) {
      __threadfence();
      __syncwarp();
      if (lane == 0) atomicAdd(CTL_UNIT(p.ctl_score) + pend_u, pend_n);
      pend_n = 0;
    }
  };
  COBS_ACC_DECL;
  if (!mbar_wait_lim(bars + kBTiles * 8, 0)) { umma_abort(p, abort_flag, lane); return; }
  for (int n = set, j = 0; n < l.total; n += 2, ++j) {
    if (*abort_flag) break;
    const int slot = n & (kUStages - 1), fpar = (n / kUStages) & 1, tfpar = j & 1;
    const uint32_t bar_empty = bars + (kBEmpty + slot) * 8, bar_tfull = bars + (kBTFull + set) * 8, bar_tempty = bars + (kBTEmpty + set) * 8;
    COBS_ACC(0);
    if (!mbar_wait_lim(bars + (kBFull + slot) * 8, fpar)) { umma_abort(p, abort_flag, lane); break; }
    COBS_ACC(1);
    const unsigned char *stg = fsm + slot * kUStageBytes;
    const int4 hdr = *reinterpret_cast<const int4 *>(stg + kUHdrOff);
    const int u = hdr.x, ck = hdr.y, n_sum = hdr.z;
    if (!(hdr.w & 1)) {                          // a bubble: pass the barriers on
      if (!mbar_wait_lim(bar_tfull, tfpar)) { umma_abort(p, abort_flag, lane); break; }
      __syncwarp();
      if (lane == 0) { mbar_arrive(bar_empty); mbar_arrive(bar_tempty); }
      continue;
    }
    if (u != my_u) {
      // ---- a new unit: query fragments for the mean product (column = head gid; k order as the rows are read) ----
      my_u = u;
      const int tile = (hdr.w >> 8) & 0xff;
      const int b_idx = u / p.Hkv, h = u - b_idx * p.Hkv;
      const __nv_bfloat16 *qg = p.q + ((size_t)b_idx * p.Hq + h * G) * 128;
#pragma unroll
      for (int m = 0; m < 4; ++m) {
        uint4 v = make_uint4(0, 0, 0, 0);
        if (gid < G) v = *reinterpret_cast<const uint4 *>(qg + gid * 128 + (tig + 4 * m) * 8);
        bm[2 * m][0] = v.x; bm[2 * m][1] = v.y; bm[2 * m + 1][0] = v.z; bm[2 * m + 1][1] = v.w;
      }
      const float fac = (i < G) ? reinterpret_cast<const float *>(fsm + kUFacOff)[tile * 8 + i] : 0.f;
      fac2 = fac * fac;
    }
    COBS_ACC(2);
    // ---- first-order term: rows 0-3 of an m16n8k16 tile = blocks 4 q .. of half 0, rows 8-11 = those of half 1 -----
    float c0 = 0.f, c1 = 0.f, c2 = 0.f, c3 = 0.f, e0 = 0.f, e1 = 0.f, e2 = 0.f, e3 = 0.f;
    {
      const uint32_t ma = (uint32_t)__cvta_generic_to_shared(stg + kUMeanOff) + (4 * q + (gid & 3)) * 256 + tig * 16;
#pragma unroll
      for (int m = 0; m < 4; ++m) {
        uint4 va = lds128(ma + m * 64), vb = lds128(ma + 16 * 256 + m * 64);
        if (gid >= 4) { va = make_uint4(0, 0, 0, 0); vb = va; }
        mma16816_bf16(c0, c1, c2, c3, va.x, vb.x, va.y, vb.y, bm[2 * m][0], bm[2 * m][1]);
        mma16816_bf16(e0, e1, e2, e3, va.z, vb.z, va.w, vb.w, bm[2 * m + 1][0], bm[2 * m + 1][1]);
      }
    }
    // lane (gid < 4, tig): block 4 q + gid of each half, heads 2 tig and 2 tig + 1
    const float fm[2][2] = {{(c0 + e0) * inv_sqrt_d, (c1 + e1) * inv_sqrt_d}, {(c2 + e2) * inv_sqrt_d, (c3 + e3) * inv_sqrt_d}};
    float sc[2];
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      const int srow = (16 * hf + 4 * q + bl) * 8 + i;
      sc[hf] = scale_f16 ? __half2float(reinterpret_cast<const __half *>(stg + kUScaleOff)[srow])
                         : reinterpret_cast<const float *>(stg + kUScaleOff)[srow];
    }
    COBS_ACC(3);
    // ---- the stage's products from tensor memory ----------------------------------------------------------------
    if (!mbar_wait_lim(bar_tfull, tfpar)) { umma_abort(p, abort_flag, lane); break; }
    COBS_ACC(4);
    tc_fence_after();
    uint32_t r[32];
    {
      const uint32_t taddr = tmem + ((uint32_t)(32 * q) << 16) + set * kUAccCols;
      asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                   "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
                   : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                     "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                     "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                     "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                   : "r"(taddr));
      asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncwarp();
    if (lane == 0) { mbar_arrive(bar_empty); mbar_arrive(bar_tempty); }   // stage and accumulator may be refilled
    float ssum[2];
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      float v[8];
#pragma unroll
      for (int h = 0; h < 8; ++h) {
        const float x = (__uint_as_float(r[16 * hf + h]) + __uint_as_float(r[16 * hf + 8 + h])) * sc[hf];
        v[h] = x * x;
      }
      // sum over the 8 factors of a block, transposing as it goes: lane i ends with head i
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float keep = (i & 4) ? v[k + 4] : v[k], send = (i & 4) ? v[k] : v[k + 4];
        v[k] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
      }
#pragma unroll
      for (int k = 0; k < 2; ++k) {
        const float keep = (i & 2) ? v[k + 2] : v[k], send = (i & 2) ? v[k] : v[k + 2];
        v[k] = keep + __shfl_xor_sync(0xffffffffu, send, 2);
      }
      const float keep = (i & 1) ? v[1] : v[0], send = (i & 1) ? v[0] : v[1];
      ssum[hf] = keep + __shfl_xor_sync(0xffffffffu, send, 1);
    }
    const int src = bl * 4 + (i >> 1);
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      const float fa = __shfl_sync(0xffffffffu, fm[hf][0], src), fb = __shfl_sync(0xffffffffu, fm[hf][1], src);
      const int blk = ck * kUBlocks + 16 * hf + 4 * q + bl;
      const bool live = (i < G) && (blk < n_sum);
      const float e = live ? ln_l + ((i & 1) ? fb : fa) + 0.5f * fac2 * ssum[hf] : -INFINITY;
      // max and sum per head over the warp's four blocks: one pair per quarter of a 16-block chunk
      float wm = fmaxf(e, __shfl_xor_sync(0xffffffffu, e, 8));
      wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, 16));
      const float t = live ? __expf(e - wm) : 0.f;
      float ws = t + __shfl_xor_sync(0xffffffffu, t, 8);
      ws += __shfl_xor_sync(0xffffffffu, ws, 16);
      if (live) __stcg(p.e + ((size_t)u * G + i) * NB + blk, t);
      if (bl == 0 && i < G && (2 * ck + hf) * 16 < n_sum)
        __stcg(reinterpret_cast<float2 *>(p.lse_part) + (((size_t)u * G + i) * cpu16 + 2 * ck + hf) * 4 + q, make_float2(wm, ws));
    }
    COBS_ACC(5);
    if (pend_u != u) flush();
    pend_u = u;
    pend_n += 1 + (((2 * ck + 1) * 16 < n_sum) ? 1 : 0);
    COBS_ACC(6);
  }
  flush();
  COBS_ACC_FLUSH(400 + (int)blockIdx.x * 8 + warp);
}

// ---------------------------------------------------------------------------------------------------
// Prologue of the subspace descriptor: q~ = U_Q^T (q / sqrt(D)) for every query head, zero padded to Ds_pad - the
// one O(s D) projection per step and head that the scoring then shares across all blocks (Method, "Per-step
// scoring").  Teams of four warps take (head, 32 consecutive subspace coordinates) tasks: lane = coordinate, so the
// reads of U_Q [Hkv][D][Ds] are coalesced; each warp sums a quarter of the head dimension (all its loads in flight at
// once) and the quarters are added in a fixed order.  The result goes to the workspace; a grid barrier (the launch
// is cooperative, so every CTA is resident) makes it visible before any warp scores.
// ---------------------------------------------------------------------------------------------------
__device__ void project_queries(const Params &p) {
  __shared__ float s_part[16][32];                // partial sums of the CTA's warps (at most 16 warps)
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int teams = (int)(blockDim.x >> 5) / 4;   // four warps share a task: each sums a quarter of the head dimension
  const int team = warp >> 2, quarter = warp & 3;
  const int nsb = p.Ds_pad / 32, n_tasks = p.B * p.Hq * nsb;
  const int dq = p.D / 4;                         // 32 or 16 coordinates per quarter: all their loads fly together
  const float inv_sqrt_d = 1.0f / sqrtf((float)p.D);
  for (int base = blockIdx.x * teams; base < n_tasks; base += gridDim.x * teams) {
    const int t = base + team;
    const bool active = team < teams && t < n_tasks;
    float v = 0.f;
    int bh = 0, sidx = 0;
    if (active) {
      bh = t / nsb;
      const int sb = t - bh * nsb, hq = bh % p.Hq, h = hq / p.G;
      sidx = sb * 32 + lane;
      const float qv = (lane < dq) ? __bfloat162float(p.q[(size_t)bh * p.D + quarter * dq + lane]) * inv_sqrt_d : 0.f;
      const bool live = sidx < p.Ds;              // padding coordinates take part in the shuffles and end as 0
      const float *uq = p.u_q + ((size_t)h * p.D + quarter * dq) * p.Ds + (live ? sidx : 0);
      float x[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) x[j] = (live && j < dq) ? __ldg(uq + (size_t)j * p.Ds) : 0.f;
#pragma unroll
      for (int j = 0; j < 32; ++j) v = fmaf(x[j], __shfl_sync(0xffffffffu, qv, j), v);
    }
    if (warp < 16) s_part[warp][lane] = v;
    __syncthreads();
    if (active && quarter == 0)                   // fixed order: the same bits every time
      __stcg(p.qtilde_out + (size_t)bh * p.Ds_pad + sidx,
             ((s_part[warp][lane] + s_part[warp + 1][lane]) + s_part[warp + 2][lane]) + s_part[warp + 3][lane]);
    __syncthreads();
  }
}

// Every CTA of the (cooperatively launched, hence fully resident) grid has arrived and its writes are visible.
// Bounded: on expiry COBS_ERR_TIMEOUT is recorded and the caller goes on (its results are then undefined).
__device__ void grid_barrier(const Params &p) {
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    atomicAdd(CTL_MISC(p.ctl_bar), 1);
    bool ok = false;
    for (long long it = 0; it < kSpinLimit; ++it) {
      if (ld_volatile(CTL_MISC(p.ctl_bar)) >= (int)gridDim.x) { ok = true; break; }
      __nanosleep(50);
    }
    if (!ok) report(p.status, COBS_ERR_TIMEOUT);
    __threadfence();
  }
  __syncthreads();
}

// ---------------------------------------------------------------------------------------------------
// the kernel
// ---------------------------------------------------------------------------------------------------
template <int DT, int D, int WPT, int NT>
__global__ void __launch_bounds__(kFThreads, 1) fused_step_kernel(Params p, int phases) {
  extern __shared__ __align__(256) unsigned char fsm[];
  __shared__ __align__(8) uint64_t s_bars[kFWarps][2];     // one mbarrier per scoring stage per streaming warp
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int wg = blockIdx.x * kFWarps + warp, n_wg = gridDim.x * kFWarps;
  // sequence lengths are consulted at every change of unit: keep them in shared memory when they fit
  __shared__ int s_len[kLenCache];
  const int *seq_lens = p.seq_lens;
  if (threadIdx.x == 0) ctl_begin(p);          // (its round trip overlaps the loads of the lengths)
  if (p.B <= kLenCache) {
    for (int i = threadIdx.x; i < p.B; i += kFThreads) s_len[i] = p.seq_lens[i];
    seq_lens = s_len;
  }
  __syncthreads();
  if (s_ctl[2]) ctl_turn(p);
  if ((phases & PH_SCORE) && p.u_q) {
    project_queries(p);
    grid_barrier(p);
  }
  if (warp < kFWarps) {
    // ---- streaming warps: score their chunks, then attend their items -------------------------------------
    unsigned char *wsm = fsm + warp * kWarpSmemBytes;
    if (lane == 0) {
      mbar_init((uint32_t)__cvta_generic_to_shared(&s_bars[warp][0]), 1);
      mbar_init((uint32_t)__cvta_generic_to_shared(&s_bars[warp][1]), 1);
      asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    __syncwarp();
    COBS_STAMP(0);
    bool ring_free = true;
    if (phases & PH_SCORE) ring_free = score_phase<DT, D, WPT, NT>(p, seq_lens, wsm, &s_bars[warp][0], wg, n_wg, lane);
    COBS_STAMP(1);
    COBS_STAMP(2);
    // after a timeout in scoring the step's outputs are undefined; this warp leaves its items to the others
    if ((phases & PH_ATTEND) && ring_free) attend_phase<D>(p, seq_lens, wsm, wg, n_wg, lane, (phases & PH_SCORE) != 0);
    COBS_STAMP(3);
  } else if (phases & PH_SCORE) {
    // ---- selection team ----------------------------------------------------------------------------------------
    select_team<1>(p, seq_lens, (int)threadIdx.x - kFWarps * 32, 1, 1);
  }
  // (nothing to clean up: the next launch works on the other set of counters, see ctl_begin)
}

// The step with phase S on tcgen05 (packed E2M1, full key space, D = 128, r = 8); phases must include PH_SCORE.
__global__ void __launch_bounds__(kUThreads, 1) fused_step_umma_kernel(Params p, int phases, const __grid_constant__ CUtensorMap tmap_xi) {
  extern __shared__ unsigned char fsm_raw[];
  __shared__ __align__(8) uint64_t ubar[kBCount];
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  __shared__ int s_len[kLenCache];
  __shared__ UmmaList s_list;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int wg = blockIdx.x * kFWarps + warp, n_wg = gridDim.x * kFWarps;
  unsigned char *fsm = fsm_raw + ((1024u - ((uint32_t)__cvta_generic_to_shared(fsm_raw) & 1023u)) & 1023u);
  const uint32_t bars = (uint32_t)__cvta_generic_to_shared(ubar);
  const int *seq_lens = p.seq_lens;
  if (p.B <= kLenCache) {
    for (int i = threadIdx.x; i < p.B; i += kUThreads) s_len[i] = p.seq_lens[i];
    seq_lens = s_len;
  }
  if (threadIdx.x == 0) {
    for (int i = 0; i < kUStages; ++i) { mbar_init(bars + (kBFull + i) * 8, 1); mbar_init(bars + (kBEmpty + i) * 8, 4); }
    for (int i = 0; i < kUAccBufs; ++i) { mbar_init(bars + (kBTFull + i) * 8, 1); mbar_init(bars + (kBTEmpty + i) * 8, 4); }
    mbar_init(bars + kBTiles * 8, kSelWarps);
    s_abort = 0;
    ctl_begin(p);
    umma_list_make(s_list, p.B * p.Hkv, p.NB, (int)gridDim.x, (int)blockIdx.x);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == kFWarps + kSelWarps + 1) {       // the MMA warp owns the tensor memory
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n"
                 ::"r"((uint32_t)__cvta_generic_to_shared(&s_tmem)), "r"(kUAccCols * kUAccBufs));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (s_ctl[2]) ctl_turn(p);
  const uint32_t tmem = s_tmem;
  volatile int *abort_flag = &s_abort;
  if (warp < kFWarps) {
    COBS_STAMP(0);
    umma_epilogue(p, s_list, fsm, bars, tmem, warp, lane, abort_flag);
    COBS_STAMP(1);
    // every streaming warp is done with the scoring stages before any of them reuses the memory for attention
    asm volatile("bar.sync 4, %0;\n" ::"n"(kFWarps * 32) : "memory");
    COBS_STAMP(2);
    if (phases & PH_ATTEND) attend_phase<128>(p, seq_lens, fsm + warp * kWarpSmemBytes, wg, n_wg, lane, true);
    COBS_STAMP(3);
  } else if (warp < kFWarps + kSelWarps) {
    umma_build_tiles(p, s_list, fsm, bars, warp - kFWarps, lane);
    select_team<4>(p, seq_lens, (int)threadIdx.x - kFWarps * 32, 4, 0);
  } else if (warp == kFWarps + kSelWarps) {
    umma_producer(p, seq_lens, s_list, fsm, bars, &tmap_xi, lane, abort_flag);
  } else {
    umma_issuer(p, s_list, fsm, bars, tmem, lane, abort_flag);
  }
  // ---- the tensor memory goes back when every role is done (the counters need no clean-up, see ctl_begin) -------
  tc_fence_before();
  __syncthreads();
  if (warp == kFWarps + kSelWarps + 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kUAccCols * kUAccBufs));
  }
}

// ---------------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------------
template <int DT, int D, int WPT, int NT>
static cudaError_t launch_fused_t(Params p, int phases, cudaStream_t stream) {
  auto kern = fused_step_kernel<DT, D, WPT, NT>;
  static int grid_cache[64] = {0};             // resident grid size of this instantiation, per device
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  if (grid_cache[dev] == 0) {
    if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kFusedSmemBytes)) != cudaSuccess) return e;
    int sms = 0, occ = 0;
    if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, kFThreads, kFusedSmemBytes)) != cudaSuccess) return e;
    if (occ < 1) return cudaErrorLaunchOutOfResources;
    grid_cache[dev] = sms * occ;
  }
  void *args[] = {&p, &phases};
  // cooperative launch: the grid is resident as a whole (or the launch fails), which the cross-warp waits rely on
  e = cudaLaunchCooperativeKernel((const void *)kern, dim3(grid_cache[dev]), dim3(kFThreads), args, kFusedSmemBytes,
                                  stream);
  count_launch();
  return e;
}

// Whether the persistent kernel covers this configuration's scoring phase.
bool fused_score_supported(const Params &p) {
  if (p.skew) return false;                                     // the third-cumulant variant is scored by the generic kernel
  if (p.NB > kSelThreads * 16 || p.NB % 4 != 0) return false;   // the selection team holds at most 16 blocks per thread
  if (p.summ_dtype == COBS_SUMM_BF16) return p.u_q == nullptr;
  if (p.summ_dtype == COBS_SUMM_FP4_E2M1) {
    if (p.Ds_pad % 32 != 0) return false;
    const int scale_sz = (p.scale_dtype == COBS_SCALE_FP16) ? 2 : 4;
    if ((p.r * scale_sz) % 4 != 0) return false;
    return true;
  }
  return false;
}

// The tcgen05 scoring path is parity-tested but, as measured, not faster than the mma.sync path (its unpacked
// 4-bit rows take twice the shared memory per byte in flight, which halves the copy depth of a bandwidth-bound
// stream), so it is opt-in: environment variable COBS_SCORE_PATH=tcgen05, read at every call.
static bool umma_requested() {
  const char *v = getenv("COBS_SCORE_PATH");
  return v != nullptr && strcmp(v, "tcgen05") == 0;
}

// Whether phase S of this configuration runs on tcgen05 (see the section on it above).
static bool umma_score_supported(const Params &p) {
  if (!umma_requested() || !fused_score_supported(p)) return false;
  if (p.summ_dtype != COBS_SUMM_FP4_E2M1 || p.u_q != nullptr) return false;
  if (p.D != 128 || p.Ds_pad != 128 || p.r != 8 || p.G > 8) return false;
  if (p.NB % kUBlocks != 0) return false;                    // whole 32-block stages
  if ((size_t)p.B * p.Hkv * p.NB * 8 >= (size_t)1 << 31) return false;
  if (reinterpret_cast<uintptr_t>(p.xi) % 32 != 0 || reinterpret_cast<uintptr_t>(p.mean) % 16 != 0 ||
      reinterpret_cast<uintptr_t>(p.scale) % 16 != 0) return false;
  return true;
}

typedef CUresult (*cobs_tmap_encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                        const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                        CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static cudaError_t launch_fused_umma(Params p, int phases, cudaStream_t stream) {
  static cobs_tmap_encode_fn encode = nullptr;
  static std::mutex mu;
  static int grid_cache[64] = {0};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!encode) {
      void *fn = nullptr;
      cudaDriverEntryPointQueryResult qres;
      if ((e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres)) != cudaSuccess) return e;
      if (!fn || qres != cudaDriverEntryPointSuccess) return cudaErrorNotSupported;
      encode = reinterpret_cast<cobs_tmap_encode_fn>(fn);
    }
    if (grid_cache[dev] == 0) {
      if ((e = cudaFuncSetAttribute(fused_step_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kUSmemBytes)) != cudaSuccess)
        return e;
      int sms = 0, occ = 0;
      if ((e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
      if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, fused_step_umma_kernel, kUThreads, kUSmemBytes)) != cudaSuccess)
        return e;
      if (occ < 1) return cudaErrorLaunchOutOfResources;
      grid_cache[dev] = sms;                                  // one CTA per SM: the CTA holds the SM's tensor memory columns it asks for
    }
  }
  for (int bid = 0; bid < grid_cache[dev]; ++bid) {          // every unit a CTA meets needs its own operand tile
    UmmaList l;
    umma_list_make(l, p.B * p.Hkv, p.NB, grid_cache[dev], bid);
    if (l.n_tiles > kUTiles) return cudaErrorNotSupported;
  }
  // the factor rows as a 2-D tensor [rows][128 codes]; the element type makes the copy engine unpack 16 codes
  // (8 bytes) into a 16-byte slot, which is what tcgen05.mma.kind::f8f6f4 reads
  CUtensorMap tmap;
  const cuuint64_t dims[2] = {128, (cuuint64_t)p.B * p.Hkv * p.NB * 8};
  const cuuint64_t strides[1] = {64};
  const cuuint32_t box[2] = {128, kUBlocks * 8}, estr[2] = {1, 1};
  if (encode(&tmap, CU_TENSOR_MAP_DATA_TYPE_16U4_ALIGN16B, 2, p.xi, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return cudaErrorInvalidValue;
  void *args[] = {&p, &phases, &tmap};
  e = cudaLaunchCooperativeKernel((const void *)fused_step_umma_kernel, dim3(grid_cache[dev]), dim3(kUThreads), args, kUSmemBytes, stream);
  count_launch();
  count_tcgen05_launch();
  return e;
}

cudaError_t launch_fused(const Params &p, int phases, cudaStream_t stream) {
  if ((phases & PH_SCORE) && umma_score_supported(p)) {
    const cudaError_t e = launch_fused_umma(p, phases, stream);
    if (e != cudaErrorNotSupported) return e;                // not supported: too many units per CTA, or no encoder
  }
  const bool fp4 = p.summ_dtype == COBS_SUMM_FP4_E2M1 && (phases & PH_SCORE);
  if (!fp4) {
    return p.D == 128 ? launch_fused_t<COBS_SUMM_BF16, 128, 1, 1>(p, phases, stream)
                      : launch_fused_t<COBS_SUMM_BF16, 64, 1, 1>(p, phases, stream);
  }
  const int wpt = p.Ds_pad / 32;
  const bool sub = p.u_q != nullptr;
#define COBS_CASE(DD, WW)                                                                                   \
  if (p.D == DD && wpt == WW)                                                                               \
    return sub ? launch_fused_t<COBS_SUMM_FP4_E2M1, DD, WW, 2>(p, phases, stream)                           \
               : launch_fused_t<COBS_SUMM_FP4_E2M1, DD, WW, 1>(p, phases, stream);
  COBS_CASE(128, 4) COBS_CASE(128, 3) COBS_CASE(128, 2) COBS_CASE(128, 1) COBS_CASE(64, 2) COBS_CASE(64, 1)
#undef COBS_CASE
  return cudaErrorInvalidValue;
}

int32_t prepare_attend_params(const cobs_config *cfg, const void *q, const cobs_kv *kv, const int32_t *sel_idx,
                              const int32_t *sel_cnt, float *out, float *lse_or_null, Params *p);

// ---------------------------------------------------------------------------------------------------
// cobs_sparse_decode_static: the attention step with its scratch in device memory the library itself
// owns, for callers that may not allocate.
// ---------------------------------------------------------------------------------------------------
// The scratch lives here, in a file-scope device array.  Every GPU that loads the library holds these
// bytes until the process exits.  In host code the name below is only a handle: the device address is
// obtained once per device with cudaGetSymbolAddress and that pointer is what the kernel is given.
static __device__ __align__(256) unsigned char g_static_scratch[COBS_STATIC_SCRATCH_BYTES];

static void *static_scratch_address(cudaError_t *err) {
  static void *addr[64] = {nullptr};
  static std::mutex mu;
  int dev = 0;
  *err = cudaGetDevice(&dev);
  if (*err != cudaSuccess) return nullptr;
  if (dev < 0 || dev >= 64) { *err = cudaErrorInvalidDevice; return nullptr; }
  std::lock_guard<std::mutex> lock(mu);
  if (!addr[dev]) {
    void *ptr = nullptr;
    *err = cudaGetSymbolAddress(&ptr, g_static_scratch);     // the current device's copy of the array
    if (*err != cudaSuccess) return nullptr;
    addr[dev] = ptr;
  }
  return addr[dev];
}

}  // namespace cobs

extern "C" int32_t cobs_sparse_decode_static(const cobs_config *cfg, const void *q, const cobs_kv *kv,
                                             const int32_t *sel_idx, const int32_t *sel_cnt, float *out,
                                             float *lse_or_null, void *stream) {
  using namespace cobs;
  Params p;
  int32_t st = prepare_attend_params(cfg, q, kv, sel_idx, sel_cnt, out, lse_or_null, &p);
  if (st != COBS_OK) return st;
  // scratch layout: [status word, epoch word, item / barrier words: 256 B][3 counters per unit][split partials]
  const size_t units = (size_t)p.B * p.Hkv;
  const size_t ctl_bytes = (3 * units * sizeof(int) + 255) / 256 * 256;     // every call starts from cleared words: set 0 only
  const size_t partial_bytes = units * p.n_splits * p.G * (size_t)(p.D + 2) * sizeof(float);
  if (kStatusBytes + ctl_bytes + partial_bytes > (size_t)COBS_STATIC_SCRATCH_BYTES) return COBS_ERR_WORKSPACE_TOO_SMALL;
  cudaError_t e = cudaSuccess;
  unsigned char *base = static_cast<unsigned char *>(static_scratch_address(&e));
  if (!base) return COBS_ERR_CUDA;
  p.status = reinterpret_cast<int32_t *>(base);
  p.ctl_epoch = reinterpret_cast<int *>(base) + 1;
  p.ctl_item = reinterpret_cast<int *>(base) + 2;
  p.ctl_bar = reinterpret_cast<int *>(base) + 3;
  p.ctl_set_stride = 0;                       // (the extent word is cleared with the rest: the other set is never touched)
  p.ctl_score = reinterpret_cast<int *>(base + kStatusBytes);
  p.ctl_ready = p.ctl_score + units;
  p.ctl_att = p.ctl_ready + units;
  p.partial = reinterpret_cast<float *>(base + kStatusBytes + ctl_bytes);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // the array keeps whatever the previous call left: the status word and the counters must start at zero
  if (cudaMemsetAsync(base, 0, kStatusBytes + ctl_bytes, s) != cudaSuccess) return COBS_ERR_CUDA;
  return launch_fused(p, PH_ATTEND, s) == cudaSuccess ? COBS_OK : COBS_ERR_CUDA;
}

#ifdef COBS_TIMING
extern "C" int cobs_debug_times(unsigned long long *host_out) {
  return (int)cudaMemcpyFromSymbol(host_out, cobs::g_dbg_times, sizeof(unsigned long long) * 4 * 4096);
}
extern "C" int cobs_debug_acc(unsigned long long *host_out, int clear) {
  int e = (int)cudaMemcpyFromSymbol(host_out, cobs::g_dbg_acc, sizeof(unsigned long long) * 8 * 4096);
  if (clear) { static unsigned long long z[8 * 4096]; cudaMemcpyToSymbol(cobs::g_dbg_acc, z, sizeof(z)); }
  return e;
}
#endif
