// Adaptive number of selected blocks: an extension, NOT in the paper (which always keeps k blocks).  It applies the
// paper's dropped mass tau (the normalised block mass outside the kept set, Background, before Eq. prop-gqa) to the
// group score of Eq. prop-gqa:
//
//   k_adapt = the smallest k such that the k largest candidate scores hold at least (1 - tau) of the candidates'
//             total score, clamped to [k_min, topk] and to the number of candidates.
//
// The kernel trims an existing selection in place: the top-`topk` blocks of cobs_score_select (ascending index) and
// the scores the same call wrote.  One CTA of 128 threads per (sequence, KV head); topk <= 128.  Sums are taken in
// double precision in a fixed order (no atomics), so the result does not depend on scheduling.
#include "common.cuh"

namespace cobs {

namespace {

constexpr int kAThreads = 128;

__global__ void __launch_bounds__(kAThreads) adaptive_trim_kernel(Params p, float tau, int k_min) {
  __shared__ double s_part[kAThreads];
  __shared__ double s_sorted[kAThreads];
  __shared__ float s_score[kAThreads];
  __shared__ int s_id[kAThreads];
  __shared__ int s_warp[kAThreads / 32];
  __shared__ int s_k;
  const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b_idx = u / p.Hkv;
  const int T = p.seq_lens[b_idx];
  const int n_sum = min(T / p.L, p.NB);
  const int n_cand = min(window_start(T, p.window, p.L) / p.L, n_sum);
  const float *sc = p.scores + (size_t)u * p.NB;
  int32_t *out = p.sel_idx + (size_t)u * p.topk;
  const int k = min(min(p.sel_cnt[u], p.topk), n_cand);
  // ---- total score of the candidates: strided partial sums, then a fixed-order tree ----------------------------
  double part = 0.0;
  for (int b = tid; b < n_cand; b += kAThreads) part += (double)sc[b];
  s_part[tid] = part;
  // ---- this thread's selected block ------------------------------------------------------------------------------
  int id = -1;
  float my = 0.f;
  if (tid < k) {
    id = out[tid];
    if (id < 0 || id >= n_cand) { report(p.status, COBS_ERR_BOUNDS); id = -1; }
    else my = sc[id];
  }
  s_id[tid] = id;
  s_score[tid] = my;
  __syncthreads();
  for (int o = kAThreads / 2; o > 0; o >>= 1) {
    if (tid < o) s_part[tid] += s_part[tid + o];
    __syncthreads();
  }
  const double total = s_part[0];
  // ---- rank among the selected: larger score first, lower index on ties ------------------------------------------
  int rank = k;
  if (tid < k && id >= 0) {
    rank = 0;
    for (int j = 0; j < k; ++j) {
      const int oj = s_id[j];
      if (oj < 0) continue;
      const float sj = s_score[j];
      rank += (sj > my || (sj == my && oj < id)) ? 1 : 0;
    }
    s_sorted[rank] = (double)my;
  }
  __syncthreads();
  if (tid == 0) {
    int valid = 0;
    for (int j = 0; j < k; ++j) valid += (s_id[j] >= 0);
    const double need = (1.0 - (double)tau) * total;
    int ka = valid;
    double cum = 0.0;
    for (int j = 0; j < valid; ++j) {
      cum += s_sorted[j];
      if (cum >= need) { ka = j + 1; break; }
    }
    ka = max(ka, min(k_min, valid));
    s_k = min(ka, valid);
  }
  __syncthreads();
  const int ka = s_k;
  // ---- keep the ka best, in ascending index order (the order they came in) ------------------------------------------
  const bool keep = tid < k && id >= 0 && rank < ka;
  const unsigned m = __ballot_sync(0xffffffffu, keep);
  if (lane == 0) s_warp[warp] = __popc(m);
  __syncthreads();
  int pos = __popc(m & ((1u << lane) - 1u));
  for (int w = 0; w < warp; ++w) pos += s_warp[w];
  __syncthreads();                               // every thread has read its block before any slot is rewritten
  if (keep) out[pos] = id;
  for (int i = ka + tid; i < p.topk; i += kAThreads) out[i] = -1;
  if (tid == 0) p.sel_cnt[u] = ka;
}

}  // namespace

cudaError_t launch_adaptive_trim(const Params &p, float tau, int k_min, cudaStream_t stream) {
  adaptive_trim_kernel<<<p.B * p.Hkv, kAThreads, 0, stream>>>(p, tau, k_min);
  count_launch();
  return cudaGetLastError();
}

}  // namespace cobs
