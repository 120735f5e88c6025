// Host side of the C ABI: argument validation, workspace carving, kernel launches.
#include <cstdio>
#include <cstring>

#include <cstdlib>

#include "common.cuh"

#include <atomic>

namespace cobs {
static std::atomic<long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
static std::atomic<long long> g_tc_launches{0};
void count_tcgen05_launch() { g_tc_launches.fetch_add(1, std::memory_order_relaxed); }

cudaError_t launch_score(const Params &p, cudaStream_t stream);
cudaError_t launch_select(const Params &p, cudaStream_t stream);
cudaError_t launch_exact_mass(const Params &p, cudaStream_t stream);
cudaError_t launch_adaptive_trim(const Params &p, float tau, int k_min, cudaStream_t stream);
cudaError_t launch_fused(const Params &p, int phases, cudaStream_t stream);
bool fused_score_supported(const Params &p);
enum { PH_SCORE = 1, PH_ATTEND = 2 };
cudaError_t launch_build(const Params &p, int block_begin, int block_end, cudaStream_t stream);
cudaError_t launch_append(const Params &p, const void *k_new, const void *v_new, void *k_pages, void *v_pages, int32_t *seq_lens,
                          int32_t *old_lens, cudaStream_t stream);
cudaError_t launch_quantise(const float *xi, long long n_vectors, int Ds, int Ds_pad, int scale_dtype, void *codes,
                            void *scale, cudaStream_t stream);
size_t build_smem_bytes(const Params &p);

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Packed FP4 rows are padded to a whole number of 16-byte units (32 codes), so that every row of
// every block starts on a 16-byte boundary.
static int padded_sub_dim(int Ds, int /*r*/) { return (Ds + 31) / 32 * 32; }

constexpr int kItemGroups = 256;         // 16-token groups one attention work item may hold
constexpr int kGridWarps = 148 * 8;      // streaming warps of the persistent kernel on a B200 (sizing heuristic only)

static int max_items(const cobs_config *c) {
  return c->topk + (c->window + c->block_size - 1) / c->block_size + 1;
}

static bool is_pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }

static int32_t validate_config(const cobs_config *c) {
  if (!c) return COBS_ERR_INVALID_ARG;
  if (c->batch < 1 || c->n_kv_heads < 1 || c->n_q_heads < 1) return COBS_ERR_INVALID_ARG;
  if (c->n_q_heads % c->n_kv_heads != 0) return COBS_ERR_INVALID_ARG;
  const int G = c->n_q_heads / c->n_kv_heads;
  if (!(G == 1 || G == 2 || G == 4 || G == 8)) return COBS_ERR_UNSUPPORTED;
  if (!(c->head_dim == 64 || c->head_dim == 128)) return COBS_ERR_UNSUPPORTED;
  if (!is_pow2(c->block_size) || c->block_size < 16 || c->block_size > 128) return COBS_ERR_UNSUPPORTED;
  if (!is_pow2(c->page_size) || c->page_size < 16 || c->page_size > c->block_size) return COBS_ERR_INVALID_ARG;
  if (c->rank < 0 || c->rank > COBS_MAX_RANK) return COBS_ERR_INVALID_ARG;
  if (c->sub_dim != 0 && (c->sub_dim < 8 || c->sub_dim > c->head_dim)) return COBS_ERR_INVALID_ARG;
  if (c->topk < 1 || c->topk > COBS_MAX_TOPK) return COBS_ERR_INVALID_ARG;
  if (c->window < 1) return COBS_ERR_INVALID_ARG;
  if (c->summary_dtype < COBS_SUMM_FP32 || c->summary_dtype > COBS_SUMM_FP4_E2M1) return COBS_ERR_INVALID_ARG;
  if (c->summary_dtype == COBS_SUMM_FP4_E2M1 && c->scale_dtype != COBS_SCALE_FP32 && c->scale_dtype != COBS_SCALE_FP16)
    return COBS_ERR_INVALID_ARG;
  if (c->max_blocks < 1) return COBS_ERR_INVALID_ARG;
  // the generic selection kernel keeps a unit's scores in shared memory (4 bytes per block, 227 KB at most)
  if (c->max_blocks > COBS_MAX_BLOCKS) return COBS_ERR_UNSUPPORTED;
  if (c->max_pages_per_seq < 1) return COBS_ERR_INVALID_ARG;
  // the page table must cover every full block (NB * L tokens); a sequence longer than max_pages_per_seq * P
  // is caught on the device (COBS_ERR_BOUNDS, the tokens beyond the table are skipped)
  if ((long long)c->max_pages_per_seq * c->page_size < (long long)c->max_blocks * c->block_size) return COBS_ERR_INVALID_ARG;
  // an attention slice holds at most kItemGroups 16-token groups and a unit at most kMaxSplits slices
  if ((long long)max_items(c) * (c->block_size / 16) > (long long)kItemGroups * kMaxSplits) return COBS_ERR_UNSUPPORTED;
  // units index grid.y of the generic scoring kernel (65535 at most) and the workspace's counters
  if ((long long)c->batch * c->n_kv_heads > kMaxUnits) return COBS_ERR_UNSUPPORTED;
  // chunk and item indices are 32-bit
  if ((long long)c->batch * c->n_kv_heads * ((c->max_blocks + 15) / 16) > 0x3fffffffLL) return COBS_ERR_UNSUPPORTED;
  return COBS_OK;
}

// Attention slices per (sequence, KV head): one slice per warp of the persistent grid when the batch is
// large enough for that, never more than there are 16-token groups to read, and enough that a slice
// fits the kernel's per-warp group table.
static int choose_splits(const cobs_config *c) {
  const int units = c->batch * c->n_kv_heads;
  const int groups = max_items(c) * (c->block_size / 16);
  // Two slices per streaming warp when the scoring runs in waves (then the second round of items absorbs the units
  // whose selection finishes last); one per warp otherwise (an item costs several microseconds beyond its bytes).
  const long long chunks = (long long)units * ((c->max_blocks + 15) / 16);
  const int per_warp = (chunks / kGridWarps >= 2) ? 2 : 1;
  int s = per_warp * kGridWarps / units;
  const int need = (groups + kItemGroups - 1) / kItemGroups;
  if (s < need) s = need;
  // small batches: more slices shorten each slice's stream (about 1.2 us per 16-token group) but lengthen the merge
  // (about 0.25 us per slice); the sum is smallest near sqrt(5 * groups)
  int cap = 1;
  while ((cap + 1) * (cap + 1) <= 5 * groups) ++cap;
  if (s > cap) s = cap;
  if (s < need) s = need;
  if (s > groups) s = groups;
  if (s > kMaxSplits) s = kMaxSplits;
  if (s < 1) s = 1;
  return s;
}

struct WorkspaceLayout {
  size_t status, ctl, e, lse_part, partial, sel_idx, sel_cnt, qtilde, q_stage, out_stage, total;
};

static WorkspaceLayout layout_workspace(const cobs_config *c) {
  WorkspaceLayout w;
  const size_t B = c->batch, Hq = c->n_q_heads, Hkv = c->n_kv_heads, G = Hq / Hkv, D = c->head_dim;
  size_t off = 0;
  w.status = off; off += kStatusBytes;
  // two sets of three counters per unit.  The area has the size of the largest shape (1.5 MB) and set 1 starts
  // 3 * kMaxUnits ints after set 0 whatever the shape, so that a workspace that serves calls of different shapes keeps
  // its counters in the same places and no call's scratch arrays lie over another shape's counters
  w.ctl = off; off = align_up(off + 6 * (size_t)kMaxUnits * sizeof(int), 256);
  w.e = off; off = align_up(off + B * Hq * (size_t)c->max_blocks * sizeof(float), 256);
  w.lse_part = off; off = align_up(off + B * Hq * (size_t)((c->max_blocks + 15) / 16) * 4 * 2 * sizeof(float), 256);   // up to four pairs per chunk
  w.partial = off; off = align_up(off + B * Hkv * (size_t)choose_splits(c) * G * (D + 2) * sizeof(float), 256);
  w.sel_idx = off; off = align_up(off + B * Hkv * (size_t)c->topk * sizeof(int32_t), 256);
  w.sel_cnt = off; off = align_up(off + B * Hkv * sizeof(int32_t), 256);
  w.qtilde = off; off = align_up(off + (c->sub_dim ? B * Hq * (size_t)((c->sub_dim + 31) / 32 * 32) * sizeof(float) : 0), 256);
  w.q_stage = off; off = align_up(off + B * Hq * D * 2, 256);
  w.out_stage = off; off = align_up(off + B * Hq * D * sizeof(float), 256);
  w.total = off;
  return w;
}

static void fill_params(Params &p, const cobs_config *c, void *workspace) {
  memset(&p, 0, sizeof(p));
  p.B = c->batch; p.Hq = c->n_q_heads; p.Hkv = c->n_kv_heads; p.G = p.Hq / p.Hkv; p.D = c->head_dim;
  p.L = c->block_size; p.P = c->page_size; p.r = c->rank;
  p.Ds = c->sub_dim ? c->sub_dim : c->head_dim;
  p.Ds_pad = (c->summary_dtype == COBS_SUMM_FP4_E2M1) ? padded_sub_dim(p.Ds, p.r) : p.Ds;
  p.topk = c->topk; p.window = c->window; p.NB = c->max_blocks; p.mpp = c->max_pages_per_seq;
  p.summ_dtype = c->summary_dtype; p.scale_dtype = c->scale_dtype;
  p.n_splits = choose_splits(c);
  if (workspace) {
    WorkspaceLayout w = layout_workspace(c);
    char *base = static_cast<char *>(workspace);
    p.status = reinterpret_cast<int32_t *>(base + w.status);
    p.ctl_epoch = reinterpret_cast<int *>(base + w.status) + 1;
    p.ctl_item = reinterpret_cast<int *>(base + w.status) + 2;
    p.ctl_bar = reinterpret_cast<int *>(base + w.status) + 3;
    p.ctl_score = reinterpret_cast<int *>(base + w.ctl);
    p.ctl_set_stride = 3 * kMaxUnits;
    p.ctl_ready = p.ctl_score + (size_t)p.B * p.Hkv;
    p.ctl_att = p.ctl_ready + (size_t)p.B * p.Hkv;
    p.qtilde_out = reinterpret_cast<float *>(base + w.qtilde);
    p.e = reinterpret_cast<float *>(base + w.e);
    p.lse_part = reinterpret_cast<float *>(base + w.lse_part);
    p.partial = reinterpret_cast<float *>(base + w.partial);
    p.sel_idx = reinterpret_cast<int32_t *>(base + w.sel_idx);
    p.sel_cnt = reinterpret_cast<int32_t *>(base + w.sel_cnt);
  }
}

static int32_t check_workspace(const cobs_config *c, void *workspace, size_t bytes) {
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return COBS_ERR_INVALID_ARG;
  if (bytes < layout_workspace(c).total) return COBS_ERR_WORKSPACE_TOO_SMALL;
  return COBS_OK;
}

static int32_t set_summaries(Params &p, const cobs_config *c, const cobs_summaries *s) {
  if (!s || !s->mean || !aligned16(s->mean)) return COBS_ERR_INVALID_ARG;
  if (c->rank > 0 && (!s->xi || !aligned16(s->xi))) return COBS_ERR_INVALID_ARG;
  if (c->rank > 0 && c->summary_dtype == COBS_SUMM_FP4_E2M1 && (!s->scale || !aligned16(s->scale)))
    return COBS_ERR_INVALID_ARG;
  if (c->sub_dim != 0 && (!s->u_q || !aligned16(s->u_q))) return COBS_ERR_INVALID_ARG;
  p.mean = s->mean; p.xi = s->xi; p.scale = s->scale;
  p.u_q = c->sub_dim ? s->u_q : nullptr;
  if (s->skew) {
    if (c->sub_dim != 0 || c->rank < 1) return COBS_ERR_UNSUPPORTED;
    if (!aligned16(s->skew)) return COBS_ERR_INVALID_ARG;
    p.skew = s->skew;
  }
  return COBS_OK;
}

static int32_t set_kv(Params &p, const cobs_kv *kv) {
  if (!kv || !kv->k_pages || !kv->v_pages || !kv->page_table || !kv->seq_lens || kv->n_pages < 1)
    return COBS_ERR_INVALID_ARG;
  if (!aligned16(kv->k_pages) || !aligned16(kv->v_pages)) return COBS_ERR_INVALID_ARG;
  p.k_pages = static_cast<const __nv_bfloat16 *>(kv->k_pages);
  p.v_pages = static_cast<const __nv_bfloat16 *>(kv->v_pages);
  p.page_table = kv->page_table; p.seq_lens = kv->seq_lens; p.n_pages = kv->n_pages;
  return COBS_OK;
}

static int32_t cuda_status(cudaError_t e) { return e == cudaSuccess ? COBS_OK : COBS_ERR_CUDA; }

// Validated kernel parameters of an attention-only call whose scratch is not a caller workspace.
// Fills everything except the scratch pointers (status, counters, partials); reports the attention
// slices per unit so that the caller can lay its scratch out.
int32_t prepare_attend_params(const cobs_config *cfg, const void *q, const cobs_kv *kv, const int32_t *sel_idx,
                              const int32_t *sel_cnt, float *out, float *lse_or_null, Params *p) {
  int32_t st = validate_config(cfg);
  if (st != COBS_OK) return st;
  if (!q || !aligned16(q) || !sel_idx || !sel_cnt || !out || !aligned16(out)) return COBS_ERR_INVALID_ARG;
  fill_params(*p, cfg, nullptr);
  if ((st = set_kv(*p, kv)) != COBS_OK) return st;
  p->q = static_cast<const __nv_bfloat16 *>(q);
  p->sel_idx = const_cast<int32_t *>(sel_idx); p->sel_cnt = const_cast<int32_t *>(sel_cnt);
  p->out = out; p->lse = lse_or_null;
  return COBS_OK;
}

}  // namespace cobs

using namespace cobs;

extern "C" {

const char *cobs_status_string(int32_t s) {
  switch (s) {
    case COBS_OK: return "ok";
    case COBS_ERR_INVALID_ARG: return "invalid argument";
    case COBS_ERR_UNSUPPORTED: return "unsupported shape";
    case COBS_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case COBS_ERR_CUDA: return "CUDA runtime error";
    case COBS_ERR_TIMEOUT: return "device-side wait ran out";
    case COBS_ERR_BOUNDS: return "index out of range on the device (access skipped)";
    default: return "unknown status";
  }
}

int64_t cobs_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }
int64_t cobs_tcgen05_launches(void) { return g_tc_launches.load(std::memory_order_relaxed); }

int32_t cobs_padded_sub_dim(const cobs_config *cfg) {
  if (validate_config(cfg) != COBS_OK) return -1;
  return padded_sub_dim(cfg->sub_dim ? cfg->sub_dim : cfg->head_dim, cfg->rank);
}

int32_t cobs_summary_bytes(const cobs_config *cfg, size_t *mean_bytes, size_t *xi_bytes, size_t *scale_bytes) {
  int32_t st = validate_config(cfg);
  if (st != COBS_OK) return st;
  if (!mean_bytes || !xi_bytes || !scale_bytes) return COBS_ERR_INVALID_ARG;
  const size_t n = (size_t)cfg->batch * cfg->n_kv_heads * cfg->max_blocks;
  const int Ds = cfg->sub_dim ? cfg->sub_dim : cfg->head_dim;
  switch (cfg->summary_dtype) {
    case COBS_SUMM_FP32:
      *mean_bytes = n * cfg->head_dim * 4; *xi_bytes = n * cfg->rank * Ds * 4; *scale_bytes = 0; break;
    case COBS_SUMM_BF16:
      *mean_bytes = n * cfg->head_dim * 2; *xi_bytes = n * cfg->rank * Ds * 2; *scale_bytes = 0; break;
    default:
      *mean_bytes = n * cfg->head_dim * 2;
      *xi_bytes = n * cfg->rank * (padded_sub_dim(Ds, cfg->rank) / 2);
      *scale_bytes = n * cfg->rank * (cfg->scale_dtype == COBS_SCALE_FP16 ? 2 : 4);
      break;
  }
  return COBS_OK;
}

int32_t cobs_workspace_bytes(const cobs_config *cfg, size_t *bytes) {
  int32_t st = validate_config(cfg);
  if (st != COBS_OK) return st;
  if (!bytes) return COBS_ERR_INVALID_ARG;
  *bytes = layout_workspace(cfg).total;
  return COBS_OK;
}

int32_t cobs_reset_status(void *workspace, size_t workspace_bytes, void *stream) {
  if (!workspace || workspace_bytes < (size_t)kStatusBytes) return COBS_ERR_INVALID_ARG;
  const size_t n = workspace_bytes < (size_t)kCtlBytes ? workspace_bytes : (size_t)kCtlBytes;
  return cuda_status(cudaMemsetAsync(workspace, 0, n, static_cast<cudaStream_t>(stream)));
}

int32_t cobs_read_status(void *workspace, size_t workspace_bytes, void *stream, int32_t *code_host) {
  if (!workspace || workspace_bytes < (size_t)kStatusBytes || !code_host) return COBS_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemcpyAsync(code_host, workspace, sizeof(int32_t), cudaMemcpyDeviceToHost, s);
  if (e != cudaSuccess) return COBS_ERR_CUDA;
  return cuda_status(cudaStreamSynchronize(s));
}

int32_t cobs_build_summaries(const cobs_config *cfg, const cobs_kv *kv, int32_t block_begin, int32_t block_end,
                             const cobs_summaries *out, void *workspace, size_t workspace_bytes, void *stream) {
  int32_t st = validate_config(cfg);
  if (st != COBS_OK) return st;
  if ((st = check_workspace(cfg, workspace, workspace_bytes)) != COBS_OK) return st;
  if (block_begin < 0 || block_end < block_begin || block_end > cfg->max_blocks) return COBS_ERR_INVALID_ARG;
  Params p;
  fill_params(p, cfg, workspace);
  if ((st = set_kv(p, kv)) != COBS_OK) return st;
  if ((st = set_summaries(p, cfg, out)) != COBS_OK) return st;
  if (build_smem_bytes(p) > 227 * 1024) return COBS_ERR_UNSUPPORTED;
  // one CTA per (sequence, KV head, block of the range): the grid's x extent is 2^31 - 1 at most
  if ((long long)p.B * p.Hkv * (block_end - block_begin) > 0x7fffffffLL) return COBS_ERR_UNSUPPORTED;
  return cuda_status(launch_build(p, block_begin, block_end, static_cast<cudaStream_t>(stream)));
}

int32_t cobs_append_token(const cobs_config *cfg, const void *k_new, const void *v_new, void *k_pages, void *v_pages,
                          const int32_t *page_table, int32_t *seq_lens, int64_t n_pages, void *workspace,
                          size_t workspace_bytes, void *stream) {
  int32_t st = validate_config(cfg);
  if (st != COBS_OK) return st;
  if ((st = check_workspace(cfg, workspace, workspace_bytes)) != COBS_OK) return st;
  if (!k_new || !v_new || !k_pages || !v_pages || !page_table || !seq_lens || n_pages < 1) return COBS_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new) | reinterpret_cast<uintptr_t>(k_pages) |
       reinterpret_cast<uintptr_t>(v_pages)) % 16 != 0) return COBS_ERR_INVALID_ARG;
  Params p;
  fill_params(p, cfg, workspace);
  p.page_table = page_table;
  p.n_pages = n_pages;
  // the snapshot of the lengths lives in the query staging area of the workspace (batch * 4 bytes of it)
  int32_t *old_lens = reinterpret_cast<int32_t *>(static_cast<unsigned char *>(workspace) + layout_workspace(cfg).q_stage);
  return cuda_status(launch_append(p, k_new, v_new, k_pages, v_pages, seq_lens, old_lens, static_cast<cudaStream_t>(stream)));
}

int32_t cobs_quantise_xi(const cobs_config *cfg, const float *xi_fp32, int64_t n_vectors, void *codes, void *scale,
                         void *stream) {
  int32_t st = validate_config(cfg);
  if (st != COBS_OK) return st;
  if (!xi_fp32 || !codes || !scale || n_vectors < 0 || cfg->rank < 1 || n_vectors % cfg->rank != 0)
    return COBS_ERR_INVALID_ARG;
  if (!aligned16(codes) || !aligned16(scale) || !aligned16(xi_fp32)) return COBS_ERR_INVALID_ARG;
  const int Ds = cfg->sub_dim ? cfg->sub_dim : cfg->head_dim;
  return cuda_status(launch_quantise(xi_fp32, n_vectors, Ds, padded_sub_dim(Ds, cfg->rank), cfg->scale_dtype, codes,
                                     scale, static_cast<cudaStream_t>(stream)));
}

int32_t cobs_score_select(const cobs_config *cfg, const void *q, const cobs_summaries *summ, const int32_t *seq_lens,
                          int32_t *sel_idx, int32_t *sel_cnt, float *scores_or_null, void *workspace,
                          size_t workspace_bytes, void *stream) {
  int32_t st = validate_config(cfg);
  if (st != COBS_OK) return st;
  if ((st = check_workspace(cfg, workspace, workspace_bytes)) != COBS_OK) return st;
  if (!q || !aligned16(q) || !seq_lens || !sel_idx || !sel_cnt) return COBS_ERR_INVALID_ARG;
  Params p;
  fill_params(p, cfg, workspace);
  if ((st = set_summaries(p, cfg, summ)) != COBS_OK) return st;
  p.q = static_cast<const __nv_bfloat16 *>(q);
  p.seq_lens = seq_lens;
  p.sel_idx = sel_idx; p.sel_cnt = sel_cnt; p.scores = scores_or_null;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (fused_score_supported(p)) {
    if (p.u_q) p.qtilde = p.qtilde_out;
    return cuda_status(launch_fused(p, PH_SCORE, s));
  }
  cudaError_t e = launch_score(p, s);
  if (e != cudaSuccess) return COBS_ERR_CUDA;
  return cuda_status(launch_select(p, s));
}

int32_t cobs_exact_select(const cobs_config *cfg, const void *q, const cobs_kv *kv, int32_t *sel_idx, int32_t *sel_cnt,
                          float *scores_or_null, void *workspace, size_t workspace_bytes, void *stream) {
  int32_t st = validate_config(cfg);
  if (st != COBS_OK) return st;
  if ((st = check_workspace(cfg, workspace, workspace_bytes)) != COBS_OK) return st;
  if (!q || !aligned16(q) || !sel_idx || !sel_cnt) return COBS_ERR_INVALID_ARG;
  Params p;
  fill_params(p, cfg, workspace);
  if ((st = set_kv(p, kv)) != COBS_OK) return st;
  p.q = static_cast<const __nv_bfloat16 *>(q);
  p.sel_idx = sel_idx; p.sel_cnt = sel_cnt; p.scores = scores_or_null;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (launch_exact_mass(p, s) != cudaSuccess) return COBS_ERR_CUDA;
  return cuda_status(launch_select(p, s));
}

int32_t cobs_adaptive_trim(const cobs_config *cfg, const float *scores, const int32_t *seq_lens, float tau, int32_t k_min,
                           int32_t *sel_idx, int32_t *sel_cnt, void *workspace, size_t workspace_bytes, void *stream) {
  int32_t st = validate_config(cfg);
  if (st != COBS_OK) return st;
  if ((st = check_workspace(cfg, workspace, workspace_bytes)) != COBS_OK) return st;
  if (!scores || !seq_lens || !sel_idx || !sel_cnt) return COBS_ERR_INVALID_ARG;
  if (!(tau >= 0.f && tau < 1.f) || k_min < 0) return COBS_ERR_INVALID_ARG;
  if (cfg->topk > 128) return COBS_ERR_UNSUPPORTED;
  Params p;
  fill_params(p, cfg, workspace);
  p.seq_lens = seq_lens;
  p.scores = const_cast<float *>(scores);
  p.sel_idx = sel_idx; p.sel_cnt = sel_cnt;
  return cuda_status(launch_adaptive_trim(p, tau, k_min, static_cast<cudaStream_t>(stream)));
}

int32_t cobs_sparse_decode(const cobs_config *cfg, const void *q, const cobs_kv *kv, const int32_t *sel_idx,
                           const int32_t *sel_cnt, float *out, float *lse_or_null, void *workspace,
                           size_t workspace_bytes, void *stream) {
  int32_t st = validate_config(cfg);
  if (st != COBS_OK) return st;
  if ((st = check_workspace(cfg, workspace, workspace_bytes)) != COBS_OK) return st;
  if (!q || !aligned16(q) || !sel_idx || !sel_cnt || !out || !aligned16(out)) return COBS_ERR_INVALID_ARG;
  Params p;
  fill_params(p, cfg, workspace);
  if ((st = set_kv(p, kv)) != COBS_OK) return st;
  p.q = static_cast<const __nv_bfloat16 *>(q);
  p.sel_idx = const_cast<int32_t *>(sel_idx); p.sel_cnt = const_cast<int32_t *>(sel_cnt);
  p.out = out; p.lse = lse_or_null;
  return cuda_status(launch_fused(p, PH_ATTEND, static_cast<cudaStream_t>(stream)));
}

int32_t cobs_decode_step(const cobs_config *cfg, const void *q, const cobs_kv *kv, const cobs_summaries *summ,
                         float *out, float *lse_or_null, int32_t *sel_idx_or_null, int32_t *sel_cnt_or_null,
                         void *workspace, size_t workspace_bytes, void *stream) {
  int32_t st = validate_config(cfg);
  if (st != COBS_OK) return st;
  if ((st = check_workspace(cfg, workspace, workspace_bytes)) != COBS_OK) return st;
  if (!q || !aligned16(q) || !out || !aligned16(out)) return COBS_ERR_INVALID_ARG;
  if ((sel_idx_or_null == nullptr) != (sel_cnt_or_null == nullptr)) return COBS_ERR_INVALID_ARG;
  Params p;
  fill_params(p, cfg, workspace);
  if ((st = set_kv(p, kv)) != COBS_OK) return st;
  if ((st = set_summaries(p, cfg, summ)) != COBS_OK) return st;
  p.q = static_cast<const __nv_bfloat16 *>(q);
  if (sel_idx_or_null) { p.sel_idx = sel_idx_or_null; p.sel_cnt = sel_cnt_or_null; }
  p.out = out; p.lse = lse_or_null;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (fused_score_supported(p)) {
    if (p.u_q) p.qtilde = p.qtilde_out;
    return cuda_status(launch_fused(p, PH_SCORE | PH_ATTEND, s));
  }
  // summaries the persistent kernel's scoring phase does not cover (fp32, odd subspace widths):
  // generic scoring and selection kernels first, then the persistent kernel for the attention
  cudaError_t e = launch_score(p, s);
  if (e != cudaSuccess) return COBS_ERR_CUDA;
  if ((e = launch_select(p, s)) != cudaSuccess) return COBS_ERR_CUDA;
  return cuda_status(launch_fused(p, PH_ATTEND, s));
}

int32_t cobs_decode_step_host(const cobs_config *cfg, const void *q_host, const cobs_kv *kv,
                              const cobs_summaries *summ, float *out_host, int32_t *sel_idx_host_or_null,
                              int32_t *sel_cnt_host_or_null, void *workspace, size_t workspace_bytes, void *stream) {
  int32_t st = validate_config(cfg);
  if (st != COBS_OK) return st;
  if ((st = check_workspace(cfg, workspace, workspace_bytes)) != COBS_OK) return st;
  if (!q_host || !out_host) return COBS_ERR_INVALID_ARG;
  if ((sel_idx_host_or_null == nullptr) != (sel_cnt_host_or_null == nullptr)) return COBS_ERR_INVALID_ARG;
  WorkspaceLayout w = layout_workspace(cfg);
  char *base = static_cast<char *>(workspace);
  void *q_dev = base + w.q_stage;
  float *out_dev = reinterpret_cast<float *>(base + w.out_stage);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t n = (size_t)cfg->batch * cfg->n_q_heads * cfg->head_dim;
  if (cudaMemcpyAsync(q_dev, q_host, n * 2, cudaMemcpyHostToDevice, s) != cudaSuccess) return COBS_ERR_CUDA;
  // Pinned, device-mapped output memory: the merge writes its rows straight into it (posted writes over PCIe, 256 KB
  // spread over the tail of the kernel), which saves a device-to-host copy and its latency after the kernel.  Any
  // other host memory goes through the staging buffer.
  float *out_direct = nullptr;
  {
    cudaPointerAttributes attr;
    if (cudaPointerGetAttributes(&attr, out_host) == cudaSuccess && attr.type == cudaMemoryTypeHost &&
        attr.devicePointer != nullptr && aligned16(attr.devicePointer))
      out_direct = static_cast<float *>(attr.devicePointer);
    else
      (void)cudaGetLastError();                  // unregistered host memory reports an error on some drivers: clear it
  }
  st = cobs_decode_step(cfg, q_dev, kv, summ, out_direct ? out_direct : out_dev, nullptr, nullptr, nullptr, workspace,
                        workspace_bytes, stream);
  if (st != COBS_OK) return st;
  if (!out_direct && cudaMemcpyAsync(out_host, out_dev, n * sizeof(float), cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return COBS_ERR_CUDA;
  if (sel_idx_host_or_null) {
    const size_t units = (size_t)cfg->batch * cfg->n_kv_heads;
    if (cudaMemcpyAsync(sel_idx_host_or_null, base + w.sel_idx, units * cfg->topk * sizeof(int32_t),
                        cudaMemcpyDeviceToHost, s) != cudaSuccess) return COBS_ERR_CUDA;
    if (cudaMemcpyAsync(sel_cnt_host_or_null, base + w.sel_cnt, units * sizeof(int32_t), cudaMemcpyDeviceToHost,
                        s) != cudaSuccess) return COBS_ERR_CUDA;
  }
  return cuda_status(cudaStreamSynchronize(s));
}

}  // extern "C"
