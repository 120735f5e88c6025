/*
 * cobs.h -- C ABI of the COBS (Cumulant Order Block Sparse attention) decode path for NVIDIA B200.
 *
 * One decode step of one attention layer, for a batch of sequences whose keys and
 * values live in a paged bf16 KV cache:
 *
 *   (a) cobs_build_summaries   per KV block: mean key, and the top-r scaled eigenvectors of the
 *                              within-block key covariance (full key space or a query subspace),
 *                              stored as fp32, bf16 or FP4 E2M1 with one scale per eigenvector
 *   (b,c) cobs_score_select    second-order estimate of every block's log attention mass for each
 *                              query head, the GQA group score, and the top-k blocks per KV head
 *   (d) cobs_sparse_decode     softmax attention over the selected blocks plus a local window
 *   fused: cobs_decode_step    (b) (c) (d) in one call
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer owned by the caller unless a parameter is named *_host.
 *     The library allocates no device memory and frees none; scratch comes from the caller as
 *     `workspace` (size from cobs_workspace_bytes, 256-byte aligned).  The workspace must not be
 *     shared by calls that may overlap on the GPU.  Calls of different configurations may use one
 *     workspace in turn if it is as large as the largest of them needs (the first 1.5 MB hold the
 *     status word and the hand-off counters of the persistent kernel, at the same places for every
 *     shape; cobs_reset_status clears them).
 *   - All work is enqueued on `stream` (a cudaStream_t passed as void*, NULL = default stream) and
 *     the call returns without synchronising, except the *_host entry point and cobs_read_status.
 *   - Arguments are validated on the host before anything is launched; a call that returns a
 *     nonzero status has launched nothing.
 *   - Device-side problems (an index outside its array, a bounded wait that ran out) do not fault:
 *     the kernel skips the access, records a code in the status word at the start of the workspace,
 *     and cobs_read_status returns it.
 *   - Shapes: B sequences, Hq query heads, Hkv KV heads, G = Hq/Hkv, head dimension D, block of L
 *     tokens, page of P tokens (P divides L), r stored eigenvectors, Ds = sub_dim or D.
 *   - The attention scale 1/sqrt(D) is folded into the query inside the library (the paper's
 *     Notation paragraph absorbs it into q); callers pass the raw query.
 *
 * Block / window rule (one per sequence of length T):
 *   summarised blocks   b < floor(T / L)          (only full blocks have summaries)
 *   window              tokens [ws, T), ws = floor(max(0, T - window) / L) * L
 *   candidates          blocks b < ws / L        (wholly before the window)
 *   selected            min(topk, ws / L) candidates with the largest group score; larger score
 *                       first, lower block index on equal scores; reported in ascending index
 *                       order, padded with -1.
 */
#ifndef COBS_H_
#define COBS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  COBS_OK = 0,
  COBS_ERR_INVALID_ARG = 1,         /* NULL pointer, misaligned pointer, inconsistent or out-of-range field */
  COBS_ERR_UNSUPPORTED = 2,         /* a shape this build has no kernel for */
  COBS_ERR_WORKSPACE_TOO_SMALL = 3,
  COBS_ERR_CUDA = 4,                /* a CUDA runtime call failed (launch configuration, copy) */
  COBS_ERR_TIMEOUT = 5,             /* device status: a bounded device-side wait ran out; the call's outputs are undefined */
  COBS_ERR_BOUNDS = 6               /* device status: a page id or block index was out of range and skipped */
} cobs_status;

typedef enum { COBS_SUMM_FP32 = 0, COBS_SUMM_BF16 = 1, COBS_SUMM_FP4_E2M1 = 2 } cobs_summary_dtype;
typedef enum { COBS_SCALE_FP32 = 0, COBS_SCALE_FP16 = 1 } cobs_scale_dtype;

#define COBS_MAX_TOPK 128
#define COBS_MAX_RANK 16
#define COBS_MAX_BLOCKS 57344       /* largest max_blocks (3.67 M tokens of context at L = 64) */
#define COBS_MAX_UNITS 65535        /* largest batch * n_kv_heads */

/* Problem statement: shapes and method parameters (paper: Background, Notation; Method). */
typedef struct {
  int32_t batch;              /* B >= 1 */
  int32_t n_q_heads;          /* Hq, a multiple of n_kv_heads; G = Hq / Hkv in {1, 2, 4, 8} */
  int32_t n_kv_heads;         /* Hkv >= 1 */
  int32_t head_dim;           /* D in {64, 128} */
  int32_t block_size;         /* L in {16, 32, 64, 128} */
  int32_t page_size;          /* P: tokens per KV page; >= 16, divides L or equals L */
  int32_t rank;               /* r in 0..COBS_MAX_RANK; 0 = first-order (mean-pool) score */
  int32_t sub_dim;            /* 0 = full-space descriptor (Ds = D); else Ds in [8, D], u_q required */
  int32_t topk;               /* k in 1..COBS_MAX_TOPK */
  int32_t window;             /* local window in tokens, >= 1 */
  int32_t summary_dtype;      /* cobs_summary_dtype */
  int32_t scale_dtype;        /* cobs_scale_dtype; read only when summary_dtype == COBS_SUMM_FP4_E2M1 */
  int32_t max_blocks;         /* NB: block capacity per sequence = stride of the summary arrays; <= COBS_MAX_BLOCKS */
  int32_t max_pages_per_seq;  /* row stride of page_table; max_pages_per_seq * P >= NB * L */
} cobs_config;

/* Paged bf16 KV cache. */
typedef struct {
  const void *k_pages;        /* [n_pages][Hkv][P][D] bf16 */
  const void *v_pages;        /* [n_pages][Hkv][P][D] bf16 */
  const int32_t *page_table;  /* [B][max_pages_per_seq]: page id of the i-th page of a sequence */
  const int32_t *seq_lens;    /* [B]: tokens in the cache, the current one included; 1 <= T <= min(NB*L + L - 1,
                                 max_pages_per_seq * P).  Tokens beyond the page-table row are not read: they are
                                 skipped and COBS_ERR_BOUNDS is left in the status word */
  int64_t n_pages;            /* page ids are checked against this */
} cobs_kv;

/*
 * Per-block summaries (paper: Method, second-order truncation, covariance compression, subspace
 * method, quantization).  Layout per (sequence, KV head, block):
 *   mean   [B][Hkv][NB][D]                fp32 (COBS_SUMM_FP32) or bf16 (BF16 and FP4 modes)
 *   xi     [B][Hkv][NB][r][Ds]            fp32 | bf16, or for FP4 [B][Hkv][NB][r * Ds_pad / 2] bytes:
 *                                         E2M1 codes (bit 3 sign, bits 2..0 magnitude index into
 *                                         {0, .5, 1, 1.5, 2, 3, 4, 6}), element 2j of a row in the low
 *                                         nibble of byte j, element 2j+1 in the high nibble; rows are
 *                                         Ds_pad = cobs_padded_sub_dim() elements long, padding codes 0
 *   scale  [B][Hkv][NB][r]                fp32 | fp16, FP4 mode only: xi_hat = magnitude * scale
 *   u_q    [Hkv][D][Ds] fp32              orthonormal columns spanning the query subspace; NULL when
 *                                         sub_dim == 0
 */
typedef struct {
  void *mean;
  void *xi;
  void *scale;
  const float *u_q;
  float *skew;                /* NULL, or [B][Hkv][NB][r] fp32: the diagonal-skew variant (see below) */
} cobs_summaries;

/*
 * Diagonal-skew variant (paper: Appendix, "Cheap diagonal skew"; it reports that the term hurts at r <= 8 and stops
 * at the covariance, so this is off unless `skew` is given).  One scalar per stored factor xi_i = sqrt(lam_i) u_i,
 *   c_i = g_i / lam_i^(3/2),   g_i = 1/L sum_{t in b} (u_i . (k_t - kbar))^3   (0 for a null factor),
 * adds 1/6 sum_i c_i (xi_i . q')^3 (= 1/6 sum_i (u_i . q')^3 g_i) to the block's log-mass estimate.
 * With skew != NULL: cobs_build_summaries writes the scalars (from the unrounded factors), cobs_score_select and
 * cobs_decode_step add the term; scoring then runs in the generic kernels, not in the one-launch step.  Full-space
 * descriptors only (sub_dim == 0), rank >= 1: otherwise COBS_ERR_UNSUPPORTED.
 */

const char *cobs_status_string(int32_t status);

/* Row length in elements of a packed FP4 factor row: Ds rounded up to a multiple of 32 codes, so that
 * every row is a whole number of 16-byte units and starts on a 16-byte boundary. */
int32_t cobs_padded_sub_dim(const cobs_config *cfg);

/* Bytes of each summary array for cfg (scale_bytes = 0 unless FP4).  Host-only arithmetic. */
int32_t cobs_summary_bytes(const cobs_config *cfg, size_t *mean_bytes, size_t *xi_bytes, size_t *scale_bytes);

/* Bytes of workspace that any entry point needs for cfg. */
int32_t cobs_workspace_bytes(const cobs_config *cfg, size_t *bytes);

/* Zero the status word of a workspace (enqueued on stream).  Call once after allocating it. */
int32_t cobs_reset_status(void *workspace, size_t workspace_bytes, void *stream);

/* Synchronise `stream`, copy the status word to *code_host (COBS_OK, COBS_ERR_TIMEOUT or COBS_ERR_BOUNDS). */
int32_t cobs_read_status(void *workspace, size_t workspace_bytes, void *stream, int32_t *code_host);

/*
 * (a) Build the summaries of blocks [block_begin, block_end) of every sequence and KV head; per
 * sequence the range is clipped to the full blocks, floor(T / L).
 *   mean   = (1/L) sum_t k_t                         (Eq. cgf-cumulants)
 *   K~     = rows k_t - mean (un-rounded mean), times U_Q when sub_dim > 0
 *   C      = K~ K~^T / L, eigenpairs (lambda_i, w_i), lambda descending
 *   xi_i   = K~^T w_i / sqrt(L), i < r                (Method, Cost: Gram trick; Eq. lowrank)
 *            sign: the entry of largest magnitude is positive; a direction whose eigenvalue is below
 *            1e-12 of the block's mean squared key norm is stored as zeros
 *   store  : fp32 / bf16 (round to nearest even) / FP4 as cobs_quantise_xi does
 * Arithmetic is fp32.  Deterministic: the same input gives the same bits.
 */
int32_t cobs_build_summaries(const cobs_config *cfg, const cobs_kv *kv, int32_t block_begin, int32_t block_end,
                             const cobs_summaries *out, void *workspace, size_t workspace_bytes, void *stream);

/*
 * The step before the decode step: write the new token's key and value rows (k_new, v_new: [batch][n_kv_heads][D]
 * bf16, 16-byte aligned) at position seq_lens[b] of every sequence's paged cache and add one to seq_lens[b]
 * (Method, Cost: a block's summary is built when the block fills, so the caller then rebuilds block
 * seq_len / L - 1 with cobs_build_summaries whenever the new length is a multiple of L).  A sequence whose page
 * table has no room for the position, or names a page outside [0, n_pages), leaves COBS_ERR_BOUNDS in the status
 * word and is not touched.  Uses the first batch * 4 bytes of the workspace's staging area for a snapshot of the
 * lengths.
 */
int32_t cobs_append_token(const cobs_config *cfg, const void *k_new, const void *v_new, void *k_pages, void *v_pages,
                          const int32_t *page_table, int32_t *seq_lens, int64_t n_pages, void *workspace,
                          size_t workspace_bytes, void *stream);

/*
 * The FP4 quantiser of step (a) on its own (Method, Quantization: E2M1, one scale per eigenvector).
 * xi_fp32 [n_vectors][Ds] -> codes [n_vectors][Ds_pad / 2] bytes, scale [n_vectors] (cfg->scale_dtype).
 *   a = max |xi_j|; scale = a / 6 (fp32 division; rounded to fp16 when the scale is fp16);
 *   t_j = xi_j / scale (fp32 division); code = sign bit of xi_j, nearest E2M1 magnitude to |t_j|,
 *   ties to the even mantissa bit, saturating at 6; scale 0 -> all codes 0.
 * Reads cfg->head_dim, sub_dim, rank, scale_dtype only.  n_vectors must be a multiple of cfg->rank.
 */
int32_t cobs_quantise_xi(const cobs_config *cfg, const float *xi_fp32, int64_t n_vectors, void *codes, void *scale,
                         void *stream);

/*
 * Test hook for the E2M1 rounding rule (Method, Quantization names the format; the rounding is the format's
 * round-to-nearest-even): codes[i] = the code the GPU's own conversion instruction (cvt.rn.satfinite.e2m1x2.f32)
 * gives x[i], one byte per value (bit 3 sign, bits 2..0 magnitude index).  x device fp32 [n], codes device bytes
 * [n]; n <= 2^31.  cobs_quantise_xi does not use that instruction (it must divide by the scale in fp32 and keep
 * the sign of a value that rounds to zero, both by its own rule); the parity tests compare the two on a dense grid.
 * Nothing on the decode path calls this.
 */
int32_t cobs_hw_e2m1_codes(const float *x, int64_t n, uint8_t *codes, void *stream);

/*
 * (b) + (c) Score every summarised block and select (Eq. trunc, Eq. gram, Eq. gqa-secondorder).
 *   q' = q / sqrt(D);  q~ = U_Q^T q' (or q')
 *   e[g][b]  = ln L + q'_g . mean_b + 1/2 sum_i (xi_{b,i} . q~_g)^2
 *   score[b] = sum_g exp(e[g][b] - logsumexp_b' e[g][b'])       over all summarised blocks b'
 * q        [B][Hq][D] bf16
 * sel_idx  [B][Hkv][topk] int32 out, ascending, padded with -1
 * sel_cnt  [B][Hkv] int32 out
 * scores_or_null [B][Hkv][NB] fp32 out (entries b >= floor(T/L) are left untouched)
 */
int32_t cobs_score_select(const cobs_config *cfg, const void *q, const cobs_summaries *summ, const int32_t *seq_lens,
                          int32_t *sel_idx, int32_t *sel_cnt, float *scores_or_null, void *workspace,
                          size_t workspace_bytes, void *stream);

/*
 * The exact-mass selector (the paper's oracle sparse attention, OSA; Eq. bg-defs, Eq. prop-gqa): as
 * cobs_score_select, but every full block's log mass is the direct sum over its keys,
 *   e[g][b] = ln sum_{t in b} exp(q'_g . k_t),
 * instead of the second-order estimate from the summaries.  Same group score, candidates, tie rule and outputs.
 * It reads every key of the cache (the work the estimator avoids): a quality reference, not a step of the
 * decode path.  Reads cfg's shapes, block_size, page_size, topk, window, max_blocks only.
 */
int32_t cobs_exact_select(const cobs_config *cfg, const void *q, const cobs_kv *kv, int32_t *sel_idx, int32_t *sel_cnt,
                          float *scores_or_null, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Adaptive number of selected blocks: an EXTENSION, not in the paper (which always keeps topk blocks).  It applies
 * the paper's dropped mass tau (the normalised block mass outside the kept set; Background, before Eq. prop-gqa) to
 * the group score of Eq. prop-gqa: per (sequence, KV head),
 *   k_adapt = the smallest k such that the k largest candidate scores hold at least (1 - tau) of the candidates'
 *             total score, clamped to [k_min, topk] and to the number of candidates.
 * Trims, in place, a selection made by cobs_score_select (or cobs_exact_select) with the same cfg:
 *   scores    device, fp32 [batch][n_kv_heads][max_blocks]: the scores that call wrote (read only);
 *   seq_lens  device, int32 [batch];
 *   tau       in [0, 1); k_min >= 0;
 *   sel_idx   device, int32 [batch][n_kv_heads][topk]: in, the topk best candidates in ascending index order;
 *             out, the k_adapt best of them in ascending index order, the rest -1 (ties: lower index first);
 *   sel_cnt   device, int32 [batch][n_kv_heads]: in, the entries in use; out, k_adapt.
 * The result feeds cobs_sparse_decode, which reads sel_cnt entries per unit.  Sums are taken in double precision
 * in a fixed order.  topk > 128: COBS_ERR_UNSUPPORTED.  An index outside the candidates is skipped and leaves
 * COBS_ERR_BOUNDS in the status word.  The caller owns every buffer; the call is asynchronous on `stream`.
 */
int32_t cobs_adaptive_trim(const cobs_config *cfg, const float *scores, const int32_t *seq_lens, float tau,
                           int32_t k_min, int32_t *sel_idx, int32_t *sel_cnt, void *workspace, size_t workspace_bytes,
                           void *stream);

/*
 * (d) Attention over the selected blocks and the window, one softmax over their union
 * (Eq. oracle-true restricted to the kept blocks and the window).
 * out [B][Hq][D] fp32; lse_or_null [B][Hq] fp32 = log of the softmax denominator (natural log).
 * sel_idx entries must be distinct candidate blocks in [0, ws/L); others are skipped and reported
 * as COBS_ERR_BOUNDS in the status word.
 */
int32_t cobs_sparse_decode(const cobs_config *cfg, const void *q, const cobs_kv *kv, const int32_t *sel_idx,
                           const int32_t *sel_cnt, float *out, float *lse_or_null, void *workspace,
                           size_t workspace_bytes, void *stream);

/*
 * Fused step: cobs_score_select followed by cobs_sparse_decode on its selection.
 * sel_idx_or_null / sel_cnt_or_null receive the selection when given.
 */
int32_t cobs_decode_step(const cobs_config *cfg, const void *q, const cobs_kv *kv, const cobs_summaries *summ,
                         float *out, float *lse_or_null, int32_t *sel_idx_or_null, int32_t *sel_cnt_or_null,
                         void *workspace, size_t workspace_bytes, void *stream);

/*
 * The fused step for a caller whose per-step tensors live in HOST memory: copies q_host to the device,
 * runs cobs_decode_step, copies the output back and synchronises `stream`.  The KV cache, page table and
 * summaries stay on the device (they are the state a decode loop keeps there).  q_host [B][Hq][D] bf16 and
 * out_host [B][Hq][D] fp32 should be pinned for the copies to be asynchronous; when out_host is pinned memory that
 * is mapped into the device's address space (cudaHostAlloc / cudaHostRegister under unified addressing) and 16-byte
 * aligned, the kernel writes the output rows straight into it and no device-to-host copy is made (measured: 10 us
 * less per step); other host memory goes through a staging buffer in the workspace.  sel_idx_host_or_null
 * [B][Hkv][topk] and sel_cnt_host_or_null [B][Hkv] receive the selection when given.  On return the stream has been
 * synchronised and out_host holds the result.
 */
int32_t cobs_decode_step_host(const cobs_config *cfg, const void *q_host, const cobs_kv *kv,
                              const cobs_summaries *summ, float *out_host, int32_t *sel_idx_host_or_null,
                              int32_t *sel_cnt_host_or_null, void *workspace, size_t workspace_bytes, void *stream);

/*
 * cobs_sparse_decode for callers that cannot provide a workspace.  (The paper has no counterpart: this is
 * a packaging variant of step (d), same arithmetic and same results as cobs_sparse_decode.)
 *
 * Who needs it: code that runs where device allocation is off limits - a decode loop inside a serving
 * process whose memory pool belongs to another component and is fully handed out, a latency-critical
 * path where cudaMalloc's device-wide synchronisation is not acceptable, a plug-in that receives only
 * its input and output tensors.  Such a caller has nowhere to get the split-KV scratch from, so this
 * variant keeps the scratch (status word, per-unit counters, split partials) in a fixed device array
 * inside the library: COBS_STATIC_SCRATCH_BYTES per GPU, held from the moment the library is loaded on
 * that GPU until the process exits.  The call allocates nothing and frees nothing.
 *
 * Limits and rules:
 *   - the configuration's scratch need, 256 + 12 * B * Hkv (rounded up to 256) + B * Hkv * slices * G *
 *     (D + 2) * 4 bytes, must fit COBS_STATIC_SCRATCH_BYTES, else COBS_ERR_WORKSPACE_TOO_SMALL is
 *     returned and nothing is launched (the benchmark's 16 x 8 units at G = 4, D = 128 need 2.4 MB);
 *   - the first call on a device looks up the array's device address (a one-off set-up step); make that
 *     first call outside any stream capture;
 *   - all calls on a device share the one array and it keeps the previous call's contents: the call
 *     itself clears the status word and the counters on `stream` before launching, but two calls that
 *     may overlap on the GPU (different streams, no dependency) race on it - serialise them;
 *   - device-side problems are not reported through a status word the caller can read here: an
 *     out-of-range selection entry or page id is skipped, as in cobs_sparse_decode.
 * Arguments as for cobs_sparse_decode.
 */
#define COBS_STATIC_SCRATCH_BYTES (4 * 1024 * 1024)
int32_t cobs_sparse_decode_static(const cobs_config *cfg, const void *q, const cobs_kv *kv, const int32_t *sel_idx,
                                  const int32_t *sel_cnt, float *out, float *lse_or_null, void *stream);

/* Number of kernels this library has launched in this process so far (host-side counter; the paper
 * has no counterpart: it exists so that a benchmark can state how many launches a timed region held). */
int64_t cobs_kernel_launches(void);

/* Number of those launches whose scoring phase ran on the tcgen05 path (opt-in: environment variable
 * COBS_SCORE_PATH=tcgen05, read at every call; packed E2M1 summaries in the full key space with head_dim 128,
 * rank 8, max_blocks a multiple of 32; any other configuration, or a grid whose CTAs would meet more units than
 * the kernel keeps query operands for, silently takes the default path).  Same results as the default path to
 * rounding; lets a test state which path it exercised.  The paper has no counterpart. */
int64_t cobs_tcgen05_launches(void);

#ifdef __cplusplus
}
#endif
#endif /* COBS_H_ */
