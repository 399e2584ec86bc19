/*
 * pact.h - C ABI of the PACT visual-token reduction library for NVIDIA B200 (sm_100a).
 *
 * The library implements, on one GPU, the per-request reduction step of
 *   "PACT: Pruning and Clustering-Based Token Reduction for Faster Visual Language Models":
 * importance scoring and pruning (EUTI, Algorithm 1), Distance Bounded Density Peak
 * Clustering of the surviving keys (DBDPC, Algorithm 2), reincorporation of pruned tokens
 * that lie close to a centre (Eq. 8-9) and the merge of every cluster into one hidden state
 * that carries its centre's position id (Eq. 10, Algorithm 3).
 *
 * Conventions that hold for every call
 * ------------------------------------
 *  - All data pointers are DEVICE pointers unless a comment says "host".  The caller owns
 *    every buffer, including the workspace; the library never allocates or frees device
 *    memory inside a stage call and never keeps a pointer after the call returns.
 *  - Work is enqueued on `stream` (a cudaStream_t passed as void*) and the call returns
 *    without synchronising.  Counts that depend on the data (q, C, r ...) stay on the device.
 *  - Matrices are row-major; a leading dimension `ld*` is the row stride in ELEMENTS.
 *    Rows must be 16-byte aligned (base pointer and ld * sizeof(element) multiples of 16).
 *  - Element type of H, K, Q is `in` given to pact_create (bf16 or fp32); H_out has type `out`.
 *  - Every call returns a pact_status.  Host-detectable errors (null pointer, bad size or
 *    alignment, workspace too small, parameter out of range) are reported before anything
 *    is launched.  Device-side problems (a bounded wait that ran out) set counters[PACT_CNT_STATUS]
 *    of the image; the library never traps, aborts or throws.
 *  - A context may be used from one host thread and one stream at a time.
 *  - Same inputs give bitwise the same outputs, run after run.
 *
 * Readings of the paper that fix the semantics (the paper is silent on them)
 * ------------------------------------------------------------------------
 *  - Softmax in Eq. 2 runs across the visual tokens, separately per head, without 1/sqrt(d_h).
 *  - Query head j reads key head floor(j * n_kvh / n_qh); the mean over heads uses n_qh.
 *  - Percentile(s, lambda): with m = min(floor(lambda*N + 1e-6), N-1) and tau the (m+1)-th
 *    smallest score, a token is important iff s_i >= tau (Eq. 3) - ties at tau are kept.
 *  - The clustering vector of a token is the concatenation of its key heads (width d_k).
 *  - Distances are clamped to [0, 2]; d_ii = 0; a key whose norm vanishes (below about 1e-19)
 *    is at distance 1 from every other key.
 *  - Density ties go to the lower token index; a vector becomes a centre iff its distance to
 *    every earlier centre is strictly greater than d_c; argmin ties go to the lower cluster id.
 *  - Cluster ids number the centres by ascending token index; merged rows are emitted in
 *    that order in place of the visual span; text rows keep their relative place.
 *  - A pruned token rejoins iff its nearest-centre distance is strictly below
 *    (float)alpha * (float)d_c.
 */
#ifndef PACT_H_
#define PACT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct pact_ctx pact_ctx; /* opaque; holds shapes and device properties, no device memory */

typedef enum { PACT_BF16 = 0, PACT_F32 = 1 } pact_dtype;

typedef enum {
  PACT_OK = 0,
  PACT_ERR_INVALID_ARG = -1, /* null pointer, bad size, stride or alignment, parameter out of range */
  PACT_ERR_UNSUPPORTED = -2, /* shape, dtype or device the library has no kernel for            */
  PACT_ERR_WORKSPACE = -3,   /* workspace pointer null, misaligned or too small                 */
  PACT_ERR_CUDA = -4,        /* a CUDA runtime call failed (see pact_last_cuda_error)           */
  PACT_ERR_TIMEOUT = -5      /* value of counters[PACT_CNT_STATUS] when a bounded device wait ran out */
} pact_status;

/* Slots of the per-image int32 counters array (device memory, 16 entries). */
enum {
  PACT_CNT_N_OUT = 0,     /* rows of H_out / P_out / size_out that are valid                   */
  PACT_CNT_Q = 1,         /* important (surviving) tokens, |S_important|                        */
  PACT_CNT_C = 2,         /* clusters                                                           */
  PACT_CNT_R = 3,         /* pruned tokens that rejoined a cluster                              */
  PACT_CNT_DISCARDED = 4, /* pruned tokens that did not                                         */
  PACT_CNT_SWEEPS = 5,    /* largest number of passes any row needed in the centre selection    */
  PACT_CNT_BAND_DC = 6,   /* unordered surviving pairs with |d - d_c| <= 1e-6                   */
  PACT_CNT_BAND_ADC = 7,  /* pruned tokens whose nearest-centre distance is within 1e-6 of alpha*d_c */
  PACT_CNT_STATUS = 8,    /* 0, or a negative pact_status raised on the device                  */
  PACT_CNT_M = 9,         /* pruned tokens, |S_unimportant|                                     */
  PACT_N_COUNTERS = 16
};

/* Flags of pact_params.flags (ablations of Sec. 4 of the paper). */
enum {
  PACT_FLAG_CENTER_ONLY = 1u, /* h'_s = h_s: the centre represents its cluster, no averaging     */
  PACT_FLAG_NO_NORM = 2u,     /* Eq. 2 without the hidden-state norm factor                      */
  PACT_FLAG_NORM_ONLY = 4u    /* Eq. 2 without the global-query factor: s_i = |h_i| / N          */
};

/* Hyper-parameters of Algorithm 3. */
typedef struct {
  double lambda;        /* pruning fraction in [0, 1]                                            */
  float d_c;            /* cutoff, cosine distance, in [0, 2]                                    */
  float d_n;            /* density normaliser of Eq. 6, > 0 (the paper uses 2)                   */
  float alpha;          /* reincorporation tolerance of Eq. 8, >= 0 (the paper uses 1.5); 0 = off */
  int32_t n_prune;      /* >= 0: use this m instead of the one derived from lambda               */
  uint32_t flags;       /* PACT_FLAG_*                                                           */
} pact_params;

/* One independent unit: an image or a video clip inside a sequence of n_total tokens. */
typedef struct {
  const void *H;        /* [n_total, d] hidden states at layer L                                 */
  int64_t ldH;
  const void *K_euti;   /* [N, n_kvh*d_h] keys BEFORE rotary embedding, visual rows only         */
  int64_t ldKe;
  const void *Q_euti;   /* [N, n_qh*d_h] queries BEFORE rotary embedding, visual rows only       */
  int64_t ldQ;
  const void *K_clu;    /* [N, n_kvh*d_h] keys AFTER rotary embedding; may alias K_euti          */
  int64_t ldKc;
  const int32_t *P;     /* [n_total] position ids                                                */
  int32_t n_total;      /* tokens in the sequence (text + visual)                                */
  int32_t vis_start;    /* the visual tokens are rows [vis_start, vis_start + N) of H and P      */
  int32_t N;            /* number of visual tokens, >= 1                                         */
  int32_t reserved;
  void *H_out;          /* [n_total, d] capacity; the first counters[N_OUT] rows are valid        */
  int64_t ldHo;
  int32_t *P_out;       /* [n_total] capacity                                                     */
  int32_t *size_out;    /* [n_total] capacity: cluster size (W of Eq. 11); 1 for text rows        */
  int32_t *label;       /* [N] cluster id of every visual token, -1 = discarded; may be NULL      */
  float *score;         /* [N] EUTI scores; may be NULL                                           */
  uint8_t *keep;        /* [N] 1 = important (survived pruning), 0 = pruned; may be NULL          */
  int32_t *counters;    /* [PACT_N_COUNTERS]                                                      */
  float *logw_out;      /* [n_total] capacity: log(size_out), the additive attention bias log W of
                           Eq. 11 for the reduced sequence (0 for text rows); may be NULL           */
} pact_image;

/* ---- context --------------------------------------------------------------------------- */

/* Creates a context for hidden size d, n_qh query heads, n_kvh key heads of width d_h, on the
 * current CUDA device.  Requirements: d_h * n_kvh and d_h * n_qh and d multiples of 8 (bf16) or
 * 4 (fp32); n_qh a multiple of n_kvh; `out` is the element type of H_out. */
pact_status pact_create(pact_ctx **ctx, int d, int n_qh, int n_kvh, int d_h, pact_dtype in,
                        pact_dtype out);
pact_status pact_destroy(pact_ctx *ctx);

/* Bytes of device workspace needed for calls with at most max_batch images of at most max_N
 * visual tokens each.  The workspace must be 256-byte aligned.  Its contents need not be
 * preserved between calls and need no initialisation. */
size_t pact_workspace_bytes(const pact_ctx *ctx, int max_batch, int max_N);

const char *pact_status_string(pact_status s);
/* Text of the last CUDA runtime error seen by this context ("" if none). */
const char *pact_last_cuda_error(const pact_ctx *ctx);

/* Bounds of the device-side waits (Algorithm 2's centre selection is resolved in sweeps over two bit masks,
 * and the member lists of Eq. 10 are built behind one barrier between CTAs).  When a bound is reached the
 * kernel stops waiting, writes PACT_ERR_TIMEOUT to counters[PACT_CNT_STATUS] of the image and carries on
 * within bounds; the call itself still returns PACT_OK and the outputs of that image are not valid.
 * barrier_polls: polls of the member-list barrier; center_sweeps: sweeps of the centre selection;
 * 0 restores the default (about a million).  Graphs recorded earlier keep the limits they were recorded with. */
pact_status pact_set_wait_limits(pact_ctx *ctx, int barrier_polls, int center_sweeps);

/* ---- instrumentation ---------------------------------------------------------------------- */

/* Number of kernels this context has launched since it was created. */
long long pact_launch_count(const pact_ctx *ctx);
/* With profiling on, pact_reduce records a CUDA event on `stream` after each of its kernels
 * (first parameter block of a call only).  pact_profile_read waits for the last one and writes
 * the duration of each kernel in milliseconds to ms[0..n), returning n (0 if nothing was
 * recorded).  pact_profile_stage_name(i) names the i-th kernel.  Off by default. */
pact_status pact_profile_enable(pact_ctx *ctx, int on);
int pact_profile_read(pact_ctx *ctx, float *ms /*host*/, int cap);
const char *pact_profile_stage_name(int i);

/* ---- stage calls (one image) ----------------------------------------------------------- */

/* EUTI score, Eq. 1-2 / Algorithm 1 steps 1-2.
 * Reads img->H (visual rows), K_euti, Q_euti; writes score[N] (fp32). */
pact_status pact_importance(pact_ctx *ctx, const pact_image *img /*host*/, const pact_params *p /*host*/,
                            float *score, void *ws, size_t ws_bytes, void *stream);

/* Percentile split, Eq. 3-4 / Algorithm 1 step 3.
 * score[N] -> keep[N] (1 = important), kept_idx[q] and pruned_idx[m] in ascending order
 * (capacity N each), counts[0] = q, counts[1] = m (device int32[2]). */
pact_status pact_prune(pact_ctx *ctx, const float *score, int N, const pact_params *p /*host*/,
                       uint8_t *keep, int32_t *kept_idx, int32_t *pruned_idx, int32_t *counts,
                       void *ws, size_t ws_bytes, void *stream);

/* The same split for callers that cannot allocate device memory (no counterpart in the paper:
 * this is a packaging variant of pact_prune, not a step of the method).  pact_prune needs a
 * workspace that somebody obtained from cudaMalloc; a host that runs inside another framework's
 * callback, a plugin that is handed tensors but no allocator, or a process whose device memory is
 * already fully parcelled out cannot provide one.  This entry point takes no context and no
 * workspace: its scratch is a fixed array inside the library image (about 256 KiB, resident on
 * every GPU that loads the library until the process exits), and it calls no allocating routine.
 *  - N must not exceed PACT_PRUNE_STATIC_MAX_N; larger N returns PACT_ERR_UNSUPPORTED and launches
 *    nothing.  Only p->lambda and p->n_prune are read.
 *  - The first call on each device looks up the array's device address (with that device
 *    current); make that first call outside any stream capture.
 *  - All calls on a device share the one array: two calls whose kernels may overlap on the GPU
 *    (different streams without an ordering between them) race.  Calls on one stream are safe.
 * Inputs, outputs and their meaning are those of pact_prune. */
#define PACT_PRUNE_STATIC_MAX_N 65536
pact_status pact_prune_static(const float *score, int N, const pact_params *p /*host*/, uint8_t *keep,
                              int32_t *kept_idx, int32_t *pruned_idx, int32_t *counts, void *stream);

/* DBDPC, Algorithm 2 (Eq. 5-7) on the rows idx[0..q) of K[N, d_k]:
 * all-pairs cosine distance, density with d_n, density-ordered centre selection under d_c
 * (the result of the sequential loop, computed by asynchronous parallel resolution, cf.
 * Algorithm 4 / Appendix D), nearest-centre assignment.
 * idx must be ascending; q is read from q_dev (device int32).
 * Writes rho[q] (in idx order), center_idx[C] (token indices, ascending), C_dev,
 * label[N] (cluster id for rows in idx, -1 elsewhere), and counters (may be NULL). */
pact_status pact_dbdpc(pact_ctx *ctx, const void *K, int64_t ldK, int N, const int32_t *idx,
                       const int32_t *q_dev, const pact_params *p /*host*/, float *rho,
                       int32_t *center_idx, int32_t *C_dev, int32_t *label, int32_t *counters,
                       void *ws, size_t ws_bytes, void *stream);

/* Reincorporation, Eq. 8-9 / Algorithm 3 step 3: each row pruned_idx[0..m) of K joins its
 * nearest centre iff that distance is < alpha * d_c.  Updates label[N] in place for those rows
 * (cluster id or -1) and writes r_dev (number that joined).  counters may be NULL. */
pact_status pact_reincorporate(pact_ctx *ctx, const void *K, int64_t ldK, int N,
                               const int32_t *pruned_idx, const int32_t *m_dev,
                               const int32_t *center_idx, const int32_t *C_dev,
                               const pact_params *p /*host*/, int32_t *label, int32_t *r_dev,
                               int32_t *counters, void *ws, size_t ws_bytes, void *stream);

/* Choice of the reduction layer L (the paragraph that follows Eq. 11 and the figure it cites): the
 * earliest layer whose visual keys are spread widely enough.  K_layers is a HOST array of n_layers
 * DEVICE pointers, each a [N, n_kvh*d_h] key matrix with row stride ldK elements (keys before the
 * rotary embedding, as in that figure).  For every layer l, max_dist[l] (device, [n_layers]) receives
 * the largest cosine distance (Eq. 5) between two of its N keys, 0 when N = 1; layer_out (device,
 * [1], may be NULL) receives the smallest l with max_dist[l] >= threshold, or -1 when no layer
 * qualifies.  Distances are formed in the arithmetic of pact_dbdpc (fp32 for bf16 keys, fp64 rounded
 * to fp32 for fp32 keys).  ws must hold pact_workspace_bytes(ctx, min(n_layers, 16), N) bytes.
 * Asynchronous on `stream`; INVALID_ARG for null or misaligned pointers, n_layers < 1, N < 1, a bad
 * stride or a NaN threshold, before anything is launched. */
pact_status pact_key_spread(pact_ctx *ctx, const void *const *K_layers /*host*/, int n_layers, int64_t ldK,
                            int N, float threshold, float *max_dist, int32_t *layer_out, void *ws,
                            size_t ws_bytes, void *stream);

/* Merge, Eq. 10 / Algorithm 3 step 4: H_out row (vis_start + c) = mean of the visual rows of H
 * whose label is c (fp32 accumulation in ascending token order), P_out = position id of the
 * centre, size_out = members, logw_out = log(members) when given (the bias log W that Eq. 11
 * adds to the attention logits of the reduced sequence; 0 for text rows); text rows are copied
 * around the merged span.
 * Uses img->H, P, H_out, P_out, size_out, logw_out, counters (N_OUT and STATUS are written, the rest is zero).
 * label[i] must lie in [-1, C) and *C_dev in [0, N]; center_idx[c] in [0, N).  A label outside that
 * range is treated as -1 and reported as PACT_ERR_INVALID_ARG in counters[PACT_CNT_STATUS]; the other
 * rows are merged as usual. */
pact_status pact_merge(pact_ctx *ctx, const pact_image *img /*host*/, const int32_t *label,
                       const int32_t *center_idx, const int32_t *C_dev, const pact_params *p /*host*/,
                       void *ws, size_t ws_bytes, void *stream);

/* ---- the whole step over a batch (Algorithm 3) ------------------------------------------ */

/* imgs: host array of B images (independent units).  params: one pact_params for all
 * (params_stride = 0) or one per image (params_stride = 1).  All outputs named in pact_image
 * are written; nothing is read back to the host. */
pact_status pact_reduce(pact_ctx *ctx, const pact_image *imgs /*host*/, int B,
                        const pact_params *params /*host*/, int params_stride, void *ws,
                        size_t ws_bytes, void *stream);

/* ---- replayable form of pact_reduce (CUDA graph) --------------------------------------------- */

/* Records the launch sequence of pact_reduce(ctx, imgs, B, params, params_stride, ws, ws_bytes) once
 * into a CUDA graph; pact_graph_launch replays it on `stream` at a fraction of the launch cost (the
 * path is a chain of short dependent kernels, so launch gaps matter).  The graph holds the pointers
 * given here: the buffers and the workspace must stay valid and in place while it is used; their
 * contents may change between launches.  One launch at a time per graph (they share the workspace).
 * Nothing runs on the device during pact_graph_create. */
typedef struct pact_graph pact_graph;
pact_status pact_graph_create(pact_ctx *ctx, const pact_image *imgs /*host*/, int B,
                              const pact_params *params /*host*/, int params_stride, void *ws,
                              size_t ws_bytes, pact_graph **graph);
pact_status pact_graph_launch(pact_graph *graph, void *stream);
pact_status pact_graph_destroy(pact_graph *graph);

/* Same computation with HOST buffers for one image: copies the inputs to the device, runs
 * pact_reduce, copies H_out/P_out/size_out/label/counters back and synchronises.
 * dev_in / dev_out are device staging buffers the caller provides (sizes from
 * pact_host_staging_bytes); every pointer inside `img` is a host pointer here. */
pact_status pact_reduce_host(pact_ctx *ctx, const pact_image *img /*host, host pointers*/,
                             const pact_params *p /*host*/, void *dev_staging, size_t staging_bytes,
                             void *ws, size_t ws_bytes, void *stream);
size_t pact_host_staging_bytes(const pact_ctx *ctx, int n_total, int N);

#ifdef __cplusplus
}
#endif
#endif /* PACT_H_ */
