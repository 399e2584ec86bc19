// Host side of the C ABI: argument checks, workspace layout, launch sequences.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <new>

#include "kernels.cuh"

using namespace pact;

constexpr int kProfStages = 9;

struct pact_ctx {
  int d, n_qh, n_kvh, d_h, d_k, n_qcols;
  pact_dtype in, out;
  int elt;                 // bytes per input element
  ClusterCfg ccfg;
  bool umma;               // bf16 keys of a width the tcgen05 tile kernels take
  int device;
  char err[256];
  long long launches;      // kernels launched by this context so far
  int spin_limit;          // polls the barrier of the member-list kernel makes before it raises PACT_ERR_TIMEOUT
  int sweep_limit;         // sweeps the centre selection makes before it raises PACT_ERR_TIMEOUT
  int prof_on;             // record an event after every stage of pact_reduce
  int prof_n;              // stages recorded by the last profiled call
  cudaEvent_t ev[kProfStages + 1];
};

struct pact_graph {
  pact_ctx *ctx;
  cudaGraphExec_t exec;
  int kernels;             // kernels one replay launches
};

static const char *const kStageNames[kProfStages] = {"qsum", "tokens", "scores", "select", "gram_density", "centers",
                                                    "assign", "label_lists", "merge"};

namespace {

constexpr size_t kAlign = 256;
inline size_t rup(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Carves the per-image workspace; with base == nullptr only the size is computed.
struct Carver {
  char *base;
  size_t off = 0;
  template <typename P> void take(P *&ptr, size_t bytes) {
    ptr = base ? reinterpret_cast<P *>(base + off) : nullptr;
    off += rup(bytes, kAlign);
  }
};

size_t carve_image(const pact_ctx *c, int N, char *base, ImgDesc *im) {
  ImgDesc tmp;
  ImgDesc &m = im ? *im : tmp;
  Carver cv{base};
  const int Np = (int)rup((size_t)N, 128);
  const int Wp = Np / 32;
  m.Np = Np;
  m.Wp = Wp;
  cv.take(m.cnt, (size_t)(kCntInts + kTickInts) * sizeof(int32_t));
  if (m.cnt) m.tick = m.cnt + kCntInts;
  cv.take(m.qpart, (size_t)kQPartRows * c->n_qcols * sizeof(double));
  cv.take(m.qg, (size_t)c->n_qcols * sizeof(double));
  cv.take(m.E, (size_t)N * c->n_qh * sizeof(double));
  cv.take(m.part, (size_t)((N + kRowsPerCta - 1) / kRowsPerCta) * c->n_qh * 2 * sizeof(double));
  cv.take(m.ghist, ((size_t)1 << kHistBits) * sizeof(int32_t));
  cv.take(m.nrm, (size_t)N * sizeof(double));
  cv.take(m.score, (size_t)N * sizeof(float));
  cv.take(m.keep, (size_t)N);
  cv.take(m.slot, (size_t)N * sizeof(int32_t));
  cv.take(m.kept_idx, (size_t)N * sizeof(int32_t));
  cv.take(m.pruned_idx, (size_t)N * sizeof(int32_t));
  cv.take(m.rn, (size_t)N * sizeof(float));
  cv.take(m.rn64, (size_t)N * sizeof(double));
  cv.take(m.Kp, (size_t)Np * c->d_k * c->elt);
  cv.take(m.rnk, (size_t)Np * sizeof(float));
  cv.take(m.rnk64, (size_t)Np * sizeof(double));
  cv.take(m.rho_fix, (size_t)Np * sizeof(unsigned long long));
  cv.take(m.rho, (size_t)Np * sizeof(float));
  cv.take(m.adj, (size_t)Np * Wp * sizeof(uint32_t));
  cv.take(m.cmask, (size_t)Wp * sizeof(uint32_t));
  cv.take(m.rmask, (size_t)Wp * sizeof(uint32_t));
  cv.take(m.Kcen, (size_t)Np * c->d_k * c->elt);
  cv.take(m.rnc, (size_t)Np * sizeof(float));
  cv.take(m.rnc64, (size_t)Np * sizeof(double));
  cv.take(m.center_idx, (size_t)Np * sizeof(int32_t));
  cv.take(m.cid, (size_t)Np * sizeof(int32_t));
  cv.take(m.best, (size_t)N * sizeof(unsigned long long));
  cv.take(m.label, (size_t)N * sizeof(int32_t));
  const size_t nblk = ((size_t)N + kListBlock - 1) / kListBlock;
  m.nbp = (int)rup(nblk, 8);
  cv.take(m.blocklist, nblk * kListBlock * sizeof(int32_t));
  cv.take(m.cnt_cb, (size_t)Np * m.nbp * sizeof(uint16_t));
  cv.take(m.members, (size_t)N * sizeof(int4));
  cv.take(m.csize, (size_t)Np * sizeof(int32_t));
  cv.take(m.cticket, (size_t)Np * sizeof(int32_t));
  cv.take(m.rtick, (size_t)Wp * sizeof(int32_t));
  // two partial sums per CTA of k_merge (a range boundary cuts at most two clusters)
  cv.take(m.mpart, (size_t)2 * merge_ctas(c->ccfg.sm_count, 1) * c->d * sizeof(float));
  return cv.off;
}

pact_status fail_cuda(pact_ctx *c, cudaError_t e, const char *where) {
  snprintf(c->err, sizeof(c->err), "%s: %s", where, cudaGetErrorString(e));
  return PACT_ERR_CUDA;
}

#define CK(call)                                                     \
  do {                                                               \
    cudaError_t e_ = (call);                                         \
    if (e_ != cudaSuccess) return fail_cuda(ctx, e_, #call);         \
  } while (0)

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool ld_ok(const pact_ctx *c, int64_t ld, int width) {
  return ld >= width && ((size_t)ld * c->elt) % 16 == 0;
}

pact_status check_params(const pact_params *p) {
  if (!p) return PACT_ERR_INVALID_ARG;
  if (!(p->lambda >= 0.0 && p->lambda <= 1.0)) return PACT_ERR_INVALID_ARG;
  if (!(p->d_c >= 0.0f && p->d_c <= 2.0f)) return PACT_ERR_INVALID_ARG;
  if (!(p->d_n > 0.0f) || !(p->alpha >= 0.0f)) return PACT_ERR_INVALID_ARG;
  if ((p->flags & PACT_FLAG_NO_NORM) && (p->flags & PACT_FLAG_NORM_ONLY)) return PACT_ERR_INVALID_ARG;
  return PACT_OK;
}

void set_params(ImgDesc &m, const pact_params *p, int N) {
  long long mt = p->n_prune >= 0 ? (long long)p->n_prune : (long long)floor(p->lambda * (double)N + 1e-6);
  if (mt > N - 1) mt = N - 1;
  if (mt < 0) mt = 0;
  m.m_target = (int)mt;
  m.d_c = p->d_c;
  m.d_c64 = (double)p->d_c;
  m.inv_dn_log2e = (float)(1.4426950408889634 / (double)p->d_n);
  m.inv_dn64 = 1.0 / (double)p->d_n;
  m.t_reinc = p->alpha * p->d_c;            // formed in float, as documented
  m.t_reinc64 = (double)m.t_reinc;
  m.flags = p->flags;
}

void set_dims(const pact_ctx *c, Batch &bt, int B) {
  bt.B = B;
  bt.d = c->d; bt.n_qh = c->n_qh; bt.n_kvh = c->n_kvh; bt.d_h = c->d_h; bt.d_k = c->d_k;
  bt.n_qcols = c->n_qcols;
}

void point_counts_at_workspace(ImgDesc &m) {
  m.q_ptr = m.cnt + PACT_CNT_Q;
  m.m_ptr = m.cnt + PACT_CNT_M;
  m.C_ptr = m.cnt + PACT_CNT_C;
  m.cidx_ptr = m.center_idx;
  m.rho_user = nullptr; m.center_idx_user = nullptr; m.C_user = nullptr; m.r_user = nullptr;
}

pact_status check_ws(const pact_ctx *c, void *ws, size_t ws_bytes, int B, int N) {
  if (!ws || (reinterpret_cast<uintptr_t>(ws) % kAlign) != 0) return PACT_ERR_WORKSPACE;
  if (ws_bytes < pact_workspace_bytes(c, B, N)) return PACT_ERR_WORKSPACE;
  return PACT_OK;
}

pact_status check_image(const pact_ctx *c, const pact_image *g, bool need_euti, bool need_clu, bool need_out) {
  if (!g) return PACT_ERR_INVALID_ARG;
  if (g->N < 1 || g->n_total < g->N || g->vis_start < 0 || g->vis_start + g->N > g->n_total)
    return PACT_ERR_INVALID_ARG;
  if (need_euti) {
    if (!g->H || !g->K_euti || !g->Q_euti) return PACT_ERR_INVALID_ARG;
    if (!aligned16(g->H) || !aligned16(g->K_euti) || !aligned16(g->Q_euti)) return PACT_ERR_INVALID_ARG;
    if (!ld_ok(c, g->ldH, c->d) || !ld_ok(c, g->ldKe, c->d_k) || !ld_ok(c, g->ldQ, c->n_qcols))
      return PACT_ERR_INVALID_ARG;
  }
  if (need_clu) {
    if (!g->K_clu || !aligned16(g->K_clu) || !ld_ok(c, g->ldKc, c->d_k)) return PACT_ERR_INVALID_ARG;
  }
  if (need_out) {
    if (g->N > kMaxTokens) return PACT_ERR_UNSUPPORTED;
    if (!g->H || !aligned16(g->H) || !ld_ok(c, g->ldH, c->d) || !g->P) return PACT_ERR_INVALID_ARG;
    if (!g->H_out || !aligned16(g->H_out) || !g->P_out || !g->size_out || !g->counters)
      return PACT_ERR_INVALID_ARG;
    const size_t oe = c->out == PACT_BF16 ? 2 : 4;
    if (g->ldHo < c->d || ((size_t)g->ldHo * oe) % 16 != 0) return PACT_ERR_INVALID_ARG;
  }
  return PACT_OK;
}

#ifdef PACT_TIMELINE
unsigned long long *g_timeline = nullptr;
#endif

void fill_user(ImgDesc &m, const pact_image *g) {
#ifdef PACT_TIMELINE
  m.tl = g_timeline;
#endif
  m.H = g->H; m.Ke = g->K_euti; m.Q = g->Q_euti; m.Kc = g->K_clu;
  m.ldH = g->ldH; m.ldKe = g->ldKe; m.ldQ = g->ldQ; m.ldKc = g->ldKc; m.ldHo = g->ldHo;
  m.P = g->P; m.H_out = g->H_out; m.P_out = g->P_out; m.size_out = g->size_out; m.logw_out = g->logw_out;
  m.label_user = g->label; m.counters_user = g->counters; m.score_user = g->score;
  m.keep_user = g->keep;
  m.n_total = g->n_total; m.vis_start = g->vis_start; m.N = g->N;
}

}  // namespace

extern "C" {

#ifdef PACT_TIMELINE
// instrumented build only: device buffer of 16 x 4096 x 2 timestamps (zeroed by the caller)
void pact_debug_set_timeline(unsigned long long *buf) { g_timeline = buf; }
#endif

const char *pact_status_string(pact_status s) {
  switch (s) {
    case PACT_OK: return "ok";
    case PACT_ERR_INVALID_ARG: return "invalid argument";
    case PACT_ERR_UNSUPPORTED: return "unsupported shape, dtype or device";
    case PACT_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case PACT_ERR_CUDA: return "CUDA runtime error";
    case PACT_ERR_TIMEOUT: return "a bounded device wait ran out";
  }
  return "unknown status";
}

const char *pact_last_cuda_error(const pact_ctx *ctx) { return ctx ? ctx->err : ""; }

pact_status pact_create(pact_ctx **out, int d, int n_qh, int n_kvh, int d_h, pact_dtype in, pact_dtype o) {
  if (!out) return PACT_ERR_INVALID_ARG;
  *out = nullptr;
  if (d < 8 || n_qh < 1 || n_kvh < 1 || d_h < 1 || n_qh % n_kvh != 0) return PACT_ERR_INVALID_ARG;
  if ((in != PACT_BF16 && in != PACT_F32) || (o != PACT_BF16 && o != PACT_F32)) return PACT_ERR_INVALID_ARG;
  const int v = in == PACT_BF16 ? 8 : 4;
  if (d % 8 != 0 || d_h % v != 0) return PACT_ERR_UNSUPPORTED;
  if (d > kMergeMaxD || n_qh > 256) return PACT_ERR_UNSUPPORTED;
  if ((n_qh * d_h / v + 7) / 8 > kTickInts) return PACT_ERR_UNSUPPORTED;   // one ticket per 128-byte column group of Q
  pact_ctx *c = new (std::nothrow) pact_ctx;
  if (!c) return PACT_ERR_INVALID_ARG;
  memset(c, 0, sizeof(*c));
  c->d = d; c->n_qh = n_qh; c->n_kvh = n_kvh; c->d_h = d_h;
  c->d_k = n_kvh * d_h; c->n_qcols = n_qh * d_h;
  c->in = in; c->out = o; c->elt = in == PACT_BF16 ? 2 : 4;
  pact_ctx *ctx = c;
  cudaError_t e = cudaGetDevice(&c->device);
  if (e == cudaSuccess) {
    cudaDeviceProp pr;
    e = cudaGetDeviceProperties(&pr, c->device);
    if (e == cudaSuccess && pr.major != 10) { delete c; return PACT_ERR_UNSUPPORTED; }
  }
  if (e == cudaSuccess) e = euti_configure(c->n_qcols, c->n_qh);
  if (e == cudaSuccess) e = cluster_configure(&c->ccfg);
  if (e == cudaSuccess) e = merge_configure();
  if (e == cudaSuccess && in == PACT_BF16) e = umma_configure();
  if (e != cudaSuccess) {
    pact_status s = fail_cuda(ctx, e, "pact_create");
    (void)s;
    delete c;
    return PACT_ERR_CUDA;
  }
  c->umma = in == PACT_BF16 && umma_supported(c->d_k);
  c->spin_limit = kSpinLimit;
  c->sweep_limit = kSpinLimit;
  *out = c;
  return PACT_OK;
}

pact_status pact_destroy(pact_ctx *ctx) {
  if (ctx && ctx->prof_on)
    for (int i = 0; i <= kProfStages; ++i) cudaEventDestroy(ctx->ev[i]);
  delete ctx;
  return PACT_OK;
}

long long pact_launch_count(const pact_ctx *ctx) { return ctx ? ctx->launches : 0; }

pact_status pact_set_wait_limits(pact_ctx *ctx, int barrier_polls, int center_sweeps) {
  if (!ctx || barrier_polls < 0 || center_sweeps < 0) return PACT_ERR_INVALID_ARG;
  ctx->spin_limit = barrier_polls ? barrier_polls : kSpinLimit;
  ctx->sweep_limit = center_sweeps ? center_sweeps : kSpinLimit;
  return PACT_OK;
}

pact_status pact_profile_enable(pact_ctx *ctx, int on) {
  if (!ctx) return PACT_ERR_INVALID_ARG;
  if (on && !ctx->prof_on) {
    for (int i = 0; i <= kProfStages; ++i) CK(cudaEventCreate(&ctx->ev[i]));
    ctx->prof_on = 1;
    ctx->prof_n = 0;
  } else if (!on && ctx->prof_on) {
    for (int i = 0; i <= kProfStages; ++i) cudaEventDestroy(ctx->ev[i]);
    ctx->prof_on = 0;
  }
  return PACT_OK;
}

int pact_profile_read(pact_ctx *ctx, float *ms, int cap) {
  if (!ctx || !ms || !ctx->prof_on || ctx->prof_n < 1) return 0;
  if (cudaEventSynchronize(ctx->ev[ctx->prof_n]) != cudaSuccess) return 0;
  int n = ctx->prof_n < cap ? ctx->prof_n : cap;
  for (int i = 0; i < n; ++i)
    if (cudaEventElapsedTime(&ms[i], ctx->ev[i], ctx->ev[i + 1]) != cudaSuccess) return 0;
  return n;
}

const char *pact_profile_stage_name(int i) { return (i >= 0 && i < kProfStages) ? kStageNames[i] : ""; }

size_t pact_workspace_bytes(const pact_ctx *ctx, int max_batch, int max_N) {
  if (!ctx || max_batch < 1 || max_N < 1) return 0;
  return (size_t)max_batch * carve_image(ctx, max_N, nullptr, nullptr);
}

pact_status pact_importance(pact_ctx *ctx, const pact_image *img, const pact_params *p, float *score,
                            void *ws, size_t ws_bytes, void *stream) {
  if (!ctx || !score) return PACT_ERR_INVALID_ARG;
  pact_status s = check_params(p);
  if (s != PACT_OK) return s;
  s = check_image(ctx, img, true, false, false);
  if (s != PACT_OK) return s;
  s = check_ws(ctx, ws, ws_bytes, 1, img->N);
  if (s != PACT_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  Batch bt;
  memset(&bt, 0, sizeof(bt));
  set_dims(ctx, bt, 1);
  ImgDesc &m = bt.img[0];
  carve_image(ctx, img->N, (char *)ws, &m);
  fill_user(m, img);
  m.Kc = nullptr;                        // no clustering keys in this stage
  m.score_user = score;
  set_params(m, p, img->N);
  point_counts_at_workspace(m);
  CK(cudaMemsetAsync(m.cnt, 0, (kCntInts + kTickInts) * sizeof(int32_t), st));
  CK(launch_euti(bt, img->N, ctx->in == PACT_BF16, 1, st));
  ctx->launches += euti_kernels(1);
  CK(cudaGetLastError());
  return PACT_OK;
}

pact_status pact_prune(pact_ctx *ctx, const float *score, int N, const pact_params *p, uint8_t *keep,
                       int32_t *kept_idx, int32_t *pruned_idx, int32_t *counts, void *ws, size_t ws_bytes,
                       void *stream) {
  if (!ctx || !score || !keep || !kept_idx || !pruned_idx || !counts || N < 1) return PACT_ERR_INVALID_ARG;
  pact_status s = check_params(p);
  if (s != PACT_OK) return s;
  s = check_ws(ctx, ws, ws_bytes, 1, N);
  if (s != PACT_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  Batch bt;
  memset(&bt, 0, sizeof(bt));
  set_dims(ctx, bt, 1);
  ImgDesc &m = bt.img[0];
  carve_image(ctx, N, (char *)ws, &m);
  m.N = N;
  set_params(m, p, N);
  point_counts_at_workspace(m);
  m.score = const_cast<float *>(score);
  m.keep = keep; m.kept_idx = kept_idx; m.pruned_idx = pruned_idx;
  launch_select_gather(bt, N, true, false, st);
  ctx->launches += 1;
  CK(cudaGetLastError());
  CK(cudaMemcpyAsync(counts, m.cnt + PACT_CNT_Q, sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
  CK(cudaMemcpyAsync(counts + 1, m.cnt + PACT_CNT_M, sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
  return PACT_OK;
}

pact_status pact_dbdpc(pact_ctx *ctx, const void *K, int64_t ldK, int N, const int32_t *idx,
                       const int32_t *q_dev, const pact_params *p, float *rho, int32_t *center_idx,
                       int32_t *C_dev, int32_t *label, int32_t *counters, void *ws, size_t ws_bytes,
                       void *stream) {
  if (!ctx || !K || !idx || !q_dev || !rho || !center_idx || !C_dev || !label || N < 1)
    return PACT_ERR_INVALID_ARG;
  if (!aligned16(K) || !ld_ok(ctx, ldK, ctx->d_k)) return PACT_ERR_INVALID_ARG;
  pact_status s = check_params(p);
  if (s != PACT_OK) return s;
  s = check_ws(ctx, ws, ws_bytes, 1, N);
  if (s != PACT_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  const bool bf = ctx->in == PACT_BF16;
  Batch bt;
  memset(&bt, 0, sizeof(bt));
  set_dims(ctx, bt, 1);
  ImgDesc &m = bt.img[0];
  carve_image(ctx, N, (char *)ws, &m);
  m.N = N; m.Kc = K; m.ldKc = ldK;
  set_params(m, p, N);
  point_counts_at_workspace(m);
  m.kept_idx = const_cast<int32_t *>(idx);
  m.q_ptr = q_dev;
  m.rho_user = rho; m.center_idx_user = center_idx; m.C_user = C_dev; m.label_user = label;
  CK(cudaMemsetAsync(m.cnt, 0, (kCntInts + kTickInts) * sizeof(int32_t), st));
  launch_keynorm_gather(bt, N, bf, false, st);
  if (ctx->umma) CK(launch_gram_umma(bt, N, ctx->ccfg, st));
  else launch_gram(bt, N, bf, ctx->ccfg, st);
  CK(launch_centers(bt, N, bf, ctx->ccfg, ctx->sweep_limit, st));
  if (ctx->umma) CK(launch_assign_umma(bt, N, true, ctx->ccfg, st));
  else launch_assign(bt, N, bf, ROWS_KEPT_LIST, ctx->ccfg, st);
  launch_label(bt, N, bf, ROWS_KEPT_LIST, st);
  ctx->launches += 5;
  CK(cudaGetLastError());
  if (counters)
    CK(cudaMemcpyAsync(counters, m.cnt, PACT_N_COUNTERS * sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
  return PACT_OK;
}

pact_status pact_key_spread(pact_ctx *ctx, const void *const *K_layers, int n_layers, int64_t ldK, int N,
                            float threshold, float *max_dist, int32_t *layer_out, void *ws, size_t ws_bytes,
                            void *stream) {
  if (!ctx || !K_layers || !max_dist || n_layers < 1 || N < 1) return PACT_ERR_INVALID_ARG;
  if (!ld_ok(ctx, ldK, ctx->d_k) || !(threshold == threshold)) return PACT_ERR_INVALID_ARG;
  for (int l = 0; l < n_layers; ++l)
    if (!K_layers[l] || !aligned16(K_layers[l])) return PACT_ERR_INVALID_ARG;
  const int per = n_layers < kMaxBatchPerLaunch ? n_layers : kMaxBatchPerLaunch;
  pact_status s = check_ws(ctx, ws, ws_bytes, per, N);
  if (s != PACT_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  const bool bf = ctx->in == PACT_BF16;
  const size_t per_img = carve_image(ctx, N, nullptr, nullptr);
  // the layers go through the tile kernels sixteen at a time, each as one image of a batch
  for (int base = 0; base < n_layers; base += kMaxBatchPerLaunch) {
    const int B = n_layers - base < kMaxBatchPerLaunch ? n_layers - base : kMaxBatchPerLaunch;
    Batch bt;
    memset(&bt, 0, sizeof(bt));
    set_dims(ctx, bt, B);
    for (int b = 0; b < B; ++b) {
      ImgDesc &m = bt.img[b];
      carve_image(ctx, N, (char *)ws + (size_t)b * per_img, &m);
      m.N = N; m.Kc = K_layers[base + b]; m.ldKc = ldK;
      point_counts_at_workspace(m);
      CK(cudaMemsetAsync(m.cnt, 0, (kCntInts + kTickInts) * sizeof(int32_t), st));
    }
    launch_key_rnorm(bt, N, bf, st);
    if (ctx->umma) CK(launch_spread_umma(bt, N, ctx->ccfg, st));
    else launch_spread(bt, N, bf, ctx->ccfg, st);
    launch_spread_finish(bt, max_dist, layer_out, base, threshold, st);
    ctx->launches += 3;
    CK(cudaGetLastError());
  }
  return PACT_OK;
}

pact_status pact_reincorporate(pact_ctx *ctx, const void *K, int64_t ldK, int N, const int32_t *pruned_idx,
                               const int32_t *m_dev, const int32_t *center_idx, const int32_t *C_dev,
                               const pact_params *p, int32_t *label, int32_t *r_dev, int32_t *counters,
                               void *ws, size_t ws_bytes, void *stream) {
  if (!ctx || !K || !pruned_idx || !m_dev || !center_idx || !C_dev || !label || !r_dev || N < 1)
    return PACT_ERR_INVALID_ARG;
  if (!aligned16(K) || !ld_ok(ctx, ldK, ctx->d_k)) return PACT_ERR_INVALID_ARG;
  pact_status s = check_params(p);
  if (s != PACT_OK) return s;
  s = check_ws(ctx, ws, ws_bytes, 1, N);
  if (s != PACT_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  const bool bf = ctx->in == PACT_BF16;
  Batch bt;
  memset(&bt, 0, sizeof(bt));
  set_dims(ctx, bt, 1);
  ImgDesc &m = bt.img[0];
  carve_image(ctx, N, (char *)ws, &m);
  m.N = N; m.Kc = K; m.ldKc = ldK;
  set_params(m, p, N);
  point_counts_at_workspace(m);
  m.pruned_idx = const_cast<int32_t *>(pruned_idx);
  m.m_ptr = m_dev; m.C_ptr = C_dev; m.cidx_ptr = center_idx;
  m.label = label;                      // updated in place
  CK(cudaMemsetAsync(m.cnt, 0, (kCntInts + kTickInts) * sizeof(int32_t), st));
  if (ctx->umma) {
    // the rows x centres pass on the tensor cores covers every token (the survivors' distances are computed
    // and not used), so every token needs its inverse key norm
    launch_key_rnorm(bt, N, bf, st);
    launch_center_key_gather(bt, N, bf, st);
    CK(launch_assign_umma(bt, N, false, ctx->ccfg, st));
    ctx->launches += 1;
  } else {
    launch_center_key_gather(bt, N, bf, st);
    launch_assign(bt, N, bf, ROWS_PRUNED_LIST, ctx->ccfg, st);
  }
  launch_label(bt, N, bf, ROWS_PRUNED_LIST, st);
  ctx->launches += 3;
  CK(cudaGetLastError());
  CK(cudaMemcpyAsync(r_dev, m.cnt + PACT_CNT_R, sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
  if (counters)
    CK(cudaMemcpyAsync(counters, m.cnt, PACT_N_COUNTERS * sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
  return PACT_OK;
}

pact_status pact_merge(pact_ctx *ctx, const pact_image *img, const int32_t *label, const int32_t *center_idx,
                       const int32_t *C_dev, const pact_params *p, void *ws, size_t ws_bytes, void *stream) {
  if (!ctx || !label || !center_idx || !C_dev) return PACT_ERR_INVALID_ARG;
  pact_status s = check_params(p);
  if (s != PACT_OK) return s;
  s = check_image(ctx, img, false, false, true);
  if (s != PACT_OK) return s;
  s = check_ws(ctx, ws, ws_bytes, 1, img->N);
  if (s != PACT_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  Batch bt;
  memset(&bt, 0, sizeof(bt));
  set_dims(ctx, bt, 1);
  ImgDesc &m = bt.img[0];
  carve_image(ctx, img->N, (char *)ws, &m);
  fill_user(m, img);
  set_params(m, p, img->N);
  point_counts_at_workspace(m);
  m.label = const_cast<int32_t *>(label);
  m.C_ptr = C_dev; m.cidx_ptr = center_idx;
  CK(cudaMemsetAsync(m.cnt, 0, (kCntInts + kTickInts) * sizeof(int32_t), st));
  CK(cudaMemsetAsync(m.csize, 0, (size_t)m.Np * sizeof(int32_t), st));
  CK(cudaMemsetAsync(m.cticket, 0, (size_t)m.Np * sizeof(int32_t), st));
  CK(cudaMemsetAsync(m.cnt_cb, 0, (size_t)m.Np * m.nbp * sizeof(uint16_t), st));
  CK(launch_lists(bt, img->N, ctx->in == PACT_BF16, false, ctx->spin_limit, st));
  CK(launch_merge(bt, ctx->in == PACT_BF16, ctx->out == PACT_BF16, ctx->ccfg, st));
  ctx->launches += lists_kernels(img->N, 1) + 1;
  CK(cudaGetLastError());
  CK(cudaMemcpyAsync(img->counters, m.cnt, PACT_N_COUNTERS * sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
  return PACT_OK;
}

pact_status pact_reduce(pact_ctx *ctx, const pact_image *imgs, int B, const pact_params *params,
                        int params_stride, void *ws, size_t ws_bytes, void *stream) {
  if (!ctx || !imgs || B < 1 || !params || (params_stride != 0 && params_stride != 1))
    return PACT_ERR_INVALID_ARG;
  int maxN = 0;
  for (int b = 0; b < B; ++b) {
    pact_status s = check_params(params + (size_t)b * params_stride);
    if (s != PACT_OK) return s;
    s = check_image(ctx, imgs + b, true, true, true);
    if (s != PACT_OK) return s;
    maxN = imgs[b].N > maxN ? imgs[b].N : maxN;
  }
  pact_status s = check_ws(ctx, ws, ws_bytes, B, maxN);
  if (s != PACT_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  const bool bf = ctx->in == PACT_BF16;
  const size_t per_img = carve_image(ctx, maxN, nullptr, nullptr);
  for (int b0 = 0; b0 < B; b0 += kMaxBatchPerLaunch) {
    const int nb = B - b0 < kMaxBatchPerLaunch ? B - b0 : kMaxBatchPerLaunch;
    Batch bt;
    memset(&bt, 0, sizeof(bt));
    set_dims(ctx, bt, nb);
    int cmaxN = 0, cmaxQ = 0;
    for (int b = 0; b < nb; ++b) {
      ImgDesc &m = bt.img[b];
      const pact_image *g = imgs + b0 + b;
      carve_image(ctx, g->N, (char *)ws + (size_t)(b0 + b) * per_img, &m);
      fill_user(m, g);
      set_params(m, params + (size_t)(b0 + b) * params_stride, g->N);
      point_counts_at_workspace(m);
      cmaxN = g->N > cmaxN ? g->N : cmaxN;
      const int qest = g->N - m.m_target + 64 < g->N ? g->N - m.m_target + 64 : g->N;   // survivors, with room for ties
      cmaxQ = qest > cmaxQ ? qest : cmaxQ;
      CK(cudaMemsetAsync(m.cnt, 0, (kCntInts + kTickInts) * sizeof(int32_t), st));
    }
    int stage = 0;
    auto mark = [&]() -> cudaError_t {
      ++stage;
      if (!ctx->prof_on || b0 != 0) return cudaSuccess;
      ctx->prof_n = stage;
      return cudaEventRecord(ctx->ev[stage], st);
    };
    if (ctx->prof_on && b0 == 0) CK(cudaEventRecord(ctx->ev[0], st));
    struct MarkFn {
      static cudaError_t call(void *p) { return (*static_cast<decltype(mark) *>(p))(); }
    };
    CK(launch_euti(bt, cmaxN, bf, 0, st, ctx->prof_on ? &MarkFn::call : nullptr, &mark));  CK(mark());
    if (ctx->umma) CK(launch_gram_umma(bt, cmaxN, ctx->ccfg, st, cmaxQ));
    else launch_gram(bt, cmaxN, bf, ctx->ccfg, st);
    CK(mark());
    CK(launch_centers(bt, cmaxQ, bf, ctx->ccfg, ctx->sweep_limit, st));  CK(mark());
    // On the tensor-core path with little work per SM (one image) the labels and member counts are formed as
    // the rows x centres pass finishes groups of rows, and one kernel places the members.  With much work per SM
    // the pass runs on pairs of CTAs, and k_lists forms labels and lists as it does on the fp32 path.
    const bool pairs = ctx->umma && umma_pairs_for_assign(cmaxN, nb, ctx->ccfg);
    const bool fused_labels = ctx->umma && !pairs;
    if (ctx->umma) CK(launch_assign_umma(bt, cmaxN, false, ctx->ccfg, st, fused_labels, pairs));
    else launch_assign(bt, cmaxN, bf, ROWS_ALL, ctx->ccfg, st);
    CK(mark());
    if (fused_labels) CK(launch_members(bt, cmaxN, st));
    else CK(launch_lists(bt, cmaxN, bf, true, ctx->spin_limit, st));
    CK(mark());
    CK(launch_merge(bt, bf, ctx->out == PACT_BF16, ctx->ccfg, st));  CK(mark());
    ctx->launches += euti_kernels(0) + 4 + (fused_labels ? 1 : lists_kernels(cmaxN, nb));
    CK(cudaGetLastError());
    for (int b = 0; b < nb; ++b)
      CK(cudaMemcpyAsync(bt.img[b].counters_user, bt.img[b].cnt, PACT_N_COUNTERS * sizeof(int32_t),
                         cudaMemcpyDeviceToDevice, st));
  }
  return PACT_OK;
}

pact_status pact_graph_create(pact_ctx *ctx, const pact_image *imgs, int B, const pact_params *params,
                              int params_stride, void *ws, size_t ws_bytes, pact_graph **out) {
  if (!ctx || !out) return PACT_ERR_INVALID_ARG;
  *out = nullptr;
  if (ctx->prof_on) return PACT_ERR_INVALID_ARG;      // per-kernel events are not recorded into graphs
  cudaStream_t cs = nullptr;
  CK(cudaStreamCreateWithFlags(&cs, cudaStreamNonBlocking));
  cudaError_t e = cudaStreamBeginCapture(cs, cudaStreamCaptureModeThreadLocal);
  if (e != cudaSuccess) { cudaStreamDestroy(cs); return fail_cuda(ctx, e, "cudaStreamBeginCapture"); }
  const long long before = ctx->launches;
  const pact_status s = pact_reduce(ctx, imgs, B, params, params_stride, ws, ws_bytes, cs);
  const int kernels = (int)(ctx->launches - before);
  ctx->launches = before;                              // nothing has run
  cudaGraph_t g = nullptr;
  e = cudaStreamEndCapture(cs, &g);
  cudaStreamDestroy(cs);
  if (s != PACT_OK) { if (g) cudaGraphDestroy(g); return s; }
  if (e != cudaSuccess || !g) return fail_cuda(ctx, e, "cudaStreamEndCapture");
  cudaGraphExec_t exec = nullptr;
  e = cudaGraphInstantiate(&exec, g, 0);
  cudaGraphDestroy(g);
  if (e != cudaSuccess) return fail_cuda(ctx, e, "cudaGraphInstantiate");
  pact_graph *pg = new (std::nothrow) pact_graph;
  if (!pg) { cudaGraphExecDestroy(exec); return PACT_ERR_INVALID_ARG; }
  pg->ctx = ctx; pg->exec = exec; pg->kernels = kernels;
  *out = pg;
  return PACT_OK;
}

pact_status pact_graph_launch(pact_graph *graph, void *stream) {
  if (!graph) return PACT_ERR_INVALID_ARG;
  pact_ctx *ctx = graph->ctx;
  CK(cudaGraphLaunch(graph->exec, (cudaStream_t)stream));
  ctx->launches += graph->kernels;
  return PACT_OK;
}

pact_status pact_graph_destroy(pact_graph *graph) {
  if (graph) {
    cudaGraphExecDestroy(graph->exec);
    delete graph;
  }
  return PACT_OK;
}

size_t pact_host_staging_bytes(const pact_ctx *ctx, int n_total, int N) {
  if (!ctx || n_total < 1 || N < 1) return 0;
  const size_t oe = ctx->out == PACT_BF16 ? 2 : 4;
  size_t b = 0;
  b += rup((size_t)n_total * ctx->d * ctx->elt, kAlign);         // H
  b += 2 * rup((size_t)N * ctx->d_k * ctx->elt, kAlign);          // K_euti, K_clu
  b += rup((size_t)N * ctx->n_qcols * ctx->elt, kAlign);          // Q
  b += rup((size_t)n_total * 4, kAlign);                          // P
  b += rup((size_t)n_total * ctx->d * oe, kAlign);                // H_out
  b += 3 * rup((size_t)n_total * 4, kAlign);                      // P_out, size_out, logw_out
  b += rup((size_t)N * 4, kAlign);                                // label
  b += rup(PACT_N_COUNTERS * 4, kAlign);                          // counters
  return b;
}

pact_status pact_reduce_host(pact_ctx *ctx, const pact_image *img, const pact_params *p, void *dev_staging,
                             size_t staging_bytes, void *ws, size_t ws_bytes, void *stream) {
  if (!ctx || !img || !p || !dev_staging) return PACT_ERR_INVALID_ARG;
  if (img->N < 1 || img->n_total < img->N) return PACT_ERR_INVALID_ARG;
  if (staging_bytes < pact_host_staging_bytes(ctx, img->n_total, img->N)) return PACT_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(dev_staging) % kAlign) != 0) return PACT_ERR_WORKSPACE;
  if (!img->H || !img->K_euti || !img->Q_euti || !img->K_clu || !img->P || !img->H_out || !img->P_out ||
      !img->size_out || !img->counters)
    return PACT_ERR_INVALID_ARG;
  if (img->ldH != ctx->d || img->ldKe != ctx->d_k || img->ldQ != ctx->n_qcols || img->ldKc != ctx->d_k ||
      img->ldHo != ctx->d)
    return PACT_ERR_INVALID_ARG;      // host buffers are dense
  cudaStream_t st = (cudaStream_t)stream;
  const size_t oe = ctx->out == PACT_BF16 ? 2 : 4;
  const int nt = img->n_total, N = img->N;
  char *base = (char *)dev_staging;
  size_t off = 0;
  auto take = [&](size_t bytes) { char *p0 = base + off; off += rup(bytes, kAlign); return p0; };
  const size_t bH = (size_t)nt * ctx->d * ctx->elt, bK = (size_t)N * ctx->d_k * ctx->elt,
               bQ = (size_t)N * ctx->n_qcols * ctx->elt, bHo = (size_t)nt * ctx->d * oe;
  char *dH = take(bH), *dKe = take(bK), *dKc = take(bK), *dQ = take(bQ), *dP = take((size_t)nt * 4);
  char *dHo = take(bHo), *dPo = take((size_t)nt * 4), *dSo = take((size_t)nt * 4), *dL = take((size_t)N * 4);
  char *dC = take(PACT_N_COUNTERS * 4);
  char *dLw = take((size_t)nt * 4);
  CK(cudaMemcpyAsync(dH, img->H, bH, cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(dKe, img->K_euti, bK, cudaMemcpyHostToDevice, st));
  const bool alias = img->K_clu == img->K_euti;
  if (!alias) CK(cudaMemcpyAsync(dKc, img->K_clu, bK, cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(dQ, img->Q_euti, bQ, cudaMemcpyHostToDevice, st));
  CK(cudaMemcpyAsync(dP, img->P, (size_t)nt * 4, cudaMemcpyHostToDevice, st));
  pact_image dv = *img;
  dv.H = dH; dv.K_euti = dKe; dv.K_clu = alias ? dKe : dKc; dv.Q_euti = dQ; dv.P = (const int32_t *)dP;
  dv.H_out = dHo; dv.P_out = (int32_t *)dPo; dv.size_out = (int32_t *)dSo; dv.label = (int32_t *)dL;
  dv.score = nullptr; dv.keep = nullptr; dv.counters = (int32_t *)dC;
  dv.logw_out = img->logw_out ? (float *)dLw : nullptr;
  pact_status s = pact_reduce(ctx, &dv, 1, p, 0, ws, ws_bytes, stream);
  if (s != PACT_OK) return s;
  // The number of valid output rows is data dependent: read the counters first, then copy
  // exactly the rows that exist.
  CK(cudaMemcpyAsync(img->counters, dC, PACT_N_COUNTERS * 4, cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  const int n_out = img->counters[PACT_CNT_N_OUT];
  if (n_out < 0 || n_out > nt) return PACT_ERR_INVALID_ARG;
  CK(cudaMemcpyAsync(img->H_out, dHo, (size_t)n_out * ctx->d * oe, cudaMemcpyDeviceToHost, st));
  CK(cudaMemcpyAsync(img->P_out, dPo, (size_t)n_out * 4, cudaMemcpyDeviceToHost, st));
  CK(cudaMemcpyAsync(img->size_out, dSo, (size_t)n_out * 4, cudaMemcpyDeviceToHost, st));
  if (img->logw_out) CK(cudaMemcpyAsync(img->logw_out, dLw, (size_t)n_out * 4, cudaMemcpyDeviceToHost, st));
  if (img->label) CK(cudaMemcpyAsync(img->label, dL, (size_t)N * 4, cudaMemcpyDeviceToHost, st));
  CK(cudaStreamSynchronize(st));
  return PACT_OK;
}

}  // extern "C"
