// Shared device-side declarations of the PACT reduction library (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/pact.h"

namespace pact {

constexpr int kMaxBatchPerLaunch = 16;   // images described by one kernel parameter block
constexpr int kRowsPerCta = 32;          // visual tokens handled by one CTA of the EUTI kernels
constexpr uint32_t kRhoShift = 30;       // density terms are summed as integers scaled by 2^30
constexpr unsigned long long kBestInit = 0xFFFFFFFFFFFFFFFFull;
constexpr int kCntSpread = 24;           // slot of cnt[]: largest key distance of a layer, as float bits
constexpr int kSpinLimit = 1 << 20;      // default number of polls a bounded device wait makes before it gives up
constexpr int kListBlock = 128;          // tokens per block of the member lists (128 measured 0.8 us faster per step than 256)
constexpr int kMaxTokens = 1 << 18;      // most visual tokens per image
constexpr int kCntInts = 64;             // counters and tickets at the head of an image's workspace ...
constexpr int kTickInts = 1024;          // ... followed by the tickets of k_qsum; both are cleared when a call starts

// Per-image device pointers: the caller's buffers and the slices of the workspace.
struct ImgDesc {
  // caller
  const void *H, *Ke, *Q, *Kc;
  long long ldH, ldKe, ldQ, ldKc, ldHo;
  const int32_t *P;
  void *H_out;
  int32_t *P_out, *size_out, *label_user, *counters_user;
  float *logw_out;
  float *score_user;
  unsigned char *keep_user;
  int n_total, vis_start, N;
  // parameters
  int m_target;          // number of tokens the percentile aims to prune
  float d_c, inv_dn_log2e, t_reinc;
  double d_c64, inv_dn64, t_reinc64;
  unsigned flags;
  // workspace
  double *qpart;         // [kQPartRows][n_qcols] partial column sums of Q
  double *qg;            // [n_qcols] global query
  double *E;             // [N][n_qh] exp(logit - CTA max)
  double *part;          // [G][n_qh][2] per-CTA (max, sum) of k_tokens, G = ceil(N / 32)
  int32_t *ghist;        // [2^kHistBits] scores per bin of their top key bits
  double *nrm;           // [N] hidden-state norms
  float *score;          // [N]
  unsigned char *keep;   // [N]
  int32_t *slot;         // [N] position in kept list, or -1-position in pruned list
  int32_t *kept_idx;     // [N]
  int32_t *pruned_idx;   // [N]
  float *rn;             // [N] 1/|k_i| of the clustering keys, token order
  double *rn64;          // [N] same in double (fp32-input path)
  void *Kp;              // [Np][d_k] gathered keys of the survivors
  float *rnk;            // [Np] 1/|k| in survivor order
  double *rnk64;         // [Np]
  unsigned long long *rho_fix;  // [Np] integer density
  float *rho;            // [Np]
  uint32_t *adj;         // [Np][Wp] adjacency bits (d <= d_c), later masked to earlier neighbours
  uint32_t *cmask;       // [Wp] centres
  uint32_t *rmask;       // [Wp] removed (within d_c of an earlier centre)
  void *Kcen;            // [Np][d_k] centre keys in cluster-id order
  float *rnc;            // [Np]
  double *rnc64;         // [Np]
  int32_t *center_idx;   // [Np] token index of centre c
  int32_t *cid;          // [Np] cluster id of survivor r if it is a centre
  unsigned long long *best;  // [N] packed (distance bits << 32 | cluster id)
  int32_t *label;        // [N]
  int32_t *blocklist;    // [ceil(N/256)][256] tokens of each block sorted by (cluster id, token); two-launch form of k_lists only
  uint16_t *cnt_cb;      // [Np][nbp] members of cluster c in token block b; zero before k_lists
  int4 *members;         // [N] {token, cluster, first member position of the cluster, cluster size}, cluster order
  int32_t *csize;        // [Np] members of cluster c
  int32_t *cticket;      // [Np] chunks of cluster c that are finished
  int32_t *rtick;        // [Wp] epilogue warps of the rows x centres pass that are done with a group of 32 tokens
  float *mpart;          // [2 * merge CTAs][d] sums of the clusters that a range boundary of k_merge cuts
  int32_t *tick;         // [kTickInts] tickets of k_qsum, one per column group; zero when a call starts (cleared with cnt)
  int32_t *cnt;          // [PACT_N_COUNTERS] + [16] ticket of the global query, [19] barrier of k_lists, [20] members of all clusters
  const int32_t *q_ptr;  // where the number of survivors lives (cnt[Q] or the caller's q_dev)
  const int32_t *m_ptr;  // where the number of pruned tokens lives
  const int32_t *C_ptr;  // where the number of clusters lives
  const int32_t *cidx_ptr;  // token index of centre c (workspace or caller)
  float *rho_user;       // optional outputs of the stage calls
  int32_t *center_idx_user, *C_user, *r_user;
  unsigned long long *tl; // timeline buffer of the instrumented build (PACT_TIMELINE), else unused
  int Np, Wp;            // padded survivor capacity and words per adjacency row
  int nbp;               // entries per row of cnt_cb: token blocks, rounded up to a multiple of 8
};

struct Batch {
  ImgDesc img[kMaxBatchPerLaunch];
  int B;
  int d, n_qh, n_kvh, d_h, d_k, n_qcols;
};

// ---- optional per-CTA timeline (instrumented build only; compiles to nothing otherwise) ----------
#ifdef PACT_TIMELINE
constexpr int kTlCtas = 4096;
struct TlScope {
  unsigned long long *slot;
  __device__ __forceinline__ TlScope(const ImgDesc &im, int kid) {
    const unsigned cta = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
    slot = (im.tl && cta < kTlCtas) ? im.tl + ((size_t)kid * kTlCtas + cta) * 2 : nullptr;
    if (slot && threadIdx.x == 0) {
      unsigned long long t;
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
      slot[0] = t;
    }
  }
  __device__ __forceinline__ ~TlScope() {
    if (slot && (threadIdx.x & 31) == 0) {
      unsigned long long t;
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
      atomicMax(slot + 1, t);
    }
  }
};
#define TL_SCOPE(im, kid) TlScope tl_scope_(im, kid)
// a point inside a kernel: the time thread 0 of each CTA passes it, stored like a start time
#define TL_POINT(im, kid) TL_POINT_IF(im, kid, threadIdx.x == 0)
#define TL_POINT_IF(im, kid, cond)                                                                   \
  do {                                                                                               \
    const unsigned cta_ = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);            \
    if ((im).tl && cta_ < kTlCtas && (cond)) {                                             \
      unsigned long long t_;                                                                         \
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_));                                          \
      (im).tl[((size_t)(kid) * kTlCtas + cta_) * 2] = t_;                                            \
      (im).tl[((size_t)(kid) * kTlCtas + cta_) * 2 + 1] = t_;                                        \
    }                                                                                                \
  } while (0)
#else
#define TL_SCOPE(im, kid)
#define TL_POINT(im, kid)
#define TL_POINT_IF(im, kid, cond)
#endif

// ---- element access ----------------------------------------------------------------------

template <typename T> struct Vec;      // 16-byte vector of T
template <> struct Vec<__nv_bfloat16> { static constexpr int N = 8; };
template <> struct Vec<float> { static constexpr int N = 4; };

// Loads 16 bytes and widens to float.
template <typename T> __device__ __forceinline__ void load_vec(const T *p, float (&out)[Vec<T>::N]);

template <> __device__ __forceinline__ void load_vec<__nv_bfloat16>(const __nv_bfloat16 *p, float (&out)[8]) {
  uint4 v = *reinterpret_cast<const uint4 *>(p);
  uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    out[2 * i] = __uint_as_float(w[i] << 16);
    out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}
template <> __device__ __forceinline__ void load_vec<float>(const float *p, float (&out)[4]) {
  float4 v = *reinterpret_cast<const float4 *>(p);
  out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
}

__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float to_float(float v) { return v; }

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Widens a 16-byte vector that is already in registers.
template <typename T> __device__ __forceinline__ void widen_vec(const uint4 &v, float (&out)[Vec<T>::N]);
template <> __device__ __forceinline__ void widen_vec<__nv_bfloat16>(const uint4 &v, float (&out)[8]) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    out[2 * i] = __uint_as_float(w[i] << 16);
    out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
  }
}
template <> __device__ __forceinline__ void widen_vec<float>(const uint4 &v, float (&out)[4]) {
  out[0] = __uint_as_float(v.x); out[1] = __uint_as_float(v.y);
  out[2] = __uint_as_float(v.z); out[3] = __uint_as_float(v.w);
}

// Sum of squares of 16-byte vectors: each vector is summed in float (the squares of bf16 values are
// exact in float) and the vectors are accumulated in double.
template <typename T> __device__ __forceinline__ void sumsq_accumulate(const uint4 &v, double &acc) {
  constexpr int V = Vec<T>::N;
  float x[V];
  widen_vec<T>(v, x);
  if (sizeof(T) == 2) {
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < V; ++i) s = fmaf(x[i], x[i], s);
    acc += (double)s;
  } else {
#pragma unroll
    for (int i = 0; i < V; ++i) acc = fma((double)x[i], (double)x[i], acc);
  }
}

// ---- programmatic dependent launch ----------------------------------------------------------------------
// The step is a chain of short kernels.  A kernel launched with the programmatic-serialization attribute may
// start while its predecessor in the stream is still running: pdl_wait() blocks until the predecessor has
// finished and its writes are visible; whatever does not depend on it (set-up, and in k_tokens the whole pass
// over the hidden states) runs before.  pdl_trigger() in the predecessor lets the successor's CTAs be
// scheduled from then on.  Every CTA of every kernel calls pdl_wait() before it returns, so completion of a
// kernel implies completion of all kernels before it.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ---- L2 eviction hints -------------------------------------------------------------------------
// The hidden states are read twice, by the scoring pass and by the merge, with everything else of the step
// in between; together that is more than the L2 keeps under its default policy.  The first pass asks for
// its lines to be evicted last, streams that are read once ask to be evicted first.
__device__ __forceinline__ unsigned long long policy_evict_last() {
  unsigned long long p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ unsigned long long policy_evict_first() {
  unsigned long long p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint4 ldg_hint(const uint4 *p, unsigned long long policy) {
  uint4 v;
  asm volatile("ld.global.nc.L2::cache_hint.v4.u32 {%0, %1, %2, %3}, [%4], %5;"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "l"(policy));
  return v;
}

// The same with a compile-time byte offset folded into the instruction: a run of such loads from one base
// needs one address register, not one per load.
template <int OFF>
__device__ __forceinline__ uint4 ldg_hint_off(const uint4 *p, unsigned long long policy) {
  uint4 v;
  asm volatile("ld.global.nc.L2::cache_hint.v4.u32 {%0, %1, %2, %3}, [%4 + %6], %5;"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "l"(policy), "n"(OFF));
  return v;
}

// buf[u] = base[32 u] for the u with v0 + 32 u < nv, all from one address register
template <int U, int I>
__device__ __forceinline__ void load_run_hint(uint4 (&buf)[U], const uint4 *base, int v0, int nv, unsigned long long policy) {
  if constexpr (I < U) {
    if (v0 + 32 * I < nv) buf[I] = ldg_hint_off<32 * I * 16>(base, policy);
    load_run_hint<U, I + 1>(buf, base, v0, nv, policy);
  }
}

// This lane's share (vectors lane, lane + 32, ... in ascending order) of the sum of squares of a
// row of n elements, starting at vector `from`.  Up to U loads per lane are in flight at once.
template <typename T, int U, bool HINT = false>
__device__ __forceinline__ double row_sumsq_lane(const T *row, int n, int lane, int from = 0,
                                                 unsigned long long policy = 0ull) {
  const int nv = n / Vec<T>::N;
  const uint4 *p = reinterpret_cast<const uint4 *>(row);
  double acc = 0.0;
  for (int v0 = from + lane; v0 < nv; v0 += 32 * U) {
    uint4 buf[U];
    if (HINT) {
      load_run_hint<U, 0>(buf, p + v0, v0, nv, policy);
    } else {
#pragma unroll
      for (int u = 0; u < U; ++u)
        if (v0 + 32 * u < nv) buf[u] = __ldg(p + v0 + 32 * u);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      if (v0 + 32 * u < nv) sumsq_accumulate<T>(buf[u], acc);
      // one vector after the other: left to itself the compiler widens all U vectors at once for the sake of
      // instruction-level parallelism and spills the loaded data, which serialises the loads
      if (u + 1 < U) asm volatile("" : "+r"(buf[u + 1].x), "+d"(acc));
    }
  }
  return acc;
}

// Sum of squares of one row by one warp.
template <typename T>
__device__ __forceinline__ double row_sumsq(const T *row, int n, int lane) {
  return warp_sum(row_sumsq_lane<T, 8>(row, n, lane));
}

// ---- distance epilogue: the one place that turns a dot product into a distance ------------

struct DistF {   // bf16 inputs: float arithmetic
  using acc_t = float;
  using rn_t = float;
  __device__ static __forceinline__ float dist(float dot, float rn_i, float rn_j) {
    float c = (dot * rn_i) * rn_j;
    return fminf(fmaxf(1.0f - c, 0.0f), 2.0f);
  }
  __device__ static __forceinline__ uint32_t term(float d, const ImgDesc &im) {
    float e = exp2f(-d * im.inv_dn_log2e);
    return __float2uint_rn(e * (float)(1u << kRhoShift));
  }
  __device__ static __forceinline__ bool within(float d, const ImgDesc &im) { return d <= im.d_c; }
  __device__ static __forceinline__ bool in_band(float d, const ImgDesc &im) { return fabsf(d - im.d_c) <= 1e-6f; }
  __device__ static __forceinline__ bool below_t(float d, const ImgDesc &im) { return d < im.t_reinc; }
  __device__ static __forceinline__ bool in_band_t(float d, const ImgDesc &im) { return fabsf(d - im.t_reinc) <= 1e-6f; }
};

struct DistD {   // fp32 inputs: double arithmetic
  using acc_t = double;
  using rn_t = double;
  __device__ static __forceinline__ double dist(double dot, double rn_i, double rn_j) {
    double c = (dot * rn_i) * rn_j;
    return fmin(fmax(1.0 - c, 0.0), 2.0);
  }
  __device__ static __forceinline__ uint32_t term(double d, const ImgDesc &im) {
    double e = exp(-d * im.inv_dn64);
    return (uint32_t)__double2uint_rn(e * (double)(1u << kRhoShift));
  }
  __device__ static __forceinline__ bool within(double d, const ImgDesc &im) { return d <= im.d_c64; }
  __device__ static __forceinline__ bool in_band(double d, const ImgDesc &im) { return fabs(d - im.d_c64) <= 1e-6; }
  __device__ static __forceinline__ bool below_t(double d, const ImgDesc &im) { return d < im.t_reinc64; }
  __device__ static __forceinline__ bool in_band_t(double d, const ImgDesc &im) { return fabs(d - im.t_reinc64) <= 1e-6; }
};

template <typename D> __device__ __forceinline__ typename D::rn_t *rn_tok(const ImgDesc &im);
template <> __device__ __forceinline__ float *rn_tok<DistF>(const ImgDesc &im) { return im.rn; }
template <> __device__ __forceinline__ double *rn_tok<DistD>(const ImgDesc &im) { return im.rn64; }
template <typename D> __device__ __forceinline__ typename D::rn_t *rn_kept(const ImgDesc &im);
template <> __device__ __forceinline__ float *rn_kept<DistF>(const ImgDesc &im) { return im.rnk; }
template <> __device__ __forceinline__ double *rn_kept<DistD>(const ImgDesc &im) { return im.rnk64; }
template <typename D> __device__ __forceinline__ typename D::rn_t *rn_cen(const ImgDesc &im);
template <> __device__ __forceinline__ float *rn_cen<DistF>(const ImgDesc &im) { return im.rnc; }
template <> __device__ __forceinline__ double *rn_cen<DistD>(const ImgDesc &im) { return im.rnc64; }

template <typename T> struct DistOf;
template <> struct DistOf<__nv_bfloat16> { using type = DistF; };
template <> struct DistOf<float> { using type = DistD; };

}  // namespace pact
