// EUTI (Algorithm 1): global query (Eq. 1), per-head softmax over the visual tokens and hidden-state
// norm (Eq. 2), percentile split (Eq. 3-4).  Every accumulation that decides an ordering is carried
// in double so that the float32 score the library returns is the correctly rounded value in all but
// rare double-rounding cases.
//
//   k_qsum           column sums of Q -> global query; also clears what later kernels accumulate into
//   k_tokens         one pass over the hidden states and the keys: |h_i|, 1 / |k_i|, k_i . Qglobal per head,
//                    CTA-local softmax pieces (HBM-bound, the first of two reads of H)
//   k_scores         merges the pieces, writes the float32 scores and the histogram of their top key bits
//   k_select         every CTA selects the threshold (histogram bin, then radix passes inside the bin) and
//                    counts the survivors before its tokens, then writes its share of the lists and gathers
//                    its share of the survivor keys
//   k_select_gather  the split for the stage call pact_prune (scores given, no histogram): radix select
//
// The kernels are short chains of dependent memory round trips; each issues all the loads it can
// before it consumes the first.
#include "kernels.cuh"

namespace pact {

__device__ __forceinline__ double ld_cg_f64(const double *p) {
  double v;
  asm volatile("ld.global.cg.f64 %0, [%1];" : "=d"(v) : "l"(p));
  return v;
}

// sort key of a score: unsigned integers that order like the floats
__device__ __forceinline__ uint32_t score_key(float s) {
  uint32_t b = __float_as_uint(s);
  if (b == 0x80000000u) b = 0;                       // -0 orders as +0
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// ---- Eq. 1: column sums of Q -----------------------------------------------------------------------------
// grid (ncg RP, B), 512 threads at no more than 64 registers, on fewer than half of the SMs: a CTA leaves room
// for one CTA of k_tokens beside it, and the other SMs take two, so that all of them start at once.  Work item
// (column group of eight 16-byte vectors, block of rows): thread t takes vector t & 7 of the group and the rows
// r0 + (t >> 3), + 64, ...; the four row lanes of a warp are added with shuffles, the warps through
// shared memory.  The CTA that finishes a column group's last
// row block adds the RP partial sums in block order and writes the group's part of the global query, so the
// result does not depend on which CTA that is.  do_init: the grid also clears what later kernels accumulate
// into.
constexpr int kQsumThreads = 512;
constexpr int kQsumRowLanes = kQsumThreads / 8;
constexpr int kQsumWarps = kQsumThreads / 32;

template <typename T>
__global__ void __launch_bounds__(kQsumThreads, 2) k_qsum(const __grid_constant__ Batch bt, int RP, int do_init) {
  constexpr int V = Vec<T>::N;
  const ImgDesc &im = bt.img[blockIdx.y];
  TL_SCOPE(im, 0);
  pdl_trigger();                                        // k_tokens may start: its first pass does not need the query
  const int t = threadIdx.x, lane = t & 31, w = t >> 5, N = im.N, n_qcols = bt.n_qcols;
  if (do_init) {
    const int gt = blockIdx.x * kQsumThreads + t, gs = gridDim.x * kQsumThreads;
    for (int r = gt; r < im.Np; r += gs) { im.rho_fix[r] = 0ull; im.csize[r] = 0; im.cticket[r] = 0; }
    for (int wd = gt; wd < im.Wp; wd += gs) { im.cmask[wd] = 0u; im.rmask[wd] = 0u; im.rtick[wd] = 0; }
    for (int i = gt; i < N; i += gs) im.best[i] = kBestInit;
    uint4 *tab = reinterpret_cast<uint4 *>(im.cnt_cb);
    const int nq = im.Np * (im.nbp / 8);
    for (int i = gt; i < nq; i += gs) tab[i] = make_uint4(0u, 0u, 0u, 0u);
    for (int i = gt; i < (1 << kHistBits); i += gs) im.ghist[i] = 0;
  }
  if (!im.Q || (im.flags & PACT_FLAG_NORM_ONLY)) return;
  const int nvq = n_qcols / V, ncg = (nvq + 7) / 8;
  const int cg = blockIdx.x % ncg, rp = blockIdx.x / ncg;
  if (rp >= RP) return;
  __shared__ double sm[kQsumWarps * 8 * V];
  __shared__ int s_last;
  const int rchunk = (N + RP - 1) / RP;
  const int r0 = min(N, rp * rchunk), r1 = min(N, r0 + rchunk);
  const int v = cg * 8 + (t & 7);
  const unsigned long long pol = policy_evict_first();   // Q is read once
  const T *Q = reinterpret_cast<const T *>(im.Q);
  double acc[V];
#pragma unroll
  for (int k = 0; k < V; ++k) acc[k] = 0.0;
  if (v < nvq) {
    constexpr int UQ = 8;
    const size_t coff = (size_t)v * V;
    for (int r = r0 + (t >> 3); r < r1; r += kQsumRowLanes * UQ) {
      uint4 buf[UQ];
#pragma unroll
      for (int u = 0; u < UQ; ++u)
        if (r + u * kQsumRowLanes < r1)
          buf[u] = ldg_hint(reinterpret_cast<const uint4 *>(Q + (size_t)(r + u * kQsumRowLanes) * im.ldQ + coff), pol);
#pragma unroll
      for (int u = 0; u < UQ; ++u) {
        if (r + u * kQsumRowLanes < r1) {
          float x[V];
          widen_vec<T>(buf[u], x);
#pragma unroll
          for (int k = 0; k < V; ++k) acc[k] += (double)x[k];
        }
      }
    }
  }
#pragma unroll
  for (int k = 0; k < V; ++k) {
    acc[k] += __shfl_xor_sync(0xffffffffu, acc[k], 8);
    acc[k] += __shfl_xor_sync(0xffffffffu, acc[k], 16);
  }
  if (lane < 8) {
#pragma unroll
    for (int k = 0; k < V; ++k) sm[(w * 8 + lane) * V + k] = acc[k];
  }
  __syncthreads();
  const bool col_ok = t < 8 * V && cg * 8 + t / V < nvq;
  const size_t col = (size_t)cg * 8 * V + t;
  double mine = 0.0;
  if (col_ok) {
#pragma unroll
    for (int ww = 0; ww < kQsumWarps; ++ww) mine += sm[ww * 8 * V + t];
  }
  if (RP == 1) {
    if (col_ok) im.qg[col] = mine / (double)N;
    return;
  }
  if (col_ok) im.qpart[(size_t)rp * n_qcols + col] = mine;
  __threadfence();
  __syncthreads();
  if (t == 0) s_last = atomicAdd(&im.tick[cg], 1) == RP - 1;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  if (col_ok) {
    double s = 0.0;
#pragma unroll
    for (int u0 = 0; u0 < kQPartRows; u0 += 16) {       // sixteen partial sums in flight, added in block order
      if (u0 < RP) {
        double pv[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) pv[u] = u0 + u < RP ? ld_cg_f64(&im.qpart[(size_t)(u0 + u) * n_qcols + col]) : 0.0;
#pragma unroll
        for (int u = 0; u < 16; ++u) s += pv[u];
      }
    }
    im.qg[col] = s / (double)N;
  }
}

// ---- Eq. 2, token pass: hidden-state norm, inverse key norm, logits, CTA-local softmax pieces ---------------
// grid (ceil(maxN / 32), B), 256 threads, two CTAs per SM; dynamic smem (n_qcols + 32 n_qh) doubles.
// A CTA takes 32 tokens, a warp four of them.  First the rows, one token after the other: the 16-byte loads of
// the token's clustering-key row and hidden-state row are all issued before the first is used (the
// hidden-state lines are asked to stay in the L2 for the merge); |h_i| in double, 1 / |k_i|.  Then the logits
// of the warp's four tokens together: k_i . Qglobal per head in double.  Then per head the largest logit of the
// CTA's tokens, exp(l - that) per token and their sum.
constexpr int kTokThreads = 256;
constexpr int kTokWarps = kTokThreads / 32;
constexpr int kTokPerWarp = kRowsPerCta / kTokWarps;

template <typename T>
__global__ void __launch_bounds__(kTokThreads, 2) k_tokens(const __grid_constant__ Batch bt) {
  using D = typename DistOf<T>::type;
  using rn_t = typename D::rn_t;
  constexpr int V = Vec<T>::N;
  constexpr int UK = 2;                                 // preloaded 16-byte vectors of the key row per lane
  const ImgDesc &im = bt.img[blockIdx.y];
  TL_SCOPE(im, 1);
  const int g = blockIdx.x, t = threadIdx.x, lane = t & 31, w = t >> 5;
  const int N = im.N, n_qh = bt.n_qh, n_qcols = bt.n_qcols;
  const int r0 = g * kRowsPerCta, r1 = min(N, r0 + kRowsPerCta);
  if (r0 >= N) { pdl_wait(); return; }
  extern __shared__ double smd[];
  double *qT = smd;                                     // [n_qcols] global query, transposed (see below)
  double *lg = smd + n_qcols;                           // [32][n_qh]
  const bool use_query = !(im.flags & PACT_FLAG_NORM_ONLY) && im.Q != nullptr;
  const int nv = bt.d_k / V, vph = bt.d_h / V, nvq = n_qcols / V;
  const T *Ke = reinterpret_cast<const T *>(im.Ke);
  const unsigned long long pol_keep = policy_evict_last();
  // fast path of the logits: one query head per key head and a power-of-two number of vectors per head, all
  // preloaded: the lanes that hold one head's vectors form a group, reduced with xor shuffles inside the group
  const bool grouped = n_qh == bt.n_kvh && (vph & (vph - 1)) == 0 && vph <= 32 && nv <= 32 * UK;

  // the global query is kept transposed, qT[k][vq] = Qglobal[vq * V + k], so that the lanes of a warp,
  // which hold consecutive 16-byte vectors of the key row, read consecutive doubles
  // the rows: |h_i| and 1 / |k_i| of one of the warp's tokens
  auto row_pass = [&](int i) {
    const int tok = r0 + w * kTokPerWarp + i;
    if (tok >= r1) return;                              // the same for the whole warp
    uint4 kb[UK];
    const T *kcrow = im.Kc ? reinterpret_cast<const T *>(im.Kc) + (size_t)tok * im.ldKc : nullptr;
    if (kcrow) {
#pragma unroll
      for (int u = 0; u < UK; ++u)
        if (lane + 32 * u < nv) kb[u] = __ldg(reinterpret_cast<const uint4 *>(kcrow) + lane + 32 * u);
    }
    double nn = 1.0;
    if (!(im.flags & PACT_FLAG_NO_NORM)) {
      const T *hrow = reinterpret_cast<const T *>(im.H) + (size_t)(im.vis_start + tok) * im.ldH;
      nn = sqrt(warp_sum(row_sumsq_lane<T, 16, true>(hrow, bt.d, lane, 0, pol_keep)));
    }
    if (lane == 0) im.nrm[tok] = nn;
    if (kcrow) {
      double a = 0.0;
#pragma unroll
      for (int u = 0; u < UK; ++u)
        if (lane + 32 * u < nv) sumsq_accumulate<T>(kb[u], a);
      if (nv > 32 * UK) a += row_sumsq_lane<T, 8>(kcrow, bt.d_k, lane, 32 * UK);
      const double ss = warp_sum(a);
      if (lane == 0) rn_tok<D>(im)[tok] = (rn_t)(1.0 / sqrt(fmax(ss, 1e-40)));
    }
  };
  // first all but the last of the warp's tokens, one after the other
#pragma unroll 1
  for (int i = 0; i + 1 < kTokPerWarp; ++i) row_pass(i);
  // the last token's hidden-state row is asked for now (into the L2) and read after the logits, which are
  // formed while it is on its way
  {
    const int tok = r0 + w * kTokPerWarp + kTokPerWarp - 1;
    if (tok < r1 && !(im.flags & PACT_FLAG_NO_NORM)) {
      const char *hrow = reinterpret_cast<const char *>(reinterpret_cast<const T *>(im.H) + (size_t)(im.vis_start + tok) * im.ldH);
      const int bytes = bt.d * (int)sizeof(T);
      for (int o = lane * 128; o < bytes; o += 32 * 128)
        asm volatile("prefetch.global.L2::evict_last [%0];" ::"l"(hrow + o));
    }
  }
  // the global query is kept transposed, qT[k][vq] = Qglobal[vq * V + k], so that the lanes of a warp,
  // which hold consecutive 16-byte vectors of the key row, read consecutive doubles
  pdl_wait();                                           // the global query is complete
  pdl_trigger();
  if (use_query)
    for (int c = t; c < n_qcols; c += kTokThreads) qT[(c % V) * nvq + c / V] = ld_cg_f64(&im.qg[c]);
  __syncthreads();
  // then the logits: the key rows of the warp's tokens (read a moment ago when the two key matrices are one)
  // are loaded together
  {
    uint4 kb[kTokPerWarp][UK];
#pragma unroll
    for (int i = 0; i < kTokPerWarp; ++i) {
      const uint4 *krow = reinterpret_cast<const uint4 *>(Ke + (size_t)min(r0 + w * kTokPerWarp + i, N - 1) * im.ldKe);
#pragma unroll
      for (int u = 0; u < UK; ++u)
        if (lane + 32 * u < nv) kb[i][u] = __ldg(krow + lane + 32 * u);
    }
    const int l0 = w * kTokPerWarp;                     // first token of the warp within the CTA
    if (grouped) {
      double acc[kTokPerWarp][UK];
#pragma unroll
      for (int u = 0; u < UK; ++u) {
        const int v = lane + 32 * u;
#pragma unroll
        for (int i = 0; i < kTokPerWarp; ++i) acc[i][u] = 0.0;
        if (use_query && v < nv) {
          double qv[V];
#pragma unroll
          for (int k = 0; k < V; ++k) qv[k] = qT[k * nvq + v];
#pragma unroll
          for (int i = 0; i < kTokPerWarp; ++i) {
            float x[V];
            widen_vec<T>(kb[i][u], x);
#pragma unroll
            for (int k = 0; k < V; ++k) acc[i][u] = fma((double)x[k], qv[k], acc[i][u]);
          }
        }
      }
      for (int o = vph >> 1; o > 0; o >>= 1)
#pragma unroll
        for (int i = 0; i < kTokPerWarp; ++i)
#pragma unroll
          for (int u = 0; u < UK; ++u) acc[i][u] += __shfl_xor_sync(0xffffffffu, acc[i][u], o);
      if ((lane & (vph - 1)) == 0) {
#pragma unroll
        for (int i = 0; i < kTokPerWarp; ++i)
#pragma unroll
          for (int u = 0; u < UK; ++u)
            if (lane + 32 * u < nv) lg[(l0 + i) * n_qh + (lane + 32 * u) / vph] = acc[i][u];
      }
    } else {
      for (int j = 0; j < n_qh; ++j) {
        double acc[kTokPerWarp];
#pragma unroll
        for (int i = 0; i < kTokPerWarp; ++i) acc[i] = 0.0;
        if (use_query) {
          const int kv = (j * bt.n_kvh) / n_qh;
          const int vshift = (j - kv) * vph;            // key-row vector v pairs with query vector v + vshift
#pragma unroll
          for (int u = 0; u < UK; ++u) {
            const int v = lane + 32 * u;
            if (v < nv && v / vph == kv) {
#pragma unroll
              for (int i = 0; i < kTokPerWarp; ++i) {
                float x[V];
                widen_vec<T>(kb[i][u], x);
#pragma unroll
                for (int k = 0; k < V; ++k) acc[i] = fma((double)x[k], qT[k * nvq + v + vshift], acc[i]);
              }
            }
          }
          for (int v = lane + 32 * UK; v < nv; v += 32) {   // rows wider than the preloaded part
            if (v / vph == kv) {
#pragma unroll
              for (int i = 0; i < kTokPerWarp; ++i) {
                const int rr = min(r0 + l0 + i, N - 1);
                float x[V];
                widen_vec<T>(__ldg(reinterpret_cast<const uint4 *>(Ke + (size_t)rr * im.ldKe) + v), x);
#pragma unroll
                for (int k = 0; k < V; ++k) acc[i] = fma((double)x[k], qT[k * nvq + v + vshift], acc[i]);
              }
            }
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
#pragma unroll
          for (int i = 0; i < kTokPerWarp; ++i) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], o);
        if (lane == 0) {
#pragma unroll
          for (int i = 0; i < kTokPerWarp; ++i) lg[(l0 + i) * n_qh + j] = acc[i];
        }
      }
    }
  }
  row_pass(kTokPerWarp - 1);
  __syncthreads();
  // per head: CTA max, exp, CTA sum; lane = token within the CTA
  for (int j = w; j < n_qh; j += kTokWarps) {
    const int rr = r0 + lane;
    const bool ok = rr < r1;
    const double l = ok ? lg[lane * n_qh + j] : -1.0e300;
    double m = l;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
    const double e = ok ? exp(l - m) : 0.0;
    if (ok) im.E[(size_t)rr * n_qh + j] = e;
    const double sum = warp_sum(e);
    if (lane == 0) {
      im.part[((size_t)g * n_qh + j) * 2] = m;
      im.part[((size_t)g * n_qh + j) * 2 + 1] = sum;
    }
  }
}

__device__ __forceinline__ void ld_cg_f64x2(const double *p, double &a, double &b) {
  asm volatile("ld.global.cg.v2.f64 {%0, %1}, [%2];" : "=d"(a), "=d"(b) : "l"(p));
}

// ---- Eq. 2, second half: merge the pieces (M = max, Z = sum S_g exp(M_g - M), fixed order), scores --------
// grid (ceil(maxN / 256), B), 256 threads.  Every CTA merges all G pieces itself: the warps share out the
// heads (and, with fewer heads than warps, the pieces of a head), four loads per lane in flight.  with_hist:
// every score also counts in the histogram of its top key bits, the first level of the threshold selection.
constexpr int kScoreWarps = 8;

__global__ void __launch_bounds__(256) k_scores(const __grid_constant__ Batch bt, int with_hist) {
  const ImgDesc &im = bt.img[blockIdx.y];
  TL_SCOPE(im, 2);
  pdl_wait();
  pdl_trigger();
  const int t = threadIdx.x, lane = t & 31, w = t >> 5;
  const int N = im.N, n_qh = bt.n_qh;
  if ((int)blockIdx.x * 256 >= N) return;
  const int G = (N + kRowsPerCta - 1) / kRowsPerCta;
  __shared__ double sM[256], sInv[256];
  __shared__ double pmx[kScoreWarps], pz[kScoreWarps];
  const int i = blockIdx.x * 256 + t;
  // this token's terms, requested before the merge so that they arrive meanwhile
  constexpr int EP = 4;
  double e_pre[EP], nrm_i = 0.0;
  const bool pre = n_qh <= EP && i < N;
  if (pre) {
#pragma unroll
    for (int j = 0; j < EP; ++j) e_pre[j] = j < n_qh ? im.E[(size_t)i * n_qh + j] : 0.0;
  }
  if (i < N) nrm_i = im.nrm[i];
  const int wph = n_qh >= kScoreWarps ? 1 : kScoreWarps / n_qh;   // warps per head
  const int hpp = kScoreWarps / wph;                    // heads per pass
  const int step = 32 * wph;
  const int nbatch = (G + 4 * step - 1) / (4 * step);
  for (int j0 = 0; j0 < n_qh; j0 += hpp) {
    const int j = j0 + w / wph, sub = w % wph;
    const bool mine = j < n_qh && w / wph < hpp;
    auto load4 = [&](int b, double (&pm)[4], double (&ps)[4]) {
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int h = sub * 32 + lane + step * (4 * b + u);
        pm[u] = -1.0e300;
        ps[u] = 0.0;
        if (mine && h < G) ld_cg_f64x2(im.part + ((size_t)h * n_qh + j) * 2, pm[u], ps[u]);
      }
    };
    double pm0[4], ps0[4];
    load4(0, pm0, ps0);
    double m = fmax(fmax(pm0[0], pm0[1]), fmax(pm0[2], pm0[3]));
    for (int b = 1; b < nbatch; ++b) {
      double pm[4], ps[4];
      load4(b, pm, ps);
      m = fmax(m, fmax(fmax(pm[0], pm[1]), fmax(pm[2], pm[3])));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
    __syncthreads();
    if (lane == 0) pmx[w] = m;
    __syncthreads();
    if (mine)
      for (int k = 0; k < wph; ++k) m = fmax(m, pmx[w - sub + k]);
    double z = 0.0;                                     // an empty slot adds 0 * exp(-huge) = 0
#pragma unroll
    for (int u = 0; u < 4; ++u) z += ps0[u] * exp(pm0[u] - m);
    for (int b = 1; b < nbatch; ++b) {
      double pm[4], ps[4];
      load4(b, pm, ps);
#pragma unroll
      for (int u = 0; u < 4; ++u) z += ps[u] * exp(pm[u] - m);
    }
    z = warp_sum(z);
    if (lane == 0) pz[w] = z;
    __syncthreads();
    if (mine && sub == 0 && lane == 0) {
      double zz = 0.0;
      for (int k = 0; k < wph; ++k) zz += pz[w + k];
      sM[j] = m;
      sInv[j] = 1.0 / (zz * (double)n_qh);
    }
  }
  __syncthreads();
  if (i >= N) return;
  const int g = i / kRowsPerCta;
  double s = 0.0;
  for (int j = 0; j < n_qh; ++j) {
    const double fac = exp(im.part[((size_t)g * n_qh + j) * 2] - sM[j]) * sInv[j];
    double e;
    if (pre) {
      e = e_pre[0];
#pragma unroll
      for (int q = 1; q < EP; ++q) if (j == q) e = e_pre[q];
    } else {
      e = im.E[(size_t)i * n_qh + j];
    }
    s = fma(e, fac, s);
  }
  const float sf = (float)(s * nrm_i);
  im.score[i] = sf;
  if (im.score_user) im.score_user[i] = sf;
  if (with_hist) atomicAdd(&im.ghist[score_key(sf) >> kHistShift], 1);
}

// ---- Eq. 3-4 in the whole step: threshold, ordered compaction, survivor keys (Eq. 7) ------------------------
// grid (X, B), 512 threads, two CTAs per SM; dynamic smem: N sort keys when they fit.  CTA x owns the tokens
// [x tpc, (x + 1) tpc).  Every CTA selects the threshold itself (identical in all of them), counts the
// survivors before its tokens, writes keep flags, lists and slots of its tokens and copies the clustering keys
// of its survivors to their rows of K'.
constexpr int kSelThreads = 512;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kHistPerThread = (1 << kHistBits) / kSelThreads;
constexpr int kSelBits = 10;                  // key bits per pass of the selection below the first-level histogram
constexpr int kSelPerThread = (1 << kSelBits) / kSelThreads;
static_assert(kHistPerThread % 4 == 0 && kHistPerThread * kSelThreads == (1 << kHistBits), "histogram split");

struct SelShared {
  int hist[1 << kSelBits];
  int wtot[kSelWarps], wtot2[kSelWarps];
  uint32_t s_prefix;
  int s_k, s_bin, s_cnt;
  int own_tok[kSelThreads], own_slot[kSelThreads];
};

// The key of the (m_target + 1)-th smallest score.  the key of the (m_target + 1)-th smallest score.  The histogram of the top kHistBits key
// bits, filled by k_scores, gives the bin of the threshold and its rank inside that bin; radix passes
// over the bits below, kSelBits at a time, finish the selection (only the keys of that bin take part, so the
// shared-memory counters see little contention; the bins of a pass are scanned by all threads).  KPT > 0: thread t holds the keys t, t + 512, ... in
// registers (N <= 512 KPT); KPT == 0: keys from shared memory (IN_SMEM) or re-read from the scores.
template <int KPT, bool IN_SMEM>
__device__ __forceinline__ uint32_t euti_threshold(const ImgDesc &im, const uint32_t *skey, const uint32_t (&kreg)[KPT > 0 ? KPT : 1],
                                                   const int (&hv)[kHistPerThread], SelShared &sh) {
  const int t = threadIdx.x, lane = t & 31, w = t >> 5, N = im.N;
  auto key_at = [&](int i) -> uint32_t { return IN_SMEM ? skey[i] : score_key(__ldcg(im.score + i)); };
  {
    int sum = 0;
#pragma unroll
    for (int u = 0; u < kHistPerThread; ++u) sum += hv[u];
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    if (lane == 31) sh.wtot[w] = incl;
    if (t == 0) { sh.s_bin = -1; sh.s_k = 0; }
#pragma unroll
    for (int u = 0; u < kSelPerThread; ++u) sh.hist[t * kSelPerThread + u] = 0;
    __syncthreads();
    int below = incl - sum;                             // keys in the bins before this thread's
#pragma unroll
    for (int k = 0; k < kSelWarps; ++k) if (k < w) below += sh.wtot[k];
    const int m_t = im.m_target;
    if (below <= m_t && m_t < below + sum) {            // exactly one thread, unless a wait ran out
      int k = m_t - below;
#pragma unroll
      for (int u = 0; u < kHistPerThread; ++u) {
        if (k >= 0 && k < hv[u]) { sh.s_k = k; sh.s_bin = t * kHistPerThread + u; k = -1; }
        else if (k >= 0) k -= hv[u];
      }
    }
    __syncthreads();
  }
  if (sh.s_bin < 0) return 0xffffffffu;                 // inconsistent histogram: keep nothing
  if (t == 0) sh.s_prefix = (uint32_t)sh.s_bin << kHistShift;
  __syncthreads();
  for (int hi = kHistShift; hi > 0; hi -= kSelBits) {
    const int lo = hi > kSelBits ? hi - kSelBits : 0;
    const uint32_t dmask = (1u << (hi - lo)) - 1u;
    const uint32_t above = ~((1u << hi) - 1u);          // bits already fixed
    const uint32_t prefix = sh.s_prefix;
    const int k = sh.s_k;
    if (KPT > 0) {
#pragma unroll
      for (int u = 0; u < (KPT > 0 ? KPT : 1); ++u) {
        const uint32_t kk = kreg[u];
        if (t + kSelThreads * u < N && (kk & above) == (prefix & above)) atomicAdd(&sh.hist[(kk >> lo) & dmask], 1);
      }
    } else {
      for (int i = t; i < N; i += kSelThreads) {
        const uint32_t kk = key_at(i);
        if ((kk & above) == (prefix & above)) atomicAdd(&sh.hist[(kk >> lo) & dmask], 1);
      }
    }
    __syncthreads();
    // every thread takes kSelPerThread bins: the one whose bins hold rank k names the digit
    int c[kSelPerThread], sum = 0;
#pragma unroll
    for (int u = 0; u < kSelPerThread; ++u) { c[u] = sh.hist[t * kSelPerThread + u]; sum += c[u]; sh.hist[t * kSelPerThread + u] = 0; }
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    if (lane == 31) sh.wtot[w] = incl;
    __syncthreads();
    int below = incl - sum;
#pragma unroll
    for (int q = 0; q < kSelWarps; ++q) if (q < w) below += sh.wtot[q];
    if (below <= k && k < below + sum) {                // exactly one thread: the candidates number more than k
      int kk = k - below;
#pragma unroll
      for (int u = 0; u < kSelPerThread; ++u) {
        if (kk >= 0 && kk < c[u]) {
          sh.s_k = kk;
          sh.s_cnt = c[u];
          sh.s_prefix = prefix | ((uint32_t)(t * kSelPerThread + u) << lo);
          kk = -1;
        } else if (kk >= 0) kk -= c[u];
      }
    }
    __syncthreads();
    if (lo > 0 && sh.s_cnt == 1) {                      // one key left under the prefix: it is the threshold
      const uint32_t fixed = ~((1u << lo) - 1u), pre2 = sh.s_prefix;
      if (KPT > 0) {
#pragma unroll
        for (int u = 0; u < (KPT > 0 ? KPT : 1); ++u)
          if (t + kSelThreads * u < N && (kreg[u] & fixed) == pre2) sh.s_prefix = kreg[u];
      } else {
        for (int i = t; i < N; i += kSelThreads) {
          const uint32_t kk = key_at(i);
          if ((kk & fixed) == pre2) sh.s_prefix = kk;
        }
      }
      __syncthreads();
      break;
    }
  }
  return sh.s_prefix;
}

// Survivors before the own tokens (every CTA counts them itself), then keep flags, lists and
// slots of the own tokens, and the clustering keys of the own survivors copied to their rows of K'.
template <typename T, int KPT, bool IN_SMEM>
__device__ __forceinline__ void euti_compact(const Batch &bt, const ImgDesc &im, const uint32_t *skey,
                                             const uint32_t (&kreg)[KPT > 0 ? KPT : 1], uint32_t tau_key, int g, int tok0,
                                             int ntok, SelShared &sh) {
  using D = typename DistOf<T>::type;
  constexpr int V = Vec<T>::N;
  const int t = threadIdx.x, lane = t & 31, w = t >> 5, N = im.N;
  auto key_at = [&](int i) -> uint32_t { return IN_SMEM ? skey[i] : score_key(__ldcg(im.score + i)); };
  int nb = 0, nall = 0;
  if (KPT > 0) {
#pragma unroll
    for (int u = 0; u < (KPT > 0 ? KPT : 1); ++u) {
      const int i = t + kSelThreads * u;
      const int kp = i < N && kreg[u] >= tau_key;
      nall += kp;
      nb += kp && i < tok0;
    }
  } else {
    for (int i = t; i < N; i += kSelThreads) {
      const int kp = key_at(i) >= tau_key;
      nall += kp;
      nb += kp && i < tok0;
    }
  }
  nb = __reduce_add_sync(0xffffffffu, nb);
  nall = __reduce_add_sync(0xffffffffu, nall);
  __syncthreads();
  if (lane == 0) { sh.wtot[w] = nb; sh.wtot2[w] = nall; }
  __syncthreads();
  int before0 = 0, q = 0;
#pragma unroll
  for (int k = 0; k < kSelWarps; ++k) { before0 += sh.wtot[k]; q += sh.wtot2[k]; }
  if (g == 0 && t == 0) {
    im.cnt[PACT_CNT_Q] = q;
    im.cnt[PACT_CNT_M] = N - q;
  }
  const int nv = bt.d_k / V;
  const T *Kc = reinterpret_cast<const T *>(im.Kc);
  T *Kp = reinterpret_cast<T *>(im.Kp);
  for (int c0 = 0; c0 < ntok; c0 += kSelThreads) {     // the own tokens, 512 at a time
    const int i = tok0 + c0 + t;
    const bool ok = c0 + t < ntok;
    const bool kp = ok && key_at(i) >= tau_key;
    const unsigned bal = __ballot_sync(0xffffffffu, kp);
    __syncthreads();
    if (lane == 0) sh.wtot[w] = __popc(bal);
    __syncthreads();
    int excl = __popc(bal & ((1u << lane) - 1u)), tot = 0;
#pragma unroll
    for (int k = 0; k < kSelWarps; ++k) { if (k < w) excl += sh.wtot[k]; tot += sh.wtot[k]; }
    if (ok) {
      const int pos = before0 + excl;                   // survivors with a lower index
      im.keep[i] = kp ? 1 : 0;
      if (im.keep_user) im.keep_user[i] = kp ? 1 : 0;
      if (kp) { im.kept_idx[pos] = i; im.slot[i] = pos; sh.own_tok[excl] = i; sh.own_slot[excl] = pos; }
      else { im.pruned_idx[i - pos] = i; im.slot[i] = -1 - (i - pos); }
    }
    __syncthreads();
    for (int e = w; e < tot; e += kSelWarps) {         // one warp per surviving row
      const int tok = sh.own_tok[e], rr = sh.own_slot[e];
      const uint4 *src = reinterpret_cast<const uint4 *>(Kc + (size_t)tok * im.ldKc);
      uint4 *dst = reinterpret_cast<uint4 *>(Kp + (size_t)rr * bt.d_k);
      for (int v0 = lane; v0 < nv; v0 += 128) {
        uint4 buf[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (v0 + 32 * u < nv) buf[u] = __ldg(src + v0 + 32 * u);
#pragma unroll
        for (int u = 0; u < 4; ++u)
          if (v0 + 32 * u < nv) dst[v0 + 32 * u] = buf[u];
      }
      if (lane == 0) rn_kept<D>(im)[rr] = rn_tok<D>(im)[tok];
    }
    before0 += tot;
    __syncthreads();                                    // own_tok / own_slot are rewritten by the next round
  }
}

template <typename T, int KPT, bool IN_SMEM>
__device__ __forceinline__ void euti_select(const Batch &bt, const ImgDesc &im, uint32_t *skey, int g, int tok0, int ntok,
                                            SelShared &sh) {
  const int t = threadIdx.x, N = im.N;
  uint32_t kreg[KPT > 0 ? KPT : 1];
  int hv[kHistPerThread];                               // bins [t kHistPerThread, (t + 1) kHistPerThread) of the histogram
  {
    const int4 *hp = reinterpret_cast<const int4 *>(im.ghist + t * kHistPerThread);
#pragma unroll
    for (int u = 0; u < kHistPerThread / 4; ++u) {
      const int4 x = __ldcg(hp + u);
      hv[4 * u] = x.x; hv[4 * u + 1] = x.y; hv[4 * u + 2] = x.z; hv[4 * u + 3] = x.w;
    }
  }
  if (KPT > 0) {
    float sc[KPT > 0 ? KPT : 1];
#pragma unroll
    for (int u = 0; u < (KPT > 0 ? KPT : 1); ++u) sc[u] = t + kSelThreads * u < N ? __ldcg(im.score + t + kSelThreads * u) : 0.f;
#pragma unroll
    for (int u = 0; u < (KPT > 0 ? KPT : 1); ++u) {
      kreg[u] = score_key(sc[u]);
      if (t + kSelThreads * u < N) skey[t + kSelThreads * u] = kreg[u];
    }
  } else if (IN_SMEM) {
    for (int i = t; i < N; i += kSelThreads) skey[i] = score_key(__ldcg(im.score + i));
  }
  // (the first barrier inside euti_threshold orders these stores before the first read)
  const uint32_t tau_key = euti_threshold<KPT, IN_SMEM>(im, skey, kreg, hv, sh);
  TL_POINT(im, 7);
  euti_compact<T, KPT, IN_SMEM>(bt, im, skey, kreg, tau_key, g, tok0, ntok, sh);
}

template <typename T>
__global__ void __launch_bounds__(kSelThreads, 2) k_select(const __grid_constant__ Batch bt, int keys_in_smem) {
  const ImgDesc &im = bt.img[blockIdx.y];
  TL_SCOPE(im, 3);
  pdl_wait();
  pdl_trigger();
  extern __shared__ uint32_t skey_dyn[];
  __shared__ SelShared sh;
  const int N = im.N, X = gridDim.x, x = blockIdx.x;
  const int tpc = (N + X - 1) / X;
  const int tok0 = min(N, x * tpc), ntok = min(N, tok0 + tpc) - tok0;
  if (keys_in_smem && N <= 16 * kSelThreads) euti_select<T, 16, true>(bt, im, skey_dyn, x, tok0, ntok, sh);
  else if (keys_in_smem) euti_select<T, 0, true>(bt, im, skey_dyn, x, tok0, ntok, sh);
  else euti_select<T, 0, false>(bt, im, skey_dyn, x, tok0, ntok, sh);
}

// ---- Eq. 3-4: order statistic, ordered compaction; survivor key gather ------------------------------

// grid (X, B), 1024 threads; dynamic smem: own_cap token indices, then (KPT == 0 and keys_in_smem) N keys.
// Every CTA computes the same threshold and the same list positions; CTA b writes the list entries of
// its block of tokens, and (do_gather) copies its block of survivor rows into Kp and their inverse
// norms into rnk, and clears its share of the arrays that later kernels accumulate into.
// KPT > 0: thread t keeps the keys of tokens [t KPT, t KPT + KPT) in registers (N <= 1024 KPT);
// KPT == 0: any N, keys in shared memory when they fit, else re-read from the scores.
template <typename T, int KPT>
__global__ void __launch_bounds__(1024) k_select_gather(const __grid_constant__ Batch bt, int do_gather,
                                                        int keys_in_smem, int own_cap) {
  using D = typename DistOf<T>::type;
  const ImgDesc &im = bt.img[blockIdx.y];
  TL_SCOPE(im, 3);
  const int t = threadIdx.x, lane = t & 31, w = t >> 5;
  const int N = im.N;
  extern __shared__ uint32_t dsm[];
  int *own = reinterpret_cast<int *>(dsm);                  // [own_cap]
  uint32_t *skey = dsm + own_cap;                           // [N] when KPT == 0 and keys_in_smem
  __shared__ int hist[256];
  __shared__ int warp_tot[32];
  __shared__ uint32_t wmin[32], wmax[32];
  __shared__ uint32_t s_prefix;
  __shared__ int s_k;
  constexpr int KR = KPT > 0 ? KPT : 1;
  const int CH = KPT > 0 ? KPT : (N + 1023) / 1024;         // tokens per thread, contiguous
  const int i0 = min(N, t * CH), i1 = min(N, i0 + CH);
  const int cnt_mine = i1 - i0;

  // keys of this thread's tokens
  uint32_t kreg[KR];
  if (KPT > 0) {
    float sc[KR];
#pragma unroll
    for (int j = 0; j < KR; ++j) sc[j] = j < cnt_mine ? __ldg(im.score + i0 + j) : 0.f;
#pragma unroll
    for (int j = 0; j < KR; ++j) kreg[j] = score_key(sc[j]);
  } else if (keys_in_smem) {
    for (int i = t; i < N; i += 1024) skey[i] = score_key(im.score[i]);
  }
  if (do_gather) {   // per-call initialisation, spread over the grid
    const int gt = blockIdx.x * 1024 + t, gs = gridDim.x * 1024;
    for (int r = gt; r < im.Np; r += gs) { im.rho_fix[r] = 0ull; im.csize[r] = 0; im.cticket[r] = 0; }
    for (int wd = gt; wd < im.Wp; wd += gs) { im.cmask[wd] = 0u; im.rmask[wd] = 0u; im.rtick[wd] = 0; }
    for (int i = gt; i < N; i += gs) im.best[i] = kBestInit;
    uint4 *tab = reinterpret_cast<uint4 *>(im.cnt_cb);
    const int nq = im.Np * (im.nbp / 8);
    for (int i = gt; i < nq; i += gs) tab[i] = make_uint4(0u, 0u, 0u, 0u);
  }
  if (t == 0) s_k = im.m_target;
  if (t < 256) hist[t] = 0;
  __syncthreads();
  // j-th key of this thread (j < cnt_mine)
  auto key = [&](int j) -> uint32_t {
    if (KPT > 0) return kreg[j < KR ? j : 0];
    return keys_in_smem ? skey[i0 + j] : score_key(im.score[i0 + j]);
  };

  // Keys are taken relative to the smallest one: that spreads them evenly over the digits of the first
  // pass (raw float bits of scores that span a few binades share most of their top bits), and the bits
  // above the highest one in which two keys differ need no pass.
  uint32_t kmin = 0xffffffffu, kmax = 0u;
  if (KPT > 0) {
#pragma unroll
    for (int j = 0; j < KR; ++j) if (j < cnt_mine) { kmin = min(kmin, kreg[j]); kmax = max(kmax, kreg[j]); }
  } else {
    for (int j = 0; j < cnt_mine; ++j) { const uint32_t kk = key(j); kmin = min(kmin, kk); kmax = max(kmax, kk); }
  }
  kmin = __reduce_min_sync(0xffffffffu, kmin);
  kmax = __reduce_max_sync(0xffffffffu, kmax);
  if (lane == 0) { wmin[w] = kmin; wmax[w] = kmax; }
  __syncthreads();
  kmin = __reduce_min_sync(0xffffffffu, wmin[lane]);
  kmax = __reduce_max_sync(0xffffffffu, wmax[lane]);
  const uint32_t kbase = kmin;
  const int top = 32 - __clz(kmax - kbase);                 // bits of the largest relative key (0: all keys equal)
  if (t == 0) s_prefix = 0u;
  __syncthreads();

  // radix select of the (m_target + 1)-th smallest key over the varying bits, up to 8 bits per pass
  for (int hi = top; hi > 0; hi -= 8) {
    const int lo = hi > 8 ? hi - 8 : 0;
    const uint32_t dmask = (1u << (hi - lo)) - 1u;
    const uint32_t above = hi >= 32 ? 0u : ~((1u << hi) - 1u);   // bits already fixed
    const uint32_t prefix = s_prefix;
    if (KPT > 0) {
#pragma unroll
      for (int j = 0; j < KR; ++j) {
        const uint32_t kk = kreg[j] - kbase;
        if (j < cnt_mine && (kk & above) == (prefix & above)) atomicAdd(&hist[(kk >> lo) & dmask], 1);
      }
    } else {
      for (int j = 0; j < cnt_mine; ++j) {
        const uint32_t kk = key(j) - kbase;
        if ((kk & above) == (prefix & above)) atomicAdd(&hist[(kk >> lo) & dmask], 1);
      }
    }
    __syncthreads();
    if (w == 0) {
      int c[8], s = 0;
#pragma unroll
      for (int b = 0; b < 8; ++b) { c[b] = hist[lane * 8 + b]; s += c[b]; }
      int incl = s;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
      }
      const int k = s_k;
      const unsigned has = __ballot_sync(0xffffffffu, incl > k);
      const int L = has ? __ffs(has) - 1 : 31;   // the candidates always number more than k
      if (lane == L) {
        int kk = k - (incl - s), dgt = 7;
        bool done = false;
#pragma unroll
        for (int b = 0; b < 7; ++b) {
          if (!done) {
            if (kk < c[b]) { dgt = b; done = true; }
            else kk -= c[b];
          }
        }
        s_k = kk;
        s_prefix = prefix | ((uint32_t)(lane * 8 + dgt) << lo);
      }
#pragma unroll
      for (int b = 0; b < 8; ++b) hist[lane * 8 + b] = 0;
    }
    __syncthreads();
  }
  const uint32_t tau_key = s_prefix + kbase;

  // ordered compaction over the contiguous blocks of tokens
  uint32_t keptbits = 0u;
  if (KPT > 0) {
#pragma unroll
    for (int j = 0; j < KR; ++j) if (j < cnt_mine && kreg[j] >= tau_key) keptbits |= 1u << j;
  } else {
    // more than 32 tokens per thread only beyond 32768 tokens: the bits are recomputed below then
    for (int j = 0; j < cnt_mine && j < 32; ++j) if (key(j) >= tau_key) keptbits |= 1u << j;
  }
  int mine = 0;
  if (KPT > 0 || CH <= 32) mine = __popc(keptbits);
  else for (int j = 0; j < cnt_mine; ++j) mine += key(j) >= tau_key;
  int incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) warp_tot[w] = incl;
  __syncthreads();
  if (w == 0) {
    const int v = warp_tot[lane];
    int x = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= o) x += y;
    }
    warp_tot[lane] = x - v;                                 // exclusive
    if (lane == 31) s_k = x;                                // q
  }
  __syncthreads();
  const int q = s_k;
  int before = warp_tot[w] + incl - mine;                   // survivors with a lower index
  const int tpc = (N + gridDim.x - 1) / gridDim.x;          // tokens whose list entries this CTA writes
  const int w0 = blockIdx.x * tpc, w1 = min(N, w0 + tpc);
  const int rpc = (q + gridDim.x - 1) / gridDim.x;          // survivor rows this CTA gathers
  const int g0 = min(q, (int)blockIdx.x * rpc), g1 = min(q, g0 + rpc);
  const bool touches = (i0 < w1 && i1 > w0) || (do_gather && before < g1 && before + mine > g0);
  if (touches) {
    for (int j = 0; j < cnt_mine; ++j) {
      const int i = i0 + j;
      const bool kp = (KPT > 0 || CH <= 32) ? ((keptbits >> j) & 1u) != 0u : key(j) >= tau_key;
      if (i >= w0 && i < w1) {
        im.keep[i] = kp ? 1 : 0;
        if (im.keep_user) im.keep_user[i] = kp ? 1 : 0;
        if (kp) { im.kept_idx[before] = i; im.slot[i] = before; }
        else { im.pruned_idx[i - before] = i; im.slot[i] = -1 - (i - before); }
      }
      if (kp) {
        if (do_gather && before >= g0 && before < g1 && before - g0 < own_cap) own[before - g0] = i;
        ++before;
      }
    }
  }
  if (blockIdx.x == 0 && t == 0) {
    im.cnt[PACT_CNT_Q] = q;
    im.cnt[PACT_CNT_M] = N - q;
  }
  if (!do_gather) return;
  __syncthreads();
  constexpr int V = Vec<T>::N;
  const int nv = bt.d_k / V;
  const T *Kc = reinterpret_cast<const T *>(im.Kc);
  T *Kp = reinterpret_cast<T *>(im.Kp);
  for (int rr = g0 + w; rr < g1; rr += 32) {
    const int tok = own[rr - g0];
    const uint4 *src = reinterpret_cast<const uint4 *>(Kc + (size_t)tok * im.ldKc);
    uint4 *dst = reinterpret_cast<uint4 *>(Kp + (size_t)rr * bt.d_k);
    for (int v0 = lane; v0 < nv; v0 += 128) {
      uint4 buf[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (v0 + 32 * u < nv) buf[u] = __ldg(src + v0 + 32 * u);
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (v0 + 32 * u < nv) dst[v0 + 32 * u] = buf[u];
    }
    if (lane == 0) rn_kept<D>(im)[rr] = rn_tok<D>(im)[tok];
  }
}

// ---- launchers -----------------------------------------------------------------------------

namespace {
int g_sm_count = 148;
size_t g_smem_optin = 48 * 1024;
constexpr size_t kSelectReserve = 4096;      // static shared memory of k_select_gather, rounded up
}  // namespace

static int qsum_row_blocks(int ncg, int B, int maxN) {
  // CTAs on 7/16 of the SMs (64 of 148) when that leaves a CTA no more than two rounds of loads (1024 rows),
  // else as many row blocks as that takes: see k_qsum
  int RP = g_sm_count * 7 / 16 / (ncg * B);
  const int need = (maxN + 1023) / 1024;
  if (RP < need) RP = need;
  return RP < 1 ? 1 : (RP > kQPartRows ? kQPartRows : RP);
}

template <typename T>
static cudaError_t launch_euti_t(const Batch &bt, int maxN, int mode, cudaStream_t st, StageMark mark, void *mark_arg) {
  constexpr int V = Vec<T>::N;
  const int ncg = (bt.n_qcols / V + 7) / 8;
  const int RP = qsum_row_blocks(ncg, bt.B, maxN);
  cudaError_t e = launch_k(k_qsum<T>, dim3(ncg * RP, bt.B), dim3(kQsumThreads), 0, st, false, bt, RP, mode == 0 ? 1 : 0);
  if (e != cudaSuccess) return e;
  if (mark && (e = mark(mark_arg)) != cudaSuccess) return e;
  const size_t sm_tok = (size_t)(bt.n_qcols + kRowsPerCta * bt.n_qh) * sizeof(double);
  e = launch_k(k_tokens<T>, dim3((maxN + kRowsPerCta - 1) / kRowsPerCta, bt.B), dim3(kTokThreads), sm_tok, st, true, bt);
  if (e != cudaSuccess) return e;
  if (mark && (e = mark(mark_arg)) != cudaSuccess) return e;
  e = launch_k(k_scores, dim3((maxN + 255) / 256, bt.B), dim3(256), 0, st, true, bt, mode == 0 ? 1 : 0);
  if (e != cudaSuccess) return e;
  if (mode == 0) {
    if (mark && (e = mark(mark_arg)) != cudaSuccess) return e;
    size_t keys = (size_t)maxN * sizeof(uint32_t);
    const int in_smem = keys <= 96 * 1024;
    if (!in_smem) keys = 0;
    int X = 2 * g_sm_count / bt.B;
    const int want = (maxN + 15) / 16;         // at least sixteen tokens per CTA
    if (X > want) X = want;
    if (X < 1) X = 1;
    e = launch_k(k_select<T>, dim3(X, bt.B), dim3(kSelThreads), keys, st, true, bt, in_smem);
    if (e != cudaSuccess) return e;
  }
  return cudaGetLastError();
}

cudaError_t launch_euti(const Batch &bt, int maxN, bool bf16, int mode, cudaStream_t st, StageMark mark, void *mark_arg) {
  return bf16 ? launch_euti_t<__nv_bfloat16>(bt, maxN, mode, st, mark, mark_arg)
              : launch_euti_t<float>(bt, maxN, mode, st, mark, mark_arg);
}

int euti_kernels(int mode) { return mode == 0 ? 4 : 3; }

template <typename T>
static void launch_select_t(const Batch &bt, int maxN, bool gather, cudaStream_t st) {
  int X = 1;
  if (gather) {
    X = g_sm_count / bt.B;
    if (X < 1) X = 1;
    const int cap = (maxN + 31) / 32;          // at least 32 survivor rows per CTA
    if (X > cap) X = cap;
  }
  const int own_cap = gather ? (maxN + X - 1) / X + 1 : 0;
  size_t sm = (size_t)own_cap * sizeof(int);
  dim3 grid(X, bt.B);
  const int g = gather ? 1 : 0;
  if (maxN <= 8 * 1024) k_select_gather<T, 8><<<grid, 1024, sm, st>>>(bt, g, 0, own_cap);
  else if (maxN <= 16 * 1024) k_select_gather<T, 16><<<grid, 1024, sm, st>>>(bt, g, 0, own_cap);
  else {
    const bool in_smem = sm + (size_t)maxN * 4 + kSelectReserve <= g_smem_optin;
    if (in_smem) sm += (size_t)maxN * 4;
    k_select_gather<T, 0><<<grid, 1024, sm, st>>>(bt, g, in_smem ? 1 : 0, own_cap);
  }
}

void launch_select_gather(const Batch &bt, int maxN, bool bf16, bool gather, cudaStream_t st) {
  if (bf16) launch_select_t<__nv_bfloat16>(bt, maxN, gather, st);
  else launch_select_t<float>(bt, maxN, gather, st);
}

cudaError_t select_configure() {
  int dev = 0, v = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  g_sm_count = v;
  e = cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e != cudaSuccess) return e;
  g_smem_optin = (size_t)v;
  const int dyn = (int)(g_smem_optin - kSelectReserve);
  e = cudaFuncSetAttribute(k_select_gather<__nv_bfloat16, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(k_select_gather<float, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn);
}

cudaError_t euti_configure(int n_qcols, int n_qh) {
  cudaError_t e = select_configure();
  if (e != cudaSuccess) return e;
  const size_t sm = (size_t)(n_qcols + kRowsPerCta * n_qh) * sizeof(double);
  if (sm > g_smem_optin - 1024) return cudaErrorInvalidConfiguration;
  e = cudaFuncSetAttribute(k_tokens<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(k_tokens<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
  if (e != cudaSuccess) return e;
  const int dyn = 96 * 1024;
  e = cudaFuncSetAttribute(k_select<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(k_select<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, dyn);
}

}  // namespace pact
