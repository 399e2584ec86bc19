// EUTI (Algorithm 1): global query (Eq. 1), per-head softmax over the visual tokens and hidden-state
// norm (Eq. 2), percentile split (Eq. 3-4).  Every accumulation that decides an ordering is carried
// in double so that the float32 score the library returns is the correctly rounded value in all but
// rare double-rounding cases.
//
//   k_prepass        one pass over Q, H and the clustering keys: column sums of Q -> global query,
//                    hidden-state norms, inverse key norms (HBM-bound, the first of two reads of H)
//   k_logits         k_i . Qglobal per head, CTA-local softmax pieces (max, sum of exp)
//   k_scores         merges the pieces, writes the float32 scores
//   k_select_gather  every CTA selects the threshold and compacts (identical results in every CTA),
//                    then writes its share of the lists and gathers its share of the survivor keys
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

constexpr int kPreThreads = 256;              // two CTAs per SM: one loads while the other reduces
constexpr int kTokWarps = kPreThreads / 32;   // tokens per CTA of the token part of k_prepass
constexpr int kQCtasMax = kQPartRows;         // CTAs that reduce Q

// ---- Eq. 1 and the norms -----------------------------------------------------------------------
// grid (GQ + ceil(maxN / 8), B), 256 threads, two CTAs per SM (on batches a third faster than one CTA of
// 512 threads, whose load and reduce phases leave the memory pipe idle in turn; the same on one image).
//  CTAs [0, GQ): column sums of a contiguous block of rows of Q; the last of them to finish adds
//                the GQ partial sums in index order and writes the global query.
//  other CTAs:   one warp per visual token (8 tokens per CTA); every 16-byte load of the token's clustering-key row and
//                hidden-state row is issued before the first is used: |h_i| (double) and 1 / |k_i|.
// (A variant that streamed the rows through a shared-memory ring with bulk copies measured the same on
// one image and worse on batches: bulk copies issued row by row complete at about 20 GB/s per SM.)
template <typename T>
__global__ void __launch_bounds__(kPreThreads, 2) k_prepass(const __grid_constant__ Batch bt, int GQ) {
  using D = typename DistOf<T>::type;
  using rn_t = typename D::rn_t;
  constexpr int V = Vec<T>::N;
  const ImgDesc &im = bt.img[blockIdx.y];
  TL_SCOPE(im, 0);
  const int t = threadIdx.x, lane = t & 31, w = t >> 5;
  if ((int)blockIdx.x >= GQ) {
    const int tok = ((int)blockIdx.x - GQ) * kTokWarps + w;
    if (tok >= im.N) return;
    constexpr int UK = 4;
    const T *krow = im.Kc ? reinterpret_cast<const T *>(im.Kc) + (size_t)tok * im.ldKc : nullptr;
    const int nvk = krow ? bt.d_k / V : 0;
    uint4 kb[UK];
#pragma unroll
    for (int u = 0; u < UK; ++u)
      if (lane + 32 * u < nvk) kb[u] = __ldg(reinterpret_cast<const uint4 *>(krow) + lane + 32 * u);
    if (im.H) {
      double nn = 1.0;
      if (!(im.flags & PACT_FLAG_NO_NORM)) {
        const T *hrow = reinterpret_cast<const T *>(im.H) + (size_t)(im.vis_start + tok) * im.ldH;
        nn = sqrt(warp_sum(row_sumsq_lane<T, 16, true>(hrow, bt.d, lane, 0, policy_evict_last())));
      }
      if (lane == 0) im.nrm[tok] = nn;
    }
    if (krow) {
      double acc = 0.0;
#pragma unroll
      for (int u = 0; u < UK; ++u)
        if (lane + 32 * u < nvk) sumsq_accumulate<T>(kb[u], acc);
      if (nvk > 32 * UK) acc += row_sumsq_lane<T, 8>(krow, bt.d_k, lane, 32 * UK);
      const double ss = warp_sum(acc);
      if (lane == 0) rn_tok<D>(im)[tok] = (rn_t)(1.0 / sqrt(fmax(ss, 1e-40)));
    }
    return;
  }
  if (!im.Q) return;
  const int g = blockIdx.x;
  const int chunk = (im.N + GQ - 1) / GQ;
  const int r0 = min(im.N, g * chunk), r1 = min(im.N, r0 + chunk);
  const int ncolv = bt.n_qcols / V;
  const int cpp = min(ncolv, kPreThreads);   // column vectors per pass
  const int groups = kPreThreads / cpp;      // row groups per pass
  __shared__ double sm[kPreThreads * V];
  const T *Q = reinterpret_cast<const T *>(im.Q);
  const int c = t % cpp, gi = t / cpp;
  constexpr int UQ = 16;
  for (int cbase = 0; cbase < ncolv; cbase += cpp) {
    double acc[V];
#pragma unroll
    for (int k = 0; k < V; ++k) acc[k] = 0.0;
    if (gi < groups && cbase + c < ncolv) {
      const size_t coff = (size_t)(cbase + c) * V;
      for (int r = r0 + gi; r < r1; r += groups * UQ) {
        uint4 buf[UQ];
#pragma unroll
        for (int u = 0; u < UQ; ++u)
          if (r + u * groups < r1) buf[u] = __ldg(reinterpret_cast<const uint4 *>(Q + (size_t)(r + u * groups) * im.ldQ + coff));
#pragma unroll
        for (int u = 0; u < UQ; ++u) {
          if (r + u * groups < r1) {
            float x[V];
            widen_vec<T>(buf[u], x);
#pragma unroll
            for (int k = 0; k < V; ++k) acc[k] += (double)x[k];
          }
        }
      }
    }
#pragma unroll
    for (int k = 0; k < V; ++k) sm[t * V + k] = acc[k];
    __syncthreads();
    if (gi == 0 && cbase + c < ncolv) {
#pragma unroll
      for (int k = 0; k < V; ++k) {
        double s = 0.0;
        for (int h = 0; h < groups; ++h) s += sm[(h * cpp + c) * V + k];
        im.qpart[(size_t)g * bt.n_qcols + (size_t)(cbase + c) * V + k] = s;
      }
    }
    __syncthreads();
  }
  __shared__ int last;
  __threadfence();
  __syncthreads();
  if (t == 0) last = (atomicAdd(&im.cnt[16], 1) == GQ - 1);
  __syncthreads();
  if (!last) return;
  __threadfence();
  for (int col = t; col < bt.n_qcols; col += 2 * kPreThreads) {   // two columns per thread at a time
    const int col2 = col + kPreThreads;
    const bool two = col2 < bt.n_qcols;
    double s = 0.0, s2 = 0.0;
    for (int h0 = 0; h0 < GQ; h0 += 16) {            // 2 x 16 partial sums in flight, added in index order
      double v[16], v2[16];
#pragma unroll
      for (int u = 0; u < 16; ++u) {
        v[u] = h0 + u < GQ ? ld_cg_f64(&im.qpart[(size_t)(h0 + u) * bt.n_qcols + col]) : 0.0;
        v2[u] = (two && h0 + u < GQ) ? ld_cg_f64(&im.qpart[(size_t)(h0 + u) * bt.n_qcols + col2]) : 0.0;
      }
#pragma unroll
      for (int u = 0; u < 16; ++u) { s += v[u]; s2 += v2[u]; }
    }
    im.qg[col] = s / (double)im.N;
    if (two) im.qg[col2] = s2 / (double)im.N;
  }
  if (t == 0) im.cnt[16] = 0;
}

// ---- Eq. 2, first half: logits and CTA-local softmax pieces ---------------------------------------
// grid (ceil(maxN / 32), B), 256 threads, dynamic smem (n_qcols + 32 n_qh) doubles.  A CTA takes 32
// tokens, a warp four of them: their key rows are loaded at once, then every head takes its part.
constexpr int kLogitThreads = 256;
constexpr int kLogitTpw = kRowsPerCta / (kLogitThreads / 32);   // tokens per warp

template <typename T>
__global__ void __launch_bounds__(kLogitThreads) k_logits(const __grid_constant__ Batch bt) {
  const ImgDesc &im = bt.img[blockIdx.y];
  TL_SCOPE(im, 1);
  constexpr int V = Vec<T>::N;
  constexpr int UK = 2;                   // preloaded 16-byte vectors per lane and token
  const int g = blockIdx.x, t = threadIdx.x, lane = t & 31, w = t >> 5;
  const int G = (im.N + kRowsPerCta - 1) / kRowsPerCta;
  if (g >= G) return;
  extern __shared__ double smd[];
  double *qg = smd;                       // [n_qcols], transposed (see below)
  double *lg = smd + bt.n_qcols;          // [32][n_qh]
  const int n_qh = bt.n_qh, d_h = bt.d_h;
  const int r0 = g * kRowsPerCta, r1 = min(im.N, r0 + kRowsPerCta);
  const bool use_query = !(im.flags & PACT_FLAG_NORM_ONLY);
  const int nv = bt.d_k / V;
  const T *K = reinterpret_cast<const T *>(im.Ke);
  uint4 kb[kLogitTpw][UK];
  if (use_query) {
#pragma unroll
    for (int i = 0; i < kLogitTpw; ++i) {
      const uint4 *krow = reinterpret_cast<const uint4 *>(K + (size_t)min(r0 + w * kLogitTpw + i, im.N - 1) * im.ldKe);
#pragma unroll
      for (int u = 0; u < UK; ++u)
        if (lane + 32 * u < nv) kb[i][u] = __ldg(krow + lane + 32 * u);
    }
  }
  // the global query is kept transposed, qT[k][vq] = Qglobal[vq * V + k], so that the lanes of a warp,
  // which hold consecutive 16-byte vectors of the key row, read consecutive doubles
  const int nvq = bt.n_qcols / V;
  for (int c = t; c < bt.n_qcols; c += kLogitThreads) qg[(c % V) * nvq + c / V] = im.qg[c];
  __syncthreads();
  const int vph = d_h / V;                                  // vectors per head
  for (int j = 0; j < n_qh; ++j) {
    // the tokens of this warp give independent chains of multiply-adds; their sums are reduced together
    double acc[kLogitTpw][UK];
#pragma unroll
    for (int i = 0; i < kLogitTpw; ++i)
#pragma unroll
      for (int u = 0; u < UK; ++u) acc[i][u] = 0.0;
    if (use_query) {
      const int kv = (j * bt.n_kvh) / n_qh;
      const int vshift = (j - kv) * vph;                    // key-row vector v pairs with query vector v + vshift
#pragma unroll
      for (int u = 0; u < UK; ++u) {
        const int v = lane + 32 * u;
        if (v < nv && v / vph == kv) {
          double qv[V];
#pragma unroll
          for (int k = 0; k < V; ++k) qv[k] = qg[k * nvq + v + vshift];
#pragma unroll
          for (int i = 0; i < kLogitTpw; ++i) {
            float x[V];
            widen_vec<T>(kb[i][u], x);
#pragma unroll
            for (int k = 0; k < V; ++k) acc[i][u] = fma((double)x[k], qv[k], acc[i][u]);
          }
        }
      }
      for (int v = lane + 32 * UK; v < nv; v += 32) {       // rows wider than the preloaded part
        if (v / vph == kv) {
#pragma unroll
          for (int i = 0; i < kLogitTpw; ++i) {
            const int rr = min(r0 + w * kLogitTpw + i, im.N - 1);
            float x[V];
            widen_vec<T>(__ldg(reinterpret_cast<const uint4 *>(K + (size_t)rr * im.ldKe) + v), x);
#pragma unroll
            for (int k = 0; k < V; ++k) acc[i][0] = fma((double)x[k], qg[k * nvq + v + vshift], acc[i][0]);
          }
        }
      }
    }
    double tot[kLogitTpw];
#pragma unroll
    for (int i = 0; i < kLogitTpw; ++i) {
      tot[i] = acc[i][0];
#pragma unroll
      for (int u = 1; u < UK; ++u) tot[i] += acc[i][u];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1)
#pragma unroll
      for (int i = 0; i < kLogitTpw; ++i) tot[i] += __shfl_xor_sync(0xffffffffu, tot[i], o);
    if (lane == 0) {
#pragma unroll
      for (int i = 0; i < kLogitTpw; ++i) lg[(w * kLogitTpw + i) * n_qh + j] = tot[i];
    }
  }
  __syncthreads();
  // per head: CTA max, exp, CTA sum; lane = token within the CTA
  for (int j = w; j < n_qh; j += kLogitThreads / 32) {
    const int rr = r0 + lane;
    const bool ok = rr < r1;
    const double l = ok ? lg[lane * n_qh + j] : -1.0e300;
    double m = l;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
    const double e = ok ? exp(l - m) : 0.0;
    if (ok) im.E[(size_t)rr * n_qh + j] = e;
    const double s = warp_sum(e);
    if (lane == 0) {
      im.part[((size_t)g * n_qh + j) * 2] = m;
      im.part[((size_t)g * n_qh + j) * 2 + 1] = s;
    }
  }
}

// ---- Eq. 2, second half: merge the pieces (M = max, Z = sum S_g exp(M_g - M), fixed order), scores --
// grid (ceil(maxN / 256), B), 256 threads.  Every CTA merges all pieces itself, one warp per head.
__global__ void __launch_bounds__(256) k_scores(const __grid_constant__ Batch bt) {
  const ImgDesc &im = bt.img[blockIdx.y];
  TL_SCOPE(im, 2);
  const int t = threadIdx.x, lane = t & 31, w = t >> 5;
  const int N = im.N, n_qh = bt.n_qh;
  if ((int)blockIdx.x * 256 >= N) return;
  const int G = (N + kRowsPerCta - 1) / kRowsPerCta;
  __shared__ double sM[256], sInv[256];
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
  for (int j = w; j < n_qh; j += 8) {
    const double *pj = im.part + (size_t)j * 2;
    const size_t stride = (size_t)n_qh * 2;
    double m = -1.0e300;
#pragma unroll 4
    for (int h = lane; h < G; h += 32) m = fmax(m, pj[(size_t)h * stride]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
    double z = 0.0;
#pragma unroll 4
    for (int h = lane; h < G; h += 32) z += pj[(size_t)h * stride + 1] * exp(pj[(size_t)h * stride] - m);
    z = warp_sum(z);
    if (lane == 0) { sM[j] = m; sInv[j] = 1.0 / (z * (double)n_qh); }
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
}

// ---- Eq. 3-4: order statistic, ordered compaction; survivor key gather ------------------------------
__device__ __forceinline__ uint32_t score_key(float s) {
  uint32_t b = __float_as_uint(s);
  if (b == 0x80000000u) b = 0;                       // -0 orders as +0
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

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
    for (int wd = gt; wd < im.Wp; wd += gs) { im.cmask[wd] = 0u; im.rmask[wd] = 0u; }
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

int q_ctas(int maxN) {
  const int g = (maxN + 63) / 64;
  return g < 1 ? 1 : (g > kQCtasMax ? kQCtasMax : g);
}
}  // namespace

void launch_prepass(const Batch &bt, int maxN, bool bf16, cudaStream_t st) {
  const int GQ = q_ctas(maxN);
  dim3 grid(GQ + (maxN + kTokWarps - 1) / kTokWarps, bt.B);
  if (bf16) k_prepass<__nv_bfloat16><<<grid, kPreThreads, 0, st>>>(bt, GQ);
  else k_prepass<float><<<grid, kPreThreads, 0, st>>>(bt, GQ);
}

void launch_logits(const Batch &bt, int maxN, bool bf16, cudaStream_t st) {
  dim3 grid((maxN + kRowsPerCta - 1) / kRowsPerCta, bt.B);
  const size_t sm = (size_t)(bt.n_qcols + kRowsPerCta * bt.n_qh) * sizeof(double);
  if (bf16) k_logits<__nv_bfloat16><<<grid, kLogitThreads, sm, st>>>(bt);
  else k_logits<float><<<grid, kLogitThreads, sm, st>>>(bt);
}

void launch_scores(const Batch &bt, int maxN, cudaStream_t st) {
  k_scores<<<dim3((maxN + 255) / 256, bt.B), 256, 0, st>>>(bt);
}

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
  if (sm > g_smem_optin) return cudaErrorInvalidConfiguration;
  e = cudaFuncSetAttribute(k_logits<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(k_logits<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
}

}  // namespace pact
