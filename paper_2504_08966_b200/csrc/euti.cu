// EUTI (Algorithm 1): global query, per-head softmax over the visual tokens, hidden-state norm,
// percentile split.  All accumulations that decide an ordering are carried in double so that the
// float32 score the library returns is the correctly rounded value in all but rare cases.
#include "kernels.cuh"

namespace pact {

__device__ __forceinline__ double ld_cg_f64(const double *p) {
  double v;
  asm volatile("ld.global.cg.f64 %0, [%1];" : "=d"(v) : "l"(p));
  return v;
}

// ---- Eq. 1: column sums of Q ---------------------------------------------------------------
// grid (G, B), 256 threads; CTA g of image b reduces rows [32g, 32g+32) and the last CTA to
// finish adds the partial sums in a fixed order.
template <typename T>
__global__ void __launch_bounds__(256) k_qsum(const __grid_constant__ Batch bt) {
  const ImgDesc &im = bt.img[blockIdx.y];
  constexpr int V = Vec<T>::N;
  const int g = blockIdx.x, t = threadIdx.x;
  const int G = (im.N + kRowsPerCta - 1) / kRowsPerCta;
  if (g >= G) return;
  const int r0 = g * kRowsPerCta, r1 = min(im.N, r0 + kRowsPerCta);
  const int ncolv = bt.n_qcols / V;
  const int cpp = min(ncolv, 256);          // column vectors per pass
  const int groups = 256 / cpp;
  __shared__ double sm[256 * V];
  const T *Q = reinterpret_cast<const T *>(im.Q);
  for (int cbase = 0; cbase < ncolv; cbase += cpp) {
    const int c = t % cpp, gi = t / cpp;
    double acc[V];
#pragma unroll
    for (int k = 0; k < V; ++k) acc[k] = 0.0;
    if (gi < groups && cbase + c < ncolv) {
      for (int r = r0 + gi; r < r1; r += groups) {
        float x[V];
        load_vec<T>(Q + (size_t)r * im.ldQ + (size_t)(cbase + c) * V, x);
#pragma unroll
        for (int k = 0; k < V; ++k) acc[k] += (double)x[k];
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
  if (t == 0) last = (atomicAdd(&im.cnt[16], 1) == G - 1);
  __syncthreads();
  if (!last) return;
  __threadfence();
  for (int col = t; col < bt.n_qcols; col += 256) {
    double s = 0.0;
    for (int h = 0; h < G; ++h) s += ld_cg_f64(&im.qpart[(size_t)h * bt.n_qcols + col]);
    im.qg[col] = s / (double)im.N;
  }
  if (t == 0) im.cnt[16] = 0;
}

// ---- Eq. 2, first half: logits, CTA-local softmax pieces, hidden-state norms -----------------
// grid (G, B), 256 threads, dynamic smem (n_qcols + 32 n_qh) doubles.  One warp per token.
template <typename T>
__global__ void __launch_bounds__(256) k_logit_norm(const __grid_constant__ Batch bt) {
  const ImgDesc &im = bt.img[blockIdx.y];
  constexpr int V = Vec<T>::N;
  const int g = blockIdx.x, t = threadIdx.x, lane = t & 31, w = t >> 5;
  const int G = (im.N + kRowsPerCta - 1) / kRowsPerCta;
  if (g >= G) return;
  extern __shared__ double smd[];
  double *qg = smd;                       // [n_qcols]
  double *lg = smd + bt.n_qcols;          // [32][n_qh]
  const int n_qh = bt.n_qh, d_h = bt.d_h;
  for (int c = t; c < bt.n_qcols; c += 256) qg[c] = ld_cg_f64(&im.qg[c]);
  __syncthreads();
  const int r0 = g * kRowsPerCta, r1 = min(im.N, r0 + kRowsPerCta);
  const T *H = reinterpret_cast<const T *>(im.H);
  const T *K = reinterpret_cast<const T *>(im.Ke);
  const bool use_norm = !(im.flags & PACT_FLAG_NO_NORM);
  const bool use_query = !(im.flags & PACT_FLAG_NORM_ONLY);
  for (int r = r0 + w; r < r1; r += 8) {
    double nn = 1.0;
    if (use_norm) nn = sqrt(row_sumsq<T>(H + (size_t)(im.vis_start + r) * im.ldH, bt.d, lane));
    if (lane == 0) im.nrm[r] = nn;
    for (int j = 0; j < n_qh; ++j) {
      double acc = 0.0;
      if (use_query) {
        const int kv = (j * bt.n_kvh) / n_qh;
        const T *kr = K + (size_t)r * im.ldKe + (size_t)kv * d_h;
        const double *qr = qg + (size_t)j * d_h;
        for (int v = lane; v * V < d_h; v += 32) {
          float x[V];
          load_vec<T>(kr + v * V, x);
#pragma unroll
          for (int k = 0; k < V; ++k) acc = fma((double)x[k], qr[v * V + k], acc);
        }
        acc = warp_sum(acc);
      }
      if (lane == 0) lg[(r - r0) * n_qh + j] = acc;
    }
  }
  __syncthreads();
  // per head: CTA max, exp, CTA sum; lane = token within the CTA
  for (int j = w; j < n_qh; j += 8) {
    const int r = r0 + lane;
    const bool ok = r < r1;
    double l = ok ? lg[lane * n_qh + j] : -1.0e300;
    double m = l;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
    double e = ok ? exp(l - m) : 0.0;
    if (ok) im.E[(size_t)r * n_qh + j] = e;
    double s = warp_sum(e);
    if (lane == 0) {
      im.part[((size_t)g * n_qh + j) * 2] = m;
      im.part[((size_t)g * n_qh + j) * 2 + 1] = s;
    }
  }
  __shared__ int last;
  __shared__ double red[8];
  __threadfence();
  __syncthreads();
  if (t == 0) last = (atomicAdd(&im.cnt[17], 1) == G - 1);
  __syncthreads();
  if (!last) return;
  __threadfence();
  // merge the CTA pieces in a fixed order: M = max, Z = sum S_g exp(M_g - M)
  for (int j = 0; j < n_qh; ++j) {
    double m = -1.0e300;
    for (int h = t; h < G; h += 256) m = fmax(m, ld_cg_f64(&im.part[((size_t)h * n_qh + j) * 2]));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmax(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) red[w] = m;
    __syncthreads();
    m = red[0];
    for (int k = 1; k < 8; ++k) m = fmax(m, red[k]);
    __syncthreads();
    double z = 0.0;
    for (int h = t; h < G; h += 256) {
      double wgt = exp(ld_cg_f64(&im.part[((size_t)h * n_qh + j) * 2]) - m);
      im.fac[(size_t)h * n_qh + j] = wgt;
      z += ld_cg_f64(&im.part[((size_t)h * n_qh + j) * 2 + 1]) * wgt;
    }
    z = warp_sum(z);
    if (lane == 0) red[w] = z;
    __syncthreads();
    z = 0.0;
    for (int k = 0; k < 8; ++k) z += red[k];
    __syncthreads();
    const double inv = 1.0 / (z * (double)n_qh);
    for (int h = t; h < G; h += 256) im.fac[(size_t)h * n_qh + j] *= inv;
  }
  if (t == 0) im.cnt[17] = 0;
}

// ---- Eq. 2 second half and Eq. 3-4: scores, order statistic, ordered compaction ---------------
// grid (1, B), 1024 threads.
__device__ __forceinline__ uint32_t score_key(float s) {
  uint32_t b = __float_as_uint(s);
  if (b == 0x80000000u) b = 0;                       // -0 orders as +0
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__global__ void __launch_bounds__(1024) k_score_select(const __grid_constant__ Batch bt, int do_score,
                                                       int do_select) {
  const ImgDesc &im = bt.img[blockIdx.y];
  const int t = threadIdx.x, lane = t & 31, w = t >> 5;
  const int N = im.N, n_qh = bt.n_qh;
  __shared__ int hist[256];
  __shared__ int warp_tot[32];
  __shared__ uint32_t s_prefix;
  __shared__ int s_k, s_running;
  if (do_score) {
    for (int i = t; i < N; i += 1024) {
      const int g = i / kRowsPerCta;
      double s = 0.0;
      for (int j = 0; j < n_qh; ++j) s = fma(im.E[(size_t)i * n_qh + j], im.fac[(size_t)g * n_qh + j], s);
      const float sf = (float)(s * im.nrm[i]);
      im.score[i] = sf;
      if (im.score_user) im.score_user[i] = sf;
    }
    __syncthreads();
  }
  if (!do_select) return;
  // radix select of the (m_target + 1)-th smallest key, most significant byte first
  if (t == 0) { s_prefix = 0; s_k = im.m_target; }
  uint32_t mask = 0;
  for (int pass = 3; pass >= 0; --pass) {
    const int shift = pass * 8;
    if (t < 256) hist[t] = 0;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    for (int i = t; i < N; i += 1024) {
      const uint32_t key = score_key(im.score[i]);
      if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255], 1);
    }
    __syncthreads();
    if (t == 0) {
      int k = s_k, dgt = 0;
      while (dgt < 255 && k >= hist[dgt]) { k -= hist[dgt]; ++dgt; }
      s_k = k;
      s_prefix = prefix | ((uint32_t)dgt << shift);
    }
    mask |= 255u << shift;
    __syncthreads();
  }
  const uint32_t tau_key = s_prefix;
  if (t == 0) s_running = 0;
  __syncthreads();
  for (int base = 0; base < N; base += 1024) {
    const int i = base + t;
    const bool kp = i < N && score_key(im.score[i]) >= tau_key;
    const unsigned bal = __ballot_sync(0xffffffffu, kp);
    if (lane == 0) warp_tot[w] = __popc(bal);
    __syncthreads();
    if (w == 0) {
      int v = warp_tot[lane], x = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int y = __shfl_up_sync(0xffffffffu, x, o);
        if (lane >= o) x += y;
      }
      warp_tot[lane] = x - v;                          // exclusive
      if (lane == 31) s_k = x;                         // kept in this chunk
    }
    __syncthreads();
    const int before = s_running + warp_tot[w] + __popc(bal & ((1u << lane) - 1u));
    if (i < N) {
      im.keep[i] = kp ? 1 : 0;
      if (im.keep_user) im.keep_user[i] = kp ? 1 : 0;
      if (kp) { im.kept_idx[before] = i; im.slot[i] = before; }
      else { im.pruned_idx[i - before] = i; im.slot[i] = -1 - (i - before); }
    }
    __syncthreads();
    if (t == 0) s_running += s_k;
    __syncthreads();
  }
  if (t == 0) {
    im.cnt[PACT_CNT_Q] = s_running;
    im.cnt[PACT_CNT_M] = N - s_running;
  }
}

// ---- launchers -----------------------------------------------------------------------------

void launch_qsum(const Batch &bt, int maxN, bool bf16, cudaStream_t st) {
  dim3 grid((maxN + kRowsPerCta - 1) / kRowsPerCta, bt.B);
  if (bf16) k_qsum<__nv_bfloat16><<<grid, 256, 0, st>>>(bt);
  else k_qsum<float><<<grid, 256, 0, st>>>(bt);
}

void launch_logit_norm(const Batch &bt, int maxN, bool bf16, cudaStream_t st) {
  dim3 grid((maxN + kRowsPerCta - 1) / kRowsPerCta, bt.B);
  const size_t sm = (size_t)(bt.n_qcols + kRowsPerCta * bt.n_qh) * sizeof(double);
  if (bf16) k_logit_norm<__nv_bfloat16><<<grid, 256, sm, st>>>(bt);
  else k_logit_norm<float><<<grid, 256, sm, st>>>(bt);
}

void launch_score_select(const Batch &bt, bool score, bool select, cudaStream_t st) {
  k_score_select<<<dim3(1, bt.B), 1024, 0, st>>>(bt, score ? 1 : 0, select ? 1 : 0);
}

size_t euti_smem_bytes(int n_qcols, int n_qh) {
  return (size_t)(n_qcols + kRowsPerCta * n_qh) * sizeof(double);
}

cudaError_t euti_configure(int n_qcols, int n_qh) {
  const size_t sm = euti_smem_bytes(n_qcols, n_qh);
  cudaError_t e = cudaFuncSetAttribute(k_logit_norm<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(k_logit_norm<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
}

}  // namespace pact
