// DBDPC (Algorithm 2) and reincorporation (Eq. 8-9): key gather and inverse norms, all-pairs
// distance tiles with the density and the d <= d_c adjacency fused into their epilogue, density
// rank, centre selection, tokens-by-centres nearest-centre pass, labels.
//
// This file holds the SIMT tile kernels (any element type and key width); the tcgen05 tile
// kernels for bf16 keys live in gram_umma.cu and share the epilogue arithmetic of common.cuh.
#include <cooperative_groups.h>

#include "kernels.cuh"

namespace pact {

__device__ __forceinline__ uint32_t ld_relaxed_u32(const uint32_t *p) {
  uint32_t v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// ---- inverse key norms, survivor gather, per-call initialisation -----------------------------
// grid (ceil(maxN / 8), B), 256 threads, one warp per work item.
//  all_tokens = 1: item = token i (inverse norm of every token; survivors are copied to Kp[slot])
//  all_tokens = 0: item = list position r (token kept_idx[r]); only listed rows are touched
template <typename T>
__global__ void __launch_bounds__(256) k_keynorm_gather(const __grid_constant__ Batch bt, int all_tokens) {
  using D = typename DistOf<T>::type;
  using rn_t = typename D::rn_t;
  constexpr int V = Vec<T>::N;
  const ImgDesc &im = bt.img[blockIdx.y];
  const int lane = threadIdx.x & 31;
  const int item = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int q = all_tokens ? 0 : *im.q_ptr;
  // per-call initialisation of the arrays later kernels accumulate into
  {
    const int gt = blockIdx.x * 256 + threadIdx.x, gs = gridDim.x * 256;
    for (int r = gt; r < im.Np; r += gs) im.rho_fix[r] = 0ull;
    for (int wd = gt; wd < im.Wp; wd += gs) { im.cmask[wd] = 0u; im.rmask[wd] = 0u; }
    for (int i = gt; i < im.N; i += gs) {
      im.best[i] = kBestInit;
      if (!all_tokens) {
        im.label[i] = -1;
        if (im.label_user) im.label_user[i] = -1;
      }
    }
  }
  int i, r;
  if (all_tokens) {
    i = item;
    if (i >= im.N) return;
    r = im.slot[i];
  } else {
    r = item;
    if (r >= q) return;
    i = im.kept_idx[r];
  }
  const T *row = reinterpret_cast<const T *>(im.Kc) + (size_t)i * im.ldKc;
  const double ss = row_sumsq<T>(row, bt.d_k, lane);
  const rn_t rn = (rn_t)(1.0 / sqrt(fmax(ss, 1e-40)));
  if (lane == 0) {
    rn_tok<D>(im)[i] = rn;
    if (r >= 0) rn_kept<D>(im)[r] = rn;
  }
  if (r >= 0) {
    T *dst = reinterpret_cast<T *>(im.Kp) + (size_t)r * bt.d_k;
    for (int v = lane; v * V < bt.d_k; v += 32)
      reinterpret_cast<uint4 *>(dst)[v] = reinterpret_cast<const uint4 *>(row)[v];
  }
}

// centre keys from a list of token indices (reincorporation as a stage of its own)
template <typename T>
__global__ void __launch_bounds__(256) k_center_key_gather(const __grid_constant__ Batch bt) {
  using D = typename DistOf<T>::type;
  using rn_t = typename D::rn_t;
  constexpr int V = Vec<T>::N;
  const ImgDesc &im = bt.img[blockIdx.y];
  const int lane = threadIdx.x & 31;
  const int c = blockIdx.x * 8 + (threadIdx.x >> 5);
  {
    const int gt = blockIdx.x * 256 + threadIdx.x, gs = gridDim.x * 256;
    for (int i = gt; i < im.N; i += gs) im.best[i] = kBestInit;
  }
  if (c < *im.m_ptr) {                       // inverse norm of the c-th pruned row
    const int i = im.pruned_idx[c];
    const double ss = row_sumsq<T>(reinterpret_cast<const T *>(im.Kc) + (size_t)i * im.ldKc, bt.d_k, lane);
    if (lane == 0) rn_tok<D>(im)[i] = (rn_t)(1.0 / sqrt(fmax(ss, 1e-40)));
  }
  if (c >= *im.C_ptr) return;
  const int i = im.cidx_ptr[c];
  const T *row = reinterpret_cast<const T *>(im.Kc) + (size_t)i * im.ldKc;
  const double ss = row_sumsq<T>(row, bt.d_k, lane);
  if (lane == 0) rn_cen<D>(im)[c] = (rn_t)(1.0 / sqrt(fmax(ss, 1e-40)));
  T *dst = reinterpret_cast<T *>(im.Kcen) + (size_t)c * bt.d_k;
  for (int v = lane; v * V < bt.d_k; v += 32)
    reinterpret_cast<uint4 *>(dst)[v] = reinterpret_cast<const uint4 *>(row)[v];
}

// ---- 64 x 64 tile of dot products, 256 threads, thread (ty, tx) owns a 4 x 4 block -----------
constexpr int TS = 64;   // tile side
constexpr int KC = 32;   // key elements staged per step

template <typename T, typename acc_t, typename RowA, typename RowB>
__device__ __forceinline__ void tile_dots(RowA rowA, RowB rowB, int d_k, float (*As)[TS + 4],
                                          float (*Bs)[TS + 4], acc_t (&acc)[4][4]) {
  constexpr int V = Vec<T>::N;
  constexpr int VPR = KC / V;                 // vectors per row per step
  const int t = threadIdx.x, ty = t >> 4, tx = t & 15;
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = (acc_t)0;
  for (int k0 = 0; k0 < d_k; k0 += KC) {
    for (int v = t; v < TS * VPR; v += 256) {
      const int row = v / VPR, kv = (v % VPR) * V;
      float x[V], y[V];
      const T *pa = rowA(row), *pb = rowB(row);
      const bool inb = k0 + kv < d_k;
      if (pa && inb) load_vec<T>(pa + k0 + kv, x);
      else {
#pragma unroll
        for (int k = 0; k < V; ++k) x[k] = 0.f;
      }
      if (pb && inb) load_vec<T>(pb + k0 + kv, y);
      else {
#pragma unroll
        for (int k = 0; k < V; ++k) y[k] = 0.f;
      }
#pragma unroll
      for (int k = 0; k < V; ++k) { As[kv + k][row] = x[k]; Bs[kv + k][row] = y[k]; }
    }
    __syncthreads();
#pragma unroll 8
    for (int k = 0; k < KC; ++k) {
      const float4 a4 = *reinterpret_cast<const float4 *>(&As[k][ty * 4]);
      const float4 b4 = *reinterpret_cast<const float4 *>(&Bs[k][tx * 4]);
      const float a[4] = {a4.x, a4.y, a4.z, a4.w}, b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (sizeof(acc_t) == 8) acc[i][j] = fma((acc_t)a[i], (acc_t)b[j], acc[i][j]);
          else acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
    }
    __syncthreads();
  }
}

// ---- Eq. 5-6: all pairs of survivors; density and adjacency in the epilogue --------------------
// grid (n_ctas, B) persistent over the tiles of the q x q matrix; nothing of it is stored except
// one bit per pair (d <= d_c) and one integer density per row.
template <typename T>
__global__ void __launch_bounds__(256) k_gram_simt(const __grid_constant__ Batch bt) {
  using D = typename DistOf<T>::type;
  using acc_t = typename D::acc_t;
  const ImgDesc &im = bt.img[blockIdx.y];
  const int q = *im.q_ptr;
  const int nt = (q + TS - 1) / TS;
  const int t = threadIdx.x, ty = t >> 4, tx = t & 15;
  __shared__ __align__(16) float As[KC][TS + 4];
  __shared__ __align__(16) float Bs[KC][TS + 4];
  __shared__ unsigned long long rowsum[TS];
  __shared__ uint32_t adjw[TS][2];
  const T *Kp = reinterpret_cast<const T *>(im.Kp);
  const auto *rnk = rn_kept<D>(im);
  int band = 0;
  for (int tile = blockIdx.x; tile < nt * nt; tile += gridDim.x) {
    const int tm = tile / nt, tn = tile % nt;
    if (t < TS) { rowsum[t] = 0ull; adjw[t][0] = 0u; adjw[t][1] = 0u; }
    acc_t acc[4][4];
    tile_dots<T, acc_t>(
        [&](int r) { const int g = tm * TS + r; return g < q ? Kp + (size_t)g * bt.d_k : (const T *)nullptr; },
        [&](int r) { const int g = tn * TS + r; return g < q ? Kp + (size_t)g * bt.d_k : (const T *)nullptr; },
        bt.d_k, As, Bs, acc);
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      const int gi = tm * TS + ty * 4 + a;
      if (gi >= q) continue;
      const auto rni = rnk[gi];
      unsigned long long s = 0ull;
      uint32_t bits = 0u;
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int gj = tn * TS + tx * 4 + b;
        if (gj >= q) continue;
        auto dd = D::dist(acc[a][b], rni, rnk[gj]);
        if (gi == gj) dd = 0;
        s += D::term(dd, im);
        if (D::within(dd, im)) bits |= 1u << b;
        if (gi < gj && D::in_band(dd, im)) ++band;
      }
      atomicAdd(&rowsum[ty * 4 + a], s);
      if (bits) atomicOr(&adjw[ty * 4 + a][tx >> 3], bits << ((tx & 7) * 4));
    }
    __syncthreads();
    if (t < TS) {
      const int gi = tm * TS + t;
      if (gi < q) atomicAdd(&im.rho_fix[gi], rowsum[t]);
    } else if (t < 3 * TS) {
      const int r = (t - TS) >> 1, wd = (t - TS) & 1;
      const int gi = tm * TS + r;
      if (gi < q) im.adj[(size_t)gi * im.Wp + tn * 2 + wd] = adjw[r][wd];
    }
    __syncthreads();
  }
  if (band) atomicAdd(&im.cnt[PACT_CNT_BAND_DC], band);
}

// ---- choice of the reduction layer: largest distance between two keys of a layer ---------------
// Each image of the batch is one layer's key matrix (Kc, N rows).  Inverse norms first (one warp per
// key), then the tiles on and above the diagonal with a max-epilogue; the result accumulates in
// cnt[kCntSpread] as the bit pattern of a non-negative float.
template <typename T>
__global__ void __launch_bounds__(256) k_key_rnorm(const __grid_constant__ Batch bt) {
  using D = typename DistOf<T>::type;
  using rn_t = typename D::rn_t;
  const ImgDesc &im = bt.img[blockIdx.y];
  const int lane = threadIdx.x & 31;
  const int i = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (i >= im.N) return;
  const T *row = reinterpret_cast<const T *>(im.Kc) + (size_t)i * im.ldKc;
  const double ss = row_sumsq<T>(row, bt.d_k, lane);
  if (lane == 0) rn_tok<D>(im)[i] = (rn_t)(1.0 / sqrt(fmax(ss, 1e-40)));
}

template <typename T>
__global__ void __launch_bounds__(256) k_spread_simt(const __grid_constant__ Batch bt) {
  using D = typename DistOf<T>::type;
  using acc_t = typename D::acc_t;
  const ImgDesc &im = bt.img[blockIdx.y];
  const int N = im.N;
  const int nt = (N + TS - 1) / TS;
  const int t = threadIdx.x, ty = t >> 4, tx = t & 15;
  __shared__ __align__(16) float As[KC][TS + 4];
  __shared__ __align__(16) float Bs[KC][TS + 4];
  const T *K = reinterpret_cast<const T *>(im.Kc);
  const auto *rn = rn_tok<D>(im);
  float mx = 0.f;
  for (int tile = blockIdx.x; tile < nt * nt; tile += gridDim.x) {
    const int tm = tile / nt, tn = tile % nt;
    if (tn < tm) continue;                         // every unordered pair once (uniform)
    acc_t acc[4][4];
    tile_dots<T, acc_t>(
        [&](int r) { const int g = tm * TS + r; return g < N ? K + (size_t)g * im.ldKc : (const T *)nullptr; },
        [&](int r) { const int g = tn * TS + r; return g < N ? K + (size_t)g * im.ldKc : (const T *)nullptr; },
        bt.d_k, As, Bs, acc);
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      const int gi = tm * TS + ty * 4 + a;
      if (gi >= N) continue;
      const auto rni = rn[gi];
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int gj = tn * TS + tx * 4 + b;
        if (gj >= N || gj == gi) continue;
        mx = fmaxf(mx, (float)D::dist(acc[a][b], rni, rn[gj]));
      }
    }
  }
  const unsigned w = __reduce_max_sync(0xffffffffu, __float_as_uint(mx));   // distances are >= 0
  if ((t & 31) == 0 && w) atomicMax(reinterpret_cast<unsigned *>(&im.cnt[kCntSpread]), w);
}

// one warp: max_dist[l] of the layers of this batch, and the earliest layer at or above the threshold
__global__ void k_spread_finish(const __grid_constant__ Batch bt, float *max_dist, int32_t *layer_out,
                                int layer_base, float threshold) {
  const int l = threadIdx.x;
  float v = -1.f;
  if (l < bt.B) {
    v = __int_as_float(bt.img[l].cnt[kCntSpread]);
    max_dist[layer_base + l] = v;
  }
  const unsigned hit = __ballot_sync(0xffffffffu, l < bt.B && v >= threshold);
  if (l == 0 && layer_out) {
    if (layer_base == 0) *layer_out = -1;
    if (hit && *layer_out < 0) *layer_out = layer_base + (__ffs(hit) - 1);
  }
}

// ---- centre selection -------------------------------------------------------------------------
// The sequential loop of Algorithm 2 picks the lexicographically first maximal independent set of
// the graph {d_ij <= d_c} in density order (ties: lower index first); that set is unique, so any
// schedule that only takes final decisions reproduces it (the argument of Appendix D.2).  A row becomes
//   removed  once an earlier neighbour is a centre,
//   a centre once every earlier neighbour is removed.
// Both facts are monotone bits, so rows are resolved asynchronously from two bit masks in global memory.
// The masks are a few hundred bytes that every row depends on: thousands of warps polling them directly
// queue up at the same few L2 lines.  Instead a CTA copies both masks to shared memory once per sweep,
// its warps decide what they can from the copy and publish decisions with atomics; a decision reaches the
// other CTAs with their next copy.
//
// One cooperative kernel (every CTA resident), one CTA of 1024 threads per SM, three parts:
//  1. "earlier" is decided from the integer densities themselves (no rank array): the densities of an
//     image are staged in shared memory, each warp masks the adjacency words of its rows down to the
//     earlier neighbours (the first row's words stay in registers, further rows are written back);
//  2. sweeps (bounded) until no row of the CTA is pending;
//  3. after a grid-wide barrier: cluster ids (number of centres with a lower index), centre list,
//     centre keys and inverse norms.
constexpr int kAdjRegs = 8;      // adjacency words per lane kept in registers: rows of up to 8192 survivors
constexpr int kCenThreads = 1024;
constexpr int kCenWarps = kCenThreads / 32;

template <typename T>
__global__ void __launch_bounds__(kCenThreads, 1) k_centers(const __grid_constant__ Batch bt, int keys_cap, int mask_cap,
                                                            int spin_limit) {
  using D = typename DistOf<T>::type;
  constexpr int V = Vec<T>::N;
  cooperative_groups::grid_group grid = cooperative_groups::this_grid();
  TL_SCOPE(bt.img[0], 5);
  extern __shared__ unsigned long long skeys[];          // [keys_cap] densities of this CTA's image
  uint32_t *cm_s = reinterpret_cast<uint32_t *>(skeys + keys_cap);   // [mask_cap] copy of the centre mask
  uint32_t *rm_s = cm_s + mask_cap;                      // [mask_cap] copy of the removed mask
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  // The CTAs are shared out evenly among the images (the last image also takes the remainder); a CTA
  // works on one image throughout, so the images of a batch are resolved side by side.
  const int per = max(1, (int)gridDim.x / bt.B);
  const int b = min((int)blockIdx.x / per, bt.B - 1);
  const int ncta = b == bt.B - 1 ? (int)gridDim.x - per * (bt.B - 1) : per;
  const int nwarps = ncta * kCenWarps;
  const int gw = ((int)blockIdx.x - b * per) * kCenWarps + wid;
  const ImgDesc &im = bt.img[b];
  pdl_wait();
  pdl_trigger();
  const int q = *im.q_ptr, nw = (q + 31) >> 5;

  // part 1: keep only the neighbours that come earlier in density order
  uint32_t cached[kAdjRegs];
  int cached_item = -1;
  {
    const bool in_smem = q <= keys_cap;
    if (in_smem)
      for (int r = threadIdx.x; r < q; r += kCenThreads) skeys[r] = im.rho_fix[r];
    __syncthreads();
    const unsigned long long *keys = in_smem ? skeys : im.rho_fix;
    for (int r = gw; r < q; r += nwarps) {
      const unsigned long long mine = keys[r];
      uint32_t *row = im.adj + (size_t)r * im.Wp;
      const bool keep_regs = cached_item < 0 && nw <= 32 * kAdjRegs;
      uint32_t w_in[kAdjRegs];
#pragma unroll
      for (int u = 0; u < kAdjRegs; ++u) w_in[u] = (lane + 32 * u < nw) ? row[lane + 32 * u] : 0u;
#pragma unroll
      for (int u = 0; u < kAdjRegs; ++u) {
        const int wd = lane + 32 * u;
        uint32_t bits = w_in[u], out = 0u;
        while (bits) {
          const int bpos = __ffs(bits) - 1;
          bits &= bits - 1;
          const int j = wd * 32 + bpos;
          const unsigned long long o = keys[j];
          if (j != r && (o > mine || (o == mine && j < r))) out |= 1u << bpos;
        }
        if (wd < nw && !keep_regs) row[wd] = out;
        if (keep_regs) cached[u] = out;
      }
      for (int wd = lane + 32 * kAdjRegs; wd < nw; wd += 32) {     // rows longer than the register part
        uint32_t bits = row[wd], out = 0u;
        while (bits) {
          const int bpos = __ffs(bits) - 1;
          bits &= bits - 1;
          const int j = wd * 32 + bpos;
          const unsigned long long o = keys[j];
          if (j != r && (o > mine || (o == mine && j < r))) out |= 1u << bpos;
        }
        row[wd] = out;
      }
      if (keep_regs) cached_item = r;
      if (lane == 0) {
        const float rf = (float)((double)mine * (1.0 / (double)(1u << kRhoShift)));
        im.rho[r] = rf;
        if (im.rho_user) im.rho_user[r] = rf;
      }
    }
  }
  TL_POINT(bt.img[0], 10);

  // part 2: resolve
  const bool masks_in_smem = nw <= mask_cap;
  int sweeps = 0;
  bool cached_done = false;
  for (;;) {
    if (masks_in_smem) {
      __syncthreads();                                  // the previous sweep has read the copy
      for (int wd = threadIdx.x; wd < nw; wd += kCenThreads) {
        cm_s[wd] = ld_relaxed_u32(&im.cmask[wd]);
        rm_s[wd] = ld_relaxed_u32(&im.rmask[wd]);
      }
      __syncthreads();
    }
    const uint32_t *cmL = masks_in_smem ? cm_s : im.cmask, *rmL = masks_in_smem ? rm_s : im.rmask;
    auto ldm = [&](const uint32_t *p) { return masks_in_smem ? *p : ld_relaxed_u32(p); };
    int pending = 0;
    ++sweeps;
    for (int r = gw; r < q; r += nwarps) {
      const uint32_t mybit = 1u << (r & 31);
      bool hit_center = false, alive = false;
      if (r == cached_item) {                     // the masked adjacency of this row is in registers
        if (cached_done) continue;
#pragma unroll
        for (int u = 0; u < kAdjRegs; ++u) {
          if (cached[u] != 0u) {
            hit_center |= (cached[u] & ldm(&cmL[lane + 32 * u])) != 0u;
            alive |= (cached[u] & ~ldm(&rmL[lane + 32 * u])) != 0u;
          }
        }
      } else {
        if ((ldm(&cmL[r >> 5]) | ldm(&rmL[r >> 5])) & mybit) continue;   // decided
        const uint32_t *row = im.adj + (size_t)r * im.Wp;
        for (int wd = lane; wd < nw; wd += 32) {
          const uint32_t e = row[wd];
          if (e) {
            hit_center |= (e & ldm(&cmL[wd])) != 0u;
            alive |= (e & ~ldm(&rmL[wd])) != 0u;
          }
        }
      }
      hit_center = __any_sync(0xffffffffu, hit_center);
      alive = __any_sync(0xffffffffu, alive);
      if (hit_center) {
        if (lane == 0) atomicOr(&im.rmask[r >> 5], mybit);
        if (r == cached_item) cached_done = true;
      } else if (!alive) {
        if (lane == 0) atomicOr(&im.cmask[r >> 5], mybit);
        if (r == cached_item) cached_done = true;
      } else {
        pending = 1;
      }
    }
    if (!__syncthreads_or(pending)) break;              // no row of this CTA is pending
    if (sweeps >= spin_limit) {
      if (threadIdx.x == 0) atomicMin(&im.cnt[PACT_CNT_STATUS], (int)PACT_ERR_TIMEOUT);
      break;
    }
  }
  if (threadIdx.x == 0 && gw < q) atomicMax(&im.cnt[PACT_CNT_SWEEPS], sweeps);

  // part 3: every decision is final once all CTAs are here
  TL_POINT(bt.img[0], 11);
  __threadfence();
  grid.sync();
  TL_POINT(bt.img[0], 12);
  // Cluster id of a centre = number of centres with a lower index.  The centre mask of an image is read
  // once per CTA into shared memory with its running bit counts; images too large for the staging buffer
  // take the words from global memory.
  __shared__ int wsum3[kCenWarps];
  __shared__ int s_carry3;
  {
    const bool staged = q <= keys_cap;              // nw words and nw counts fit where the densities were
    uint32_t *cm = reinterpret_cast<uint32_t *>(skeys);
    int *pref = reinterpret_cast<int *>(skeys) + nw;
    __syncthreads();
    if (staged) {
      if (threadIdx.x == 0) s_carry3 = 0;
      __syncthreads();
      for (int base = 0; base < nw; base += kCenThreads) {
        const int wd = base + threadIdx.x;
        const uint32_t m = wd < nw ? __ldcg(&im.cmask[wd]) : 0u;
        const int pc = __popc(m);
        int x = pc;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int y = __shfl_up_sync(0xffffffffu, x, o);
          if (lane >= o) x += y;
        }
        if (lane == 31) wsum3[wid] = x;
        __syncthreads();
        int off = s_carry3;
        for (int k = 0; k < wid; ++k) off += wsum3[k];
        if (wd < nw) { cm[wd] = m; pref[wd] = off + x - pc; }
        __syncthreads();
        if (threadIdx.x == kCenThreads - 1) s_carry3 = off + x;
        __syncthreads();
      }
    }
    for (int r = gw; r < q; r += nwarps) {
      int c, all;
      bool is_center;
      if (staged) {
        const uint32_t m = cm[r >> 5];
        is_center = ((m >> (r & 31)) & 1u) != 0u;
        c = pref[r >> 5] + __popc(m & ((1u << (r & 31)) - 1u));
        all = s_carry3;
      } else {
        int below = 0;
        all = 0;
        uint32_t myword = 0u;
        for (int wd = lane; wd < nw; wd += 32) {
          const uint32_t m = __ldcg(&im.cmask[wd]);
          const int pc = __popc(m);
          all += pc;
          if (wd < (r >> 5)) below += pc;
          else if (wd == (r >> 5)) { below += __popc(m & ((1u << (r & 31)) - 1u)); myword = m; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          below += __shfl_xor_sync(0xffffffffu, below, o);
          all += __shfl_xor_sync(0xffffffffu, all, o);
          myword |= __shfl_xor_sync(0xffffffffu, myword, o);
        }
        c = below;
        is_center = ((myword >> (r & 31)) & 1u) != 0u;
      }
      if (r == 0 && lane == 0) {
        im.cnt[PACT_CNT_C] = all;
        if (im.C_user) *im.C_user = all;
      }
      if (!is_center) continue;
      const T *src = reinterpret_cast<const T *>(im.Kp) + (size_t)r * bt.d_k;
      const int nv = bt.d_k / V;
      uint4 buf[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (lane + 32 * u < nv) buf[u] = __ldcg(reinterpret_cast<const uint4 *>(src) + lane + 32 * u);
      if (lane == 0) {
        const int tok = im.kept_idx[r];
        im.cid[r] = c;
        im.center_idx[c] = tok;
        if (im.center_idx_user) im.center_idx_user[c] = tok;
        rn_cen<D>(im)[c] = rn_kept<D>(im)[r];
      }
      uint4 *dst = reinterpret_cast<uint4 *>(reinterpret_cast<T *>(im.Kcen) + (size_t)c * bt.d_k);
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (lane + 32 * u < nv) dst[lane + 32 * u] = buf[u];
      for (int v = lane + 128; v < nv; v += 32) dst[v] = __ldcg(reinterpret_cast<const uint4 *>(src) + v);
    }
  }
}

// ---- nearest centre of every row (Algorithm 2 assignment; Eq. 8 argmin) ---------------------------
// grid (n_ctas, B) persistent over 64 x 64 tiles of rows x centres; the running minimum of a row
// is one 64-bit word (distance bits, cluster id) reduced with atomicMin, so ties go to the lower id.
template <typename T>
__global__ void __launch_bounds__(256) k_assign_simt(const __grid_constant__ Batch bt, int mode) {
  using D = typename DistOf<T>::type;
  using acc_t = typename D::acc_t;
  const ImgDesc &im = bt.img[blockIdx.y];
  const int C = *im.C_ptr;
  const int nrows = mode == ROWS_ALL ? im.N : (mode == ROWS_KEPT_LIST ? *im.q_ptr : *im.m_ptr);
  const int32_t *list = mode == ROWS_KEPT_LIST ? im.kept_idx : im.pruned_idx;
  const int ntm = (nrows + TS - 1) / TS, ntn = (C + TS - 1) / TS;
  const int t = threadIdx.x, ty = t >> 4, tx = t & 15;
  __shared__ __align__(16) float As[KC][TS + 4];
  __shared__ __align__(16) float Bs[KC][TS + 4];
  __shared__ unsigned long long rowbest[TS];
  __shared__ int rowtok[TS];
  const T *Kc = reinterpret_cast<const T *>(im.Kc);
  const T *Kcen = reinterpret_cast<const T *>(im.Kcen);
  const auto *rnt = rn_tok<D>(im);
  const auto *rnc = rn_cen<D>(im);
  for (int tile = blockIdx.x; tile < ntm * ntn; tile += gridDim.x) {
    const int tm = tile / ntn, tn = tile % ntn;
    if (t < TS) {
      rowbest[t] = kBestInit;
      const int g = tm * TS + t;
      rowtok[t] = g < nrows ? (mode == ROWS_ALL ? g : list[g]) : -1;
    }
    __syncthreads();
    acc_t acc[4][4];
    tile_dots<T, acc_t>(
        [&](int r) { const int tok = rowtok[r]; return tok >= 0 ? Kc + (size_t)tok * im.ldKc : (const T *)nullptr; },
        [&](int r) { const int g = tn * TS + r; return g < C ? Kcen + (size_t)g * bt.d_k : (const T *)nullptr; },
        bt.d_k, As, Bs, acc);
#pragma unroll
    for (int a = 0; a < 4; ++a) {
      const int tok = rowtok[ty * 4 + a];
      if (tok < 0) continue;
      const auto rni = rnt[tok];
      unsigned long long bestv = kBestInit;
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const int c = tn * TS + tx * 4 + b;
        if (c >= C) continue;
        const float dd = (float)D::dist(acc[a][b], rni, rnc[c]);
        const unsigned long long pk = ((unsigned long long)__float_as_uint(dd) << 32) | (unsigned)c;
        bestv = pk < bestv ? pk : bestv;
      }
      atomicMin(&rowbest[ty * 4 + a], bestv);
    }
    __syncthreads();
    if (t < TS && rowtok[t] >= 0) atomicMin(&im.best[rowtok[t]], rowbest[t]);
    __syncthreads();
  }
}

// ---- labels -----------------------------------------------------------------------------------
// survivors: cluster id of the nearest centre (a centre: its own id); pruned tokens: that id iff
// the distance is strictly below alpha * d_c, else -1.
template <typename T>
__global__ void __launch_bounds__(256) k_label(const __grid_constant__ Batch bt, int mode) {
  using D = typename DistOf<T>::type;
  const ImgDesc &im = bt.img[blockIdx.y];
  TL_SCOPE(im, 7);
  const int nrows = mode == ROWS_ALL ? im.N : (mode == ROWS_KEPT_LIST ? *im.q_ptr : *im.m_ptr);
  int joined = 0, dropped = 0, band = 0;
  for (int g = blockIdx.x * 256 + threadIdx.x; g < nrows; g += gridDim.x * 256) {
    int tok, r;                                   // r >= 0: survivor position; < 0: pruned
    if (mode == ROWS_ALL) { tok = g; r = im.slot[g]; }
    else if (mode == ROWS_KEPT_LIST) { tok = im.kept_idx[g]; r = g; }
    else { tok = im.pruned_idx[g]; r = -1; }
    const unsigned long long pk = im.best[tok];
    int lab = (int)(pk & 0xFFFFFFFFull);
    const float dd = __uint_as_float((uint32_t)(pk >> 32));
    if (r >= 0) {
      if ((im.cmask[r >> 5] >> (r & 31)) & 1u) lab = im.cid[r];
    } else {
      if (D::in_band_t(dd, im)) ++band;
      if (D::below_t(dd, im)) ++joined; else { lab = -1; ++dropped; }
    }
    im.label[tok] = lab;
    if (im.label_user) im.label_user[tok] = lab;
  }
  // warp-aggregated counters
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    joined += __shfl_xor_sync(0xffffffffu, joined, o);
    dropped += __shfl_xor_sync(0xffffffffu, dropped, o);
    band += __shfl_xor_sync(0xffffffffu, band, o);
  }
  if ((threadIdx.x & 31) == 0) {
    if (joined) { atomicAdd(&im.cnt[PACT_CNT_R], joined); }
    if (dropped) atomicAdd(&im.cnt[PACT_CNT_DISCARDED], dropped);
    if (band) atomicAdd(&im.cnt[PACT_CNT_BAND_ADC], band);
  }
}

// ---- launchers ---------------------------------------------------------------------------------

cudaError_t cluster_configure(ClusterCfg *cfg) {
  int dev = 0, sms = 0, optin = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e != cudaSuccess) return e;
  cfg->sm_count = sms;
  cfg->centers_smem_max = optin - 1024;
  e = cudaFuncSetAttribute(k_centers<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, cfg->centers_smem_max);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(k_centers<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, cfg->centers_smem_max);
}

#define PACT_DISPATCH(bf16, KERNEL, ...)                       \
  do {                                                         \
    if (bf16) KERNEL<__nv_bfloat16> __VA_ARGS__;               \
    else KERNEL<float> __VA_ARGS__;                            \
  } while (0)

void launch_keynorm_gather(const Batch &bt, int maxN, bool bf16, bool all_tokens, cudaStream_t st) {
  dim3 grid((maxN + 7) / 8, bt.B);
  PACT_DISPATCH(bf16, k_keynorm_gather, <<<grid, 256, 0, st>>>(bt, all_tokens ? 1 : 0));
}

void launch_center_key_gather(const Batch &bt, int maxN, bool bf16, cudaStream_t st) {
  dim3 grid((maxN + 7) / 8, bt.B);
  PACT_DISPATCH(bf16, k_center_key_gather, <<<grid, 256, 0, st>>>(bt));
}

static int tile_grid(long long tiles, int cap) { return (int)(tiles < 1 ? 1 : (tiles > cap ? cap : tiles)); }

void launch_gram(const Batch &bt, int maxN, bool bf16, const ClusterCfg &cfg, cudaStream_t st) {
  const long long nt = (maxN + TS - 1) / TS;
  dim3 grid(tile_grid(nt * nt, cfg.sm_count * 8), bt.B);
  PACT_DISPATCH(bf16, k_gram_simt, <<<grid, 256, 0, st>>>(bt));
}

cudaError_t launch_centers(const Batch &bt, int maxQ, bool bf16, const ClusterCfg &cfg, int spin_limit, cudaStream_t st) {
  // the densities of one image are staged in shared memory when they fit in half of it; maxQ is an estimate of
  // the largest survivor count, an image with more reads them from global memory.  The two mask copies
  // take a word per 32 survivors each.
  const size_t budget = (size_t)cfg.centers_smem_max / 2;
  int keys_cap = (size_t)maxQ * sizeof(unsigned long long) <= budget ? maxQ : 0;
  int mask_cap = (maxQ + 31) / 32 + 1;
  if ((size_t)mask_cap * 8 > budget) mask_cap = 0;
  const size_t smem = (size_t)keys_cap * sizeof(unsigned long long) + (size_t)mask_cap * 8;
  int per_sm = 0;
  cudaError_t e = bf16 ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_centers<__nv_bfloat16>, kCenThreads, smem)
                       : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_centers<float>, kCenThreads, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorLaunchOutOfResources;
  return bf16 ? launch_coop(k_centers<__nv_bfloat16>, dim3(cfg.sm_count), dim3(kCenThreads), smem, st, true, bt, keys_cap, mask_cap, spin_limit)
              : launch_coop(k_centers<float>, dim3(cfg.sm_count), dim3(kCenThreads), smem, st, true, bt, keys_cap, mask_cap, spin_limit);
}

void launch_assign(const Batch &bt, int maxN, bool bf16, RowMode mode, const ClusterCfg &cfg, cudaStream_t st) {
  const long long nt = (maxN + TS - 1) / TS;
  dim3 grid(tile_grid(nt * nt, cfg.sm_count * 8), bt.B);
  PACT_DISPATCH(bf16, k_assign_simt, <<<grid, 256, 0, st>>>(bt, (int)mode));
}

void launch_key_rnorm(const Batch &bt, int maxN, bool bf16, cudaStream_t st) {
  dim3 grid((maxN + 7) / 8, bt.B);
  PACT_DISPATCH(bf16, k_key_rnorm, <<<grid, 256, 0, st>>>(bt));
}

void launch_spread(const Batch &bt, int maxN, bool bf16, const ClusterCfg &cfg, cudaStream_t st) {
  const long long nt = (maxN + TS - 1) / TS;
  dim3 grid(tile_grid(nt * (nt + 1) / 2, cfg.sm_count * 8), bt.B);
  PACT_DISPATCH(bf16, k_spread_simt, <<<grid, 256, 0, st>>>(bt));
}

void launch_spread_finish(const Batch &bt, float *max_dist, int32_t *layer_out, int layer_base, float threshold,
                          cudaStream_t st) {
  k_spread_finish<<<1, 32, 0, st>>>(bt, max_dist, layer_out, layer_base, threshold);
}

void launch_label(const Batch &bt, int maxN, bool bf16, RowMode mode, cudaStream_t st) {
  dim3 grid(tile_grid((maxN + 255) / 256, 1 << 16), bt.B);
  PACT_DISPATCH(bf16, k_label, <<<grid, 256, 0, st>>>(bt, (int)mode));
}

}  // namespace pact
