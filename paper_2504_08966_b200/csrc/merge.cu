// Merge (Eq. 10, Algorithm 3 step 4): one hidden state per cluster = mean of its members in
// float accumulation and ascending token order; position id of the centre; cluster sizes;
// text rows copied around the merged span.
#include "kernels.cuh"
#include "tma.cuh"

namespace pact {

template <typename O> __device__ __forceinline__ void store_vec8(O *p, const float (&x)[8]);
template <> __device__ __forceinline__ void store_vec8<float>(float *p, const float (&x)[8]) {
  reinterpret_cast<float4 *>(p)[0] = make_float4(x[0], x[1], x[2], x[3]);
  reinterpret_cast<float4 *>(p)[1] = make_float4(x[4], x[5], x[6], x[7]);
}
template <> __device__ __forceinline__ void store_vec8<__nv_bfloat16>(__nv_bfloat16 *p, const float (&x)[8]) {
  uint32_t w[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 h = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
    w[i] = *reinterpret_cast<uint32_t *>(&h);
  }
  *reinterpret_cast<uint4 *>(p) = make_uint4(w[0], w[1], w[2], w[3]);
}

// Loads 8 consecutive elements as float (one or two 16-byte loads).
template <typename T> __device__ __forceinline__ void load8(const T *p, float (&x)[8]);
template <> __device__ __forceinline__ void load8<__nv_bfloat16>(const __nv_bfloat16 *p, float (&x)[8]) {
  load_vec<__nv_bfloat16>(p, x);
}
template <> __device__ __forceinline__ void load8<float>(const float *p, float (&x)[8]) {
  float a[4], b[4];
  load_vec<float>(p, a);
  load_vec<float>(p + 4, b);
#pragma unroll
  for (int i = 0; i < 4; ++i) { x[i] = a[i]; x[4 + i] = b[i]; }
}

// Eight consecutive elements of a row as loaded (not yet widened), so that many can be in flight.
template <typename T> struct Raw8;
template <> struct Raw8<__nv_bfloat16> {
  uint4 a;
  __device__ __forceinline__ void load(const __nv_bfloat16 *p) { a = __ldg(reinterpret_cast<const uint4 *>(p)); }
  __device__ __forceinline__ void add_to(float (&acc)[8]) const {
    float x[8];
    widen_vec<__nv_bfloat16>(a, x);
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] += x[e];
  }
};
template <> struct Raw8<float> {
  uint4 a, b;
  __device__ __forceinline__ void load(const float *p) {
    a = __ldg(reinterpret_cast<const uint4 *>(p));
    b = __ldg(reinterpret_cast<const uint4 *>(p) + 1);
  }
  __device__ __forceinline__ void add_to(float (&acc)[8]) const {
    float x[4], y[4];
    widen_vec<float>(a, x);
    widen_vec<float>(b, y);
#pragma unroll
    for (int e = 0; e < 4; ++e) { acc[e] += x[e]; acc[4 + e] += y[e]; }
  }
};

constexpr int kListBlock = 256;      // tokens per block of the member lists
constexpr int kChunk = 16;           // members summed by one work item; the chunk-sum scratch of the workspace
                                     // (N / 8 + 2 rows) is sized for this value: clusters of more than one chunk
                                     // have at most 0.118 N chunks between them

__device__ __forceinline__ int ld_cg_i32(const int *p) {
  int v;
  asm volatile("ld.global.cg.s32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ float4 ld_cg_f4(const float *p) {
  float4 v;
  asm volatile("ld.global.cg.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
}

// ---- member lists --------------------------------------------------------------------------------
// grid (ceil(maxN / 256), B), 256 threads.  Block b sorts its 256 tokens by (cluster id, token) into
// blocklist[b] (discarded tokens last) and writes bstart[b][c] = number of its tokens with a cluster id
// below c, for c = 0..C.  The members of cluster c are then, in ascending token order, the entries
// [bstart[b][c], bstart[b][c+1]) of blocklist[b] for b = 0, 1, ...  Cluster sizes are added up with
// integer atomics.
// FROM_BEST: the labels are first formed here from the nearest-centre pass (survivors: cluster id of the
// nearest centre, a centre its own id; pruned tokens: that id iff the distance is strictly below
// alpha * d_c, else -1) and written out; otherwise label[] is given.
template <typename T, bool FROM_BEST>
__global__ void __launch_bounds__(kListBlock) k_lists(const __grid_constant__ Batch bt) {
  using D = typename DistOf<T>::type;
  const ImgDesc &im = bt.img[blockIdx.y];
  TL_SCOPE(im, 8);
  const int N = im.N;
  const int nblk = (N + kListBlock - 1) / kListBlock;
  const int b = blockIdx.x, t = threadIdx.x;
  if (b >= nblk) return;
  __shared__ int slab[kListBlock], sorted_lab[kListBlock];
  const int i = b * kListBlock + t;
  int lab = -1;
  if (FROM_BEST) {
    int joined = 0, dropped = 0, band = 0;
    if (i < N) {
      const int r = im.slot[i];                     // >= 0: survivor position; < 0: pruned
      const unsigned long long pk = im.best[i];
      lab = (int)(pk & 0xFFFFFFFFull);
      const float dd = __uint_as_float((uint32_t)(pk >> 32));
      if (r >= 0) {
        if ((im.cmask[r >> 5] >> (r & 31)) & 1u) lab = im.cid[r];
      } else {
        if (D::in_band_t(dd, im)) ++band;
        if (D::below_t(dd, im)) ++joined; else { lab = -1; ++dropped; }
      }
      im.label[i] = lab;
      if (im.label_user) im.label_user[i] = lab;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      joined += __shfl_xor_sync(0xffffffffu, joined, o);
      dropped += __shfl_xor_sync(0xffffffffu, dropped, o);
      band += __shfl_xor_sync(0xffffffffu, band, o);
    }
    if ((t & 31) == 0) {
      if (joined) atomicAdd(&im.cnt[PACT_CNT_R], joined);
      if (dropped) atomicAdd(&im.cnt[PACT_CNT_DISCARDED], dropped);
      if (band) atomicAdd(&im.cnt[PACT_CNT_BAND_ADC], band);
    }
  } else {
    lab = i < N ? im.label[i] : -1;
  }
  const int C = *im.C_ptr;
  const int key = lab < 0 ? 0x7fffffff : lab;
  slab[t] = key;
  __syncthreads();
  int rank = 0;
#pragma unroll 8
  for (int u = 0; u < kListBlock; ++u) {
    const int o = slab[u];
    rank += (o < key) || (o == key && u < t);
  }
  sorted_lab[rank] = key;
  im.blocklist[(size_t)b * kListBlock + rank] = i;
  __syncthreads();
  // first position whose cluster id is >= c
  auto lower = [&](int c) {
    int lo = 0, hi = kListBlock;
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (sorted_lab[mid] < c) lo = mid + 1; else hi = mid;
    }
    return lo;
  };
  uint16_t *row = im.bstart + (size_t)b * im.bstride;
  for (int c = t; c <= C; c += kListBlock) row[c] = (uint16_t)lower(c);
  {
    const int c = sorted_lab[t];
    if (c != 0x7fffffff && (t == 0 || sorted_lab[t - 1] != c)) atomicAdd(&im.csize[c], lower(c + 1) - t);
  }
}

// ---- Eq. 10 ------------------------------------------------------------------------------------------
// Grid (X, B) with three CTAs of 256 threads per SM.  Work units are the chunks (kChunk members of one
// cluster, ascending token order) followed by the text rows; CTA x takes units x, x + X, ...  For a unit
// the CTA looks up the members (thread = block of the member lists), then every thread adds its columns
// of the member rows in float with kMrgRows rows in flight, divides and stores.  A cluster of one chunk
// is finished on the spot; otherwise the chunk sums go to scratch and the CTA that finishes the cluster's
// last chunk adds them in chunk order.  Plain 16-byte loads: many small CTAs keep enough of them in
// flight, and a CTA that waits on its look-up loads does not hold back the others.
constexpr int kMrgThreads = 256;
constexpr int kMrgRows = 4;                        // member rows in flight per thread
constexpr int kMrgVpl = kMergeMaxD / 8 / kMrgThreads;   // 8-column groups per thread at the widest d

template <typename T, typename O, int VPL>
__global__ void __launch_bounds__(kMrgThreads, (VPL <= 2 && sizeof(T) == 2) ? 3 : 1)
k_merge(const __grid_constant__ Batch bt) {
  const ImgDesc &im = bt.img[blockIdx.y];
  TL_SCOPE(im, 9);
  const int t = threadIdx.x, lane = t & 31, w = t >> 5;
  extern __shared__ int chunk_off[];               // [C + 1] first chunk of cluster c
  __shared__ int wsum[kMrgThreads / 32];
  __shared__ int s_carry, s_last;
  __shared__ int members2[2][kChunk];              // member lists of the current and the previous unit
  const int C = *im.C_ptr;
  const int n_text = im.n_total - im.N;
  const int d = bt.d, ng = d / 8;
  const bool center_only = (im.flags & PACT_FLAG_CENTER_ONLY) != 0;
  const T *H = reinterpret_cast<const T *>(im.H);
  O *Ho = reinterpret_cast<O *>(im.H_out);
  if (blockIdx.x == 0 && t == 0) im.cnt[PACT_CNT_N_OUT] = n_text + C;
  if (t == 0) s_carry = 0;
  __syncthreads();
  // chunk offsets: exclusive prefix sum of the chunks per cluster
  for (int base = 0; base < C; base += kMrgThreads) {
    const int c = base + t;
    int nch = 0;
    if (c < C) nch = center_only ? 1 : (im.csize[c] + kChunk - 1) / kChunk;
    int x = nch;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= o) x += y;
    }
    if (lane == 31) wsum[w] = x;
    __syncthreads();
    int off = s_carry;
    for (int k = 0; k < w; ++k) off += wsum[k];
    if (c < C) chunk_off[c] = off + x - nch;
    __syncthreads();
    if (t == kMrgThreads - 1) s_carry = off + x;
    __syncthreads();
  }
  const int n_chunks = s_carry;
  if (t == 0) chunk_off[C] = n_chunks;
  __syncthreads();
  TL_POINT(im, 13);
  const int n_units = n_chunks + n_text;
  const int nblk = (im.N + kListBlock - 1) / kListBlock;

  // units are handed out first come, first served (the order does not change any result)
  // The member list and the next unit's number alternate between two slots: a thread can be at most one
  // barrier behind, so the slots of unit n are rewritten (for unit n + 2) only after every thread has
  // passed the barrier of unit n + 1, i.e. is done with unit n.  One CTA-wide barrier per unit.
  __shared__ int s_next2[2];
  int u = blockIdx.x, par = 0;
  while (u < n_units) {
    int c = -1, k = 0, nch = 1, size = 1, nm = 1, dst, ptok;
    int *members = members2[par];
    if (t == 0) s_next2[par] = gridDim.x + atomicAdd(&im.cnt[21], 1);   // needed only after this unit's rows
    if (u >= n_chunks) {                           // a text row
      const int tr = u - n_chunks;
      const int src = tr < im.vis_start ? tr : tr + im.N;
      dst = tr < im.vis_start ? tr : tr + C;
      ptok = src;
      if (t == 0) members[0] = src - im.vis_start; // relative to the visual span
    } else {
      int lo = 0, hi = C - 1;                      // last c with chunk_off[c] <= u
      while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (chunk_off[mid] <= u) lo = mid; else hi = mid - 1;
      }
      c = lo;
      k = u - chunk_off[c];
      nch = chunk_off[c + 1] - chunk_off[c];
      size = im.csize[c];
      const int ctok = im.cidx_ptr[c];
      dst = im.vis_start + c;
      ptok = im.vis_start + ctok;
      if (center_only) {
        if (t == 0) members[0] = ctok;
      } else {
        const int m0 = k * kChunk, m1 = min(size, m0 + kChunk);
        nm = m1 - m0;
        int carry = 0;
        if (nblk <= 32) {                           // one warp covers all blocks: no CTA-wide scan
          if (w == 0) {
            int s0 = 0, cntb = 0;
            if (lane < nblk) {
              const uint16_t *row = im.bstart + (size_t)lane * im.bstride;
              s0 = row[c];
              cntb = (int)row[c + 1] - s0;
            }
            int x = cntb;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
              const int y = __shfl_up_sync(0xffffffffu, x, o);
              if (lane >= o) x += y;
            }
            const int off = x - cntb;               // list position of this block's first member
            const int a0 = max(off, m0), a1 = min(off + cntb, m1);
            for (int m = a0; m < a1; ++m) members[m - m0] = im.blocklist[(size_t)lane * kListBlock + s0 + (m - off)];
          }
        } else
        for (int bb0 = 0; bb0 < nblk; bb0 += kMrgThreads) {   // thread = block of the member lists
          const int bb = bb0 + t;
          int s0 = 0, cntb = 0;
          if (bb < nblk) {                         // does not wait for the cluster size
            const uint16_t *row = im.bstart + (size_t)bb * im.bstride;
            s0 = row[c];
            cntb = (int)row[c + 1] - s0;
          }
          int x = cntb;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
          }
          if (bb0 > 0) __syncthreads();            // wsum of the previous round is consumed
          if (lane == 31) wsum[w] = x;
          __syncthreads();
          int off = carry, tot = 0;
#pragma unroll
          for (int q = 0; q < kMrgThreads / 32; ++q) { if (q < w) off += wsum[q]; tot += wsum[q]; }
          off += x - cntb;                         // list position of this block's first member
          const int a0 = max(off, m0), a1 = min(off + cntb, m1);
          for (int m = a0; m < a1; ++m) members[m - m0] = im.blocklist[(size_t)bb * kListBlock + s0 + (m - off)];
          carry += tot;
          if (carry >= m1) break;                  // uniform
        }
      }
    }
    __syncthreads();
    float acc[VPL][8];
#pragma unroll
    for (int v = 0; v < VPL; ++v)
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[v][e] = 0.f;
#pragma unroll 1
    for (int mi = 0; mi < nm; mi += kMrgRows) {
      Raw8<T> x[kMrgRows][VPL];
#pragma unroll
      for (int r = 0; r < kMrgRows; ++r) {
        if (mi + r < nm) {
          const T *row = H + (size_t)(im.vis_start + members[mi + r]) * im.ldH;
#pragma unroll
          for (int v = 0; v < VPL; ++v) {
            const int g = t + v * kMrgThreads;
            if (g < ng) x[r][v].load(row + g * 8);
          }
        }
      }
#pragma unroll
      for (int r = 0; r < kMrgRows; ++r) {
        if (mi + r < nm) {
#pragma unroll
          for (int v = 0; v < VPL; ++v) {
            const int g = t + v * kMrgThreads;
            if (g < ng) x[r][v].add_to(acc[v]);
          }
        }
      }
    }
    const float inv = center_only ? 1.0f : 1.0f / (float)size;   // one division per unit, not one per element
    if (nch > 1) {
      // scratch rows: the clusters that are summed in several chunks take theirs in cluster order
      int base = 0;
      for (int cc = lane; cc < c; cc += 32) {
        const int n = chunk_off[cc + 1] - chunk_off[cc];
        base += n > 1 ? n : 0;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) base += __shfl_xor_sync(0xffffffffu, base, o);
      float *part = im.mpart + (size_t)(base + k) * d;
#pragma unroll
      for (int v = 0; v < VPL; ++v) {
        const int g = t + v * kMrgThreads;
        if (g < ng) {
          reinterpret_cast<float4 *>(part + g * 8)[0] = make_float4(acc[v][0], acc[v][1], acc[v][2], acc[v][3]);
          reinterpret_cast<float4 *>(part + g * 8)[1] = make_float4(acc[v][4], acc[v][5], acc[v][6], acc[v][7]);
        }
      }
      __threadfence();
      __syncthreads();
      if (t == 0) s_last = (atomicAdd(&im.cticket[c], 1) == nch - 1);
      __syncthreads();
      if (!s_last) { u = s_next2[par]; par ^= 1; continue; }
      __threadfence();
      const float *p0 = im.mpart + (size_t)base * d;
#pragma unroll
      for (int v = 0; v < VPL; ++v) {
        const int g = t + v * kMrgThreads;
        if (g < ng) {
#pragma unroll
          for (int e = 0; e < 8; ++e) acc[v][e] = 0.f;
          for (int kk = 0; kk < nch; ++kk) {
            const float4 a = ld_cg_f4(p0 + (size_t)kk * d + g * 8), bq = ld_cg_f4(p0 + (size_t)kk * d + g * 8 + 4);
            acc[v][0] += a.x; acc[v][1] += a.y; acc[v][2] += a.z; acc[v][3] += a.w;
            acc[v][4] += bq.x; acc[v][5] += bq.y; acc[v][6] += bq.z; acc[v][7] += bq.w;
          }
        }
      }
      if (t == 0) im.cticket[c] = 0;
    }
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
      const int g = t + v * kMrgThreads;
      if (g < ng) {
        float y[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) y[e] = acc[v][e] * inv;
        store_vec8<O>(Ho + (size_t)dst * im.ldHo + g * 8, y);
      }
    }
    if (t == 0) {
      im.P_out[dst] = im.P[ptok];
      im.size_out[dst] = size;
      if (im.logw_out) im.logw_out[dst] = logf((float)size);   // Eq. 11: log of the token weight
    }
    u = s_next2[par];
    par ^= 1;
  }
}

void launch_lists(const Batch &bt, int maxN, bool bf16, bool from_best, cudaStream_t st) {
  const dim3 grid((maxN + kListBlock - 1) / kListBlock, bt.B);
  if (from_best) {
    if (bf16) k_lists<__nv_bfloat16, true><<<grid, kListBlock, 0, st>>>(bt);
    else k_lists<float, true><<<grid, kListBlock, 0, st>>>(bt);
  } else {
    k_lists<float, false><<<grid, kListBlock, 0, st>>>(bt);
  }
}

static size_t g_merge_smem_max = 48 * 1024;

template <typename T, typename O>
static cudaError_t launch_merge_t(const Batch &bt, int maxN, const ClusterCfg &cfg, cudaStream_t st) {
  const size_t smem = ((size_t)maxN + 2) * sizeof(int);
  if (smem > g_merge_smem_max) return cudaErrorInvalidConfiguration;
  int X = 3 * cfg.sm_count / bt.B;
  if (X < 1) X = 1;
  dim3 grid(X, bt.B);
  if (bt.d <= kMrgThreads * 2 * 8) k_merge<T, O, 2><<<grid, kMrgThreads, smem, st>>>(bt);
  else k_merge<T, O, kMrgVpl><<<grid, kMrgThreads, smem, st>>>(bt);
  return cudaGetLastError();
}

template <typename T, typename O> static cudaError_t merge_attr(int v) {
  cudaError_t e = cudaFuncSetAttribute(k_merge<T, O, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, v);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(k_merge<T, O, kMrgVpl>, cudaFuncAttributeMaxDynamicSharedMemorySize, v);
}

cudaError_t merge_configure() {
  int dev = 0, optin = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e != cudaSuccess) return e;
  g_merge_smem_max = (size_t)optin - 2048;
  const int v = (int)g_merge_smem_max;
  e = merge_attr<__nv_bfloat16, __nv_bfloat16>(v);
  if (e == cudaSuccess) e = merge_attr<__nv_bfloat16, float>(v);
  if (e == cudaSuccess) e = merge_attr<float, __nv_bfloat16>(v);
  if (e == cudaSuccess) e = merge_attr<float, float>(v);
  return e;
}

// largest N the merge kernel takes: its chunk offsets live in shared memory
int merge_max_tokens(int d, int elt) {
  (void)d; (void)elt;
  return (int)(g_merge_smem_max / sizeof(int)) - 2;
}

cudaError_t launch_merge(const Batch &bt, int maxN, bool in_bf16, bool out_bf16, const ClusterCfg &cfg, cudaStream_t st) {
  if (in_bf16) return out_bf16 ? launch_merge_t<__nv_bfloat16, __nv_bfloat16>(bt, maxN, cfg, st)
                               : launch_merge_t<__nv_bfloat16, float>(bt, maxN, cfg, st);
  return out_bf16 ? launch_merge_t<float, __nv_bfloat16>(bt, maxN, cfg, st) : launch_merge_t<float, float>(bt, maxN, cfg, st);
}

}  // namespace pact
