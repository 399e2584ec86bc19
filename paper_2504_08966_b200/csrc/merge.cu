// Merge (Eq. 10, Algorithm 3 step 4): one hidden state per cluster = mean of its members in
// float accumulation and ascending token order; position id of the centre; cluster sizes;
// text rows copied around the merged span.
#include "kernels.cuh"

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

constexpr int kMergeThreads = 256;
constexpr int kListBlock = 256;      // tokens per block of the member lists
constexpr int kChunk = 16;           // members summed by one work item
constexpr int kChunkLanes = 8;       // CTAs that share the chunks of one cluster (grid.y)

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
// integer atomics; the last block to finish turns them into chunk offsets for the merge.
__global__ void __launch_bounds__(kListBlock) k_lists(const __grid_constant__ Batch bt) {
  const ImgDesc &im = bt.img[blockIdx.y];
  TL_SCOPE(im, 8);
  const int N = im.N;
  const int nblk = (N + kListBlock - 1) / kListBlock;
  const int b = blockIdx.x, t = threadIdx.x;
  if (b >= nblk) return;
  __shared__ int slab[kListBlock], sorted_lab[kListBlock];
  const int i = b * kListBlock + t;
  const int lab = i < N ? im.label[i] : -1;
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
  // the last block: chunk offsets of the clusters that need more than one chunk
  __shared__ int last;
  __threadfence();
  __syncthreads();
  if (t == 0) last = (atomicAdd(&im.cnt[19], 1) == nblk - 1);
  __syncthreads();
  if (!last) return;
  __threadfence();
  __shared__ int wsum[kListBlock / 32];
  __shared__ int carry;
  if (t == 0) carry = 0;
  __syncthreads();
  const int lane = t & 31, w = t >> 5;
  for (int base = 0; base < C; base += kListBlock) {
    const int c = base + t;
    int nch = 0;
    if (c < C) {
      nch = (ld_cg_i32(&im.csize[c]) + kChunk - 1) / kChunk;
      if (nch <= 1) nch = 0;
    }
    int x = nch;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= o) x += y;
    }
    if (lane == 31) wsum[w] = x;
    __syncthreads();
    int off = carry;
    for (int k = 0; k < w; ++k) off += wsum[k];
    if (c < C) im.cbase[c] = off + x - nch;
    __syncthreads();
    if (t == kListBlock - 1) carry = off + x;
    __syncthreads();
  }
  if (t == 0) im.cnt[19] = 0;
}

// ---- Eq. 10 ------------------------------------------------------------------------------------------
// grid (X, kChunkLanes + 1, B), 256 threads.  CTAs with blockIdx.y < kChunkLanes: cluster c = blockIdx.x,
// blockIdx.x + X, ...; the chunks k = blockIdx.y, blockIdx.y + kChunkLanes, ... of its member list
// (kChunk members each, ascending token order) are summed in float.  A cluster of one chunk is finished
// on the spot; otherwise the chunk sums go to scratch and the CTA that finishes the cluster's last chunk
// adds them in chunk order.  CTAs with blockIdx.y == kChunkLanes copy the text rows.
template <typename T, typename O, int VPT>
__global__ void __launch_bounds__(kMergeThreads) k_merge(const __grid_constant__ Batch bt) {
  constexpr int R = (sizeof(T) == 2 ? 16 : 8) / VPT;    // member rows in flight per thread
  const ImgDesc &im = bt.img[blockIdx.z];
  TL_SCOPE(im, 9);
  const int t = threadIdx.x, lane = t & 31, w = t >> 5;
  const int C = *im.C_ptr;
  const int n_text = im.n_total - im.N;
  const int d = bt.d, ng = d / 8;
  const T *H = reinterpret_cast<const T *>(im.H);
  O *Ho = reinterpret_cast<O *>(im.H_out);
  if (blockIdx.y == kChunkLanes) {
    if (blockIdx.x == 0 && t == 0) im.cnt[PACT_CNT_N_OUT] = n_text + C;
    for (int tr = blockIdx.x; tr < n_text; tr += gridDim.x) {
      const int src = tr < im.vis_start ? tr : tr + im.N;
      const int dst = tr < im.vis_start ? tr : tr + C;
      for (int gcol = t; gcol < ng; gcol += kMergeThreads) {
        float x[8];
        load8<T>(H + (size_t)src * im.ldH + gcol * 8, x);
        store_vec8<O>(Ho + (size_t)dst * im.ldHo + gcol * 8, x);
      }
      if (t == 0) { im.P_out[dst] = im.P[src]; im.size_out[dst] = 1; }
    }
    return;
  }
  const int nblk = (im.N + kListBlock - 1) / kListBlock;
  __shared__ int members[kChunk];
  __shared__ int wsum[kMergeThreads / 32];
  __shared__ int s_last;
  for (int c = blockIdx.x; c < C; c += gridDim.x) {
    const int size = im.csize[c];
    const int nch = (size + kChunk - 1) / kChunk;
    if ((int)blockIdx.y >= nch) continue;
    const int dst = im.vis_start + c;
    if (im.flags & PACT_FLAG_CENTER_ONLY) {             // the centre stands for its cluster
      if (blockIdx.y == 0) {
        const int ctok = im.cidx_ptr[c];
        const T *row = H + (size_t)(im.vis_start + ctok) * im.ldH;
        for (int gcol = t; gcol < ng; gcol += kMergeThreads) {
          float x[8];
          load8<T>(row + gcol * 8, x);
          store_vec8<O>(Ho + (size_t)dst * im.ldHo + gcol * 8, x);
        }
        if (t == 0) { im.P_out[dst] = im.P[im.vis_start + ctok]; im.size_out[dst] = size; }
      }
      continue;
    }
    for (int k = blockIdx.y; k < nch; k += kChunkLanes) {
      const int m0 = k * kChunk, m1 = min(size, m0 + kChunk);
      // member list positions [m0, m1) -> token indices
      int carry = 0;
      for (int bb0 = 0; bb0 < nblk && carry < m1; bb0 += kMergeThreads) {
        const int bb = bb0 + t;
        int s0 = 0, cntb = 0;
        if (bb < nblk) {
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
        __syncthreads();                                // wsum and members of the previous round are consumed
        if (lane == 31) wsum[w] = x;
        __syncthreads();
        int off = carry, tot = 0;
#pragma unroll
        for (int q = 0; q < kMergeThreads / 32; ++q) { if (q < w) off += wsum[q]; tot += wsum[q]; }
        off += x - cntb;                                // list position of this block's first member
        const int lo = max(off, m0), hi = min(off + cntb, m1);
        for (int m = lo; m < hi; ++m) members[m - m0] = im.blocklist[(size_t)bb * kListBlock + s0 + (m - off)];
        carry += tot;
      }
      __syncthreads();
      float acc[VPT][8];
#pragma unroll
      for (int v = 0; v < VPT; ++v)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[v][e] = 0.f;
      const int nm = m1 - m0;
      for (int mi = 0; mi < nm; mi += R) {
        Raw8<T> x[R][VPT];
#pragma unroll
        for (int r = 0; r < R; ++r) {
          if (mi + r < nm) {
            const T *row = H + (size_t)(im.vis_start + members[mi + r]) * im.ldH;
#pragma unroll
            for (int v = 0; v < VPT; ++v) {
              const int gcol = t + v * kMergeThreads;
              if (gcol < ng) x[r][v].load(row + gcol * 8);
            }
          }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
          if (mi + r < nm) {
#pragma unroll
            for (int v = 0; v < VPT; ++v) {
              const int gcol = t + v * kMergeThreads;
              if (gcol < ng) x[r][v].add_to(acc[v]);
            }
          }
        }
      }
      bool finish = nch == 1;
      if (!finish) {
        float *part = im.mpart + (size_t)(im.cbase[c] + k) * d;
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
          const int gcol = t + v * kMergeThreads;
          if (gcol < ng) {
            reinterpret_cast<float4 *>(part + gcol * 8)[0] = make_float4(acc[v][0], acc[v][1], acc[v][2], acc[v][3]);
            reinterpret_cast<float4 *>(part + gcol * 8)[1] = make_float4(acc[v][4], acc[v][5], acc[v][6], acc[v][7]);
          }
        }
        __threadfence();
        __syncthreads();
        if (t == 0) s_last = (atomicAdd(&im.cticket[c], 1) == nch - 1);
        __syncthreads();
        finish = s_last != 0;
        if (finish) {
          __threadfence();
          const float *p0 = im.mpart + (size_t)im.cbase[c] * d;
#pragma unroll
          for (int v = 0; v < VPT; ++v) {
            const int gcol = t + v * kMergeThreads;
            if (gcol < ng) {
#pragma unroll
              for (int e = 0; e < 8; ++e) acc[v][e] = 0.f;
              for (int kk = 0; kk < nch; ++kk) {
                const float4 a = ld_cg_f4(p0 + (size_t)kk * d + gcol * 8), bq = ld_cg_f4(p0 + (size_t)kk * d + gcol * 8 + 4);
                acc[v][0] += a.x; acc[v][1] += a.y; acc[v][2] += a.z; acc[v][3] += a.w;
                acc[v][4] += bq.x; acc[v][5] += bq.y; acc[v][6] += bq.z; acc[v][7] += bq.w;
              }
            }
          }
          if (t == 0) im.cticket[c] = 0;
        }
      }
      if (finish) {
        const float fs = (float)size;
#pragma unroll
        for (int v = 0; v < VPT; ++v) {
          const int gcol = t + v * kMergeThreads;
          if (gcol < ng) {
            float y[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) y[e] = acc[v][e] / fs;
            store_vec8<O>(Ho + (size_t)dst * im.ldHo + gcol * 8, y);
          }
        }
        if (t == 0) {
          im.P_out[dst] = im.P[im.vis_start + im.cidx_ptr[c]];
          im.size_out[dst] = size;
        }
      }
    }
  }
}

void launch_lists(const Batch &bt, int maxN, cudaStream_t st) {
  k_lists<<<dim3((maxN + kListBlock - 1) / kListBlock, bt.B), kListBlock, 0, st>>>(bt);
}

template <typename T, typename O>
static void launch_merge_t(const Batch &bt, int maxN, const ClusterCfg &cfg, cudaStream_t st) {
  int X = 2 * cfg.sm_count;
  if (X > maxN) X = maxN;
  dim3 grid(X, kChunkLanes + 1, bt.B);
  if (bt.d <= kMergeThreads * 2 * 8) k_merge<T, O, 2><<<grid, kMergeThreads, 0, st>>>(bt);
  else k_merge<T, O, 4><<<grid, kMergeThreads, 0, st>>>(bt);
}

void launch_merge(const Batch &bt, int maxN, bool in_bf16, bool out_bf16, const ClusterCfg &cfg, cudaStream_t st) {
  if (in_bf16) {
    if (out_bf16) launch_merge_t<__nv_bfloat16, __nv_bfloat16>(bt, maxN, cfg, st);
    else launch_merge_t<__nv_bfloat16, float>(bt, maxN, cfg, st);
  } else {
    if (out_bf16) launch_merge_t<float, __nv_bfloat16>(bt, maxN, cfg, st);
    else launch_merge_t<float, float>(bt, maxN, cfg, st);
  }
}

}  // namespace pact
