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

constexpr int kMergeThreads = 256;
constexpr int kMergeVPT = 4;    // 8-element column groups per thread: d <= 256 * 4 * 8

// grid (n_ctas, B), persistent over work items: clusters 0..C-1, then the text rows.
template <typename T, typename O>
__global__ void __launch_bounds__(kMergeThreads) k_merge(const __grid_constant__ Batch bt) {
  const ImgDesc &im = bt.img[blockIdx.y];
  const int t = threadIdx.x, lane = t & 31, w = t >> 5;
  const int C = *im.C_ptr;
  const int n_text = im.n_total - im.N;
  const int d = bt.d, ng = d / 8;
  const T *H = reinterpret_cast<const T *>(im.H);
  O *Ho = reinterpret_cast<O *>(im.H_out);
  __shared__ int members[kMergeThreads];
  __shared__ int wcount[kMergeThreads / 32];
  if (blockIdx.x == 0 && t == 0) im.cnt[PACT_CNT_N_OUT] = n_text + C;
  for (int item = blockIdx.x; item < C + n_text; item += gridDim.x) {
    if (item >= C) {                                    // a text row
      const int tr = item - C;
      const int src = tr < im.vis_start ? tr : tr + im.N;
      const int dst = tr < im.vis_start ? tr : tr - im.vis_start + im.vis_start + C;
      for (int gcol = t; gcol < ng; gcol += kMergeThreads) {
        float x[8];
        load8<T>(H + (size_t)src * im.ldH + gcol * 8, x);
        store_vec8<O>(Ho + (size_t)dst * im.ldHo + gcol * 8, x);
      }
      if (t == 0) { im.P_out[dst] = im.P[src]; im.size_out[dst] = 1; }
      continue;
    }
    const int c = item;
    const int ctok = im.cidx_ptr[c];
    float acc[kMergeVPT][8];
#pragma unroll
    for (int v = 0; v < kMergeVPT; ++v)
#pragma unroll
      for (int k = 0; k < 8; ++k) acc[v][k] = 0.f;
    int size = 0;
    for (int base = 0; base < im.N; base += kMergeThreads) {
      const int i = base + t;
      const bool mine = i < im.N && im.label[i] == c;
      const unsigned bal = __ballot_sync(0xffffffffu, mine);
      if (lane == 0) wcount[w] = __popc(bal);
      __syncthreads();
      int off = 0, tot = 0;
#pragma unroll
      for (int k = 0; k < kMergeThreads / 32; ++k) { if (k < w) off += wcount[k]; tot += wcount[k]; }
      if (mine) members[off + __popc(bal & ((1u << lane) - 1u))] = i;
      __syncthreads();
      size += tot;
      if (!(im.flags & PACT_FLAG_CENTER_ONLY)) {
        for (int mi = 0; mi < tot; ++mi) {
          const T *row = H + (size_t)(im.vis_start + members[mi]) * im.ldH;
#pragma unroll
          for (int v = 0; v < kMergeVPT; ++v) {
            const int gcol = t + v * kMergeThreads;
            if (gcol < ng) {
              float x[8];
              load8<T>(row + gcol * 8, x);
#pragma unroll
              for (int k = 0; k < 8; ++k) acc[v][k] += x[k];
            }
          }
        }
      }
      __syncthreads();
    }
    const int dst = im.vis_start + c;
    if (im.flags & PACT_FLAG_CENTER_ONLY) {
      const T *row = H + (size_t)(im.vis_start + ctok) * im.ldH;
      for (int gcol = t; gcol < ng; gcol += kMergeThreads) {
        float x[8];
        load8<T>(row + gcol * 8, x);
        store_vec8<O>(Ho + (size_t)dst * im.ldHo + gcol * 8, x);
      }
    } else {
      const float fs = (float)size;
#pragma unroll
      for (int v = 0; v < kMergeVPT; ++v) {
        const int gcol = t + v * kMergeThreads;
        if (gcol < ng) {
          float x[8];
#pragma unroll
          for (int k = 0; k < 8; ++k) x[k] = acc[v][k] / fs;
          store_vec8<O>(Ho + (size_t)dst * im.ldHo + gcol * 8, x);
        }
      }
    }
    if (t == 0) {
      im.P_out[dst] = im.P[im.vis_start + ctok];
      im.size_out[dst] = size;
    }
  }
}

void launch_merge(const Batch &bt, bool in_bf16, bool out_bf16, const ClusterCfg &cfg, cudaStream_t st) {
  dim3 grid(cfg.sm_count * 8, bt.B);
  if (in_bf16) {
    if (out_bf16) k_merge<__nv_bfloat16, __nv_bfloat16><<<grid, kMergeThreads, 0, st>>>(bt);
    else k_merge<__nv_bfloat16, float><<<grid, kMergeThreads, 0, st>>>(bt);
  } else {
    if (out_bf16) k_merge<float, __nv_bfloat16><<<grid, kMergeThreads, 0, st>>>(bt);
    else k_merge<float, float><<<grid, kMergeThreads, 0, st>>>(bt);
  }
}

}  // namespace pact
