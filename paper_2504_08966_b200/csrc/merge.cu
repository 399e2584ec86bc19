// Merge (Eq. 10, Algorithm 3 step 4): one hidden state per cluster = mean of its members in
// float accumulation and ascending token order; position id of the centre; cluster sizes;
// text rows copied around the merged span.
//
//   k_lists  labels (reincorporation test of Eq. 8), then a stable counting sort of the tokens by
//            cluster id: every block of 128 tokens sorts its own, an image-wide barrier, and every
//            token writes one 16-byte record {token, cluster, first member position, cluster size}
//            at its place in the cluster-sorted member array.  Also P', sizes and log sizes.
//   k_merge  the member array (followed by the text rows) is cut into one contiguous range per CTA;
//            a CTA streams the rows of its range with many loads in flight and no look-ups, keeps the
//            running cluster in registers and writes a row out whenever the cluster id changes.
//            Clusters cut by a range boundary leave partial sums; the last CTA to arrive adds them in
//            range order, so the result does not depend on timing.
#include <cooperative_groups.h>

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

// Eight consecutive elements of a row as loaded (not yet widened), so that many can be in flight.
template <typename T> struct Raw8;
template <> struct Raw8<__nv_bfloat16> {
  uint4 a;
  __device__ __forceinline__ void from_ring(const uint4 *p) { a = p[0]; }
  __device__ __forceinline__ void add_to(float (&acc)[8]) const {
    float x[8];
    widen_vec<__nv_bfloat16>(a, x);
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] += x[e];
  }
};
template <> struct Raw8<float> {
  uint4 a, b;
  __device__ __forceinline__ void from_ring(const uint4 *p) { a = p[0]; b = p[1]; }
  __device__ __forceinline__ void add_to(float (&acc)[8]) const {
    float x[4], y[4];
    widen_vec<float>(a, x);
    widen_vec<float>(b, y);
#pragma unroll
    for (int e = 0; e < 4; ++e) { acc[e] += x[e]; acc[4 + e] += y[e]; }
  }
};

__device__ __forceinline__ int ld_cg_i32(const int *p) {
  int v;
  asm volatile("ld.global.cg.s32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ int ld_acquire_i32(const int *p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ float4 ld_cg_f4(const float *p) {
  float4 v;
  asm volatile("ld.global.cg.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
}

// ---- member lists --------------------------------------------------------------------------------
// grid (ceil(maxN / 128), B), 128 threads.
// Part 1: block b sorts its 128 tokens by (cluster id, token), discarded tokens last; the first token of
//   every run writes the run length to cnt_cb[c][b] (a table that is zero before the kernel) and adds it
//   to csize[c].
// Part 2 (after every block of the image has finished part 1): the member in sorted position t of block b
//   belongs at  member_off[c] + (members of c in the blocks before b) + (its place in the run),  where
//   member_off is the exclusive prefix sum of csize.  It writes its record there; the first member of a
//   cluster also writes P', the size and its logarithm for the cluster's output row.
// mode 0: both parts, separated by a barrier over the blocks of the image (all blocks must be resident:
//         cooperative launch); mode 1: part 1 only, the sorted blocks go to blocklist; mode 2: part 2 only.
// FROM_BEST: the labels are first formed here from the nearest-centre pass (survivors: cluster id of the
// nearest centre, a centre its own id; pruned tokens: that id iff the distance is strictly below
// alpha * d_c, else -1) and written out; otherwise label[] is given, and an id outside [-1, C) is
// dropped like -1 and reported through the status word.
constexpr int kScanTile = kListBlock * 8;   // cluster sizes scanned per step of part 2
constexpr int kNoLabel = 0x7fffffff;

template <typename T, bool FROM_BEST>
__global__ void __launch_bounds__(kListBlock) k_lists(const __grid_constant__ Batch bt, int mode, int spin_limit) {
  using D = typename DistOf<T>::type;
  const ImgDesc &im = bt.img[blockIdx.y];
  TL_SCOPE(im, 8);
  pdl_wait();
  pdl_trigger();
  const int N = im.N;
  const int nblk = (N + kListBlock - 1) / kListBlock;
  const int b = blockIdx.x, t = threadIdx.x, lane = t & 31, w = t >> 5;
  if (b >= nblk) return;
  __shared__ int slab[kListBlock], s_lab[kListBlock], s_tok[kListBlock];
  __shared__ int excl[kScanTile];
  __shared__ int wsum[kListBlock / 32];
  __shared__ int s_carry;
  const int C = min(*im.C_ptr, im.Np);
  const int i = b * kListBlock + t;

  if (mode != 2) {
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
        if (lab >= C) lab = -1;                       // only after a failed earlier stage
        im.label[i] = lab;
        if (im.label_user) im.label_user[i] = lab;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        joined += __shfl_xor_sync(0xffffffffu, joined, o);
        dropped += __shfl_xor_sync(0xffffffffu, dropped, o);
        band += __shfl_xor_sync(0xffffffffu, band, o);
      }
      if (lane == 0) {
        if (joined) atomicAdd(&im.cnt[PACT_CNT_R], joined);
        if (dropped) atomicAdd(&im.cnt[PACT_CNT_DISCARDED], dropped);
        if (band) atomicAdd(&im.cnt[PACT_CNT_BAND_ADC], band);
      }
    } else {
      lab = i < N ? im.label[i] : -1;
      if (lab >= C || lab < -1) {                     // a label the caller should not have passed
        lab = -1;
        atomicMin(&im.cnt[PACT_CNT_STATUS], (int)PACT_ERR_INVALID_ARG);
      }
    }
    const int key = lab < 0 ? kNoLabel : lab;
    slab[t] = key;
    __syncthreads();
    int rank = 0;
#pragma unroll 8
    for (int u = 0; u < kListBlock; ++u) {
      const int o = slab[u];
      rank += (o < key) || (o == key && u < t);
    }
    s_lab[rank] = key;
    s_tok[rank] = i;
    __syncthreads();
    if (mode == 1) im.blocklist[(size_t)b * kListBlock + t] = s_tok[t];
  } else {
    const int tok = im.blocklist[(size_t)b * kListBlock + t];
    const int lab = tok < N ? im.label[tok] : -1;
    s_tok[t] = tok;
    s_lab[t] = (lab < 0 || lab >= C) ? kNoLabel : lab;
    __syncthreads();
  }
  // first position whose cluster id is >= c
  auto lower = [&](int c) {
    int lo = 0, hi = kListBlock;
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (s_lab[mid] < c) lo = mid + 1; else hi = mid;
    }
    return lo;
  };
  const int c = s_lab[t];
  const bool valid = c != kNoLabel;
  const int run0 = valid ? lower(c) : t;
  if (mode != 2 && valid && run0 == t) {
    const int len = lower(c + 1) - t;
    im.cnt_cb[(size_t)c * im.nbp + b] = (uint16_t)len;
    atomicAdd(&im.csize[c], len);
  }
  if (mode == 1) return;
  TL_POINT(im, 13);
  if (mode == 0) {
    // every block of the image has published its run lengths before anyone reads them
    __threadfence();
    __syncthreads();
    if (t == 0) {
      atomicAdd(&im.cnt[19], 1);
      int spins = 0;
      while (ld_acquire_i32(&im.cnt[19]) < nblk) {
        if (++spins > spin_limit) { atomicMin(&im.cnt[PACT_CNT_STATUS], (int)PACT_ERR_TIMEOUT); break; }
        __nanosleep(40);
      }
    }
    __syncthreads();
    __threadfence();
  }
  TL_POINT(im, 14);

  // part 2
  int before = 0, size = 0;                          // members of c in earlier blocks; members of c
  if (valid) {
    const uint4 *row = reinterpret_cast<const uint4 *>(im.cnt_cb + (size_t)c * im.nbp);
    for (int v = 0; v * 8 < b; ++v) {
      const uint4 x = __ldcg(row + v);
      const uint32_t xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int cntk = (int)((xs[k >> 1] >> ((k & 1) * 16)) & 0xFFFFu);
        if (v * 8 + k < b) before += cntk;
      }
    }
    size = ld_cg_i32(&im.csize[c]);
  }
  // member_off[c] = cluster sizes below c, scanned kScanTile at a time
  if (t == 0) s_carry = 0;
  __syncthreads();
  int moff = 0;
  for (int base = 0; base < C; base += kScanTile) {
    int v8[8], s = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int cc = base + t * 8 + k;
      v8[k] = cc < C ? ld_cg_i32(&im.csize[cc]) : 0;
      s += v8[k];
    }
    int x = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= o) x += y;
    }
    if (lane == 31) wsum[w] = x;
    __syncthreads();
    int off = s_carry;
    for (int k = 0; k < w; ++k) off += wsum[k];
    int run = off + x - s;
#pragma unroll
    for (int k = 0; k < 8; ++k) { excl[t * 8 + k] = run; run += v8[k]; }
    __syncthreads();
    if (valid && c >= base && c < base + kScanTile) moff = excl[c - base];
    if (t == kListBlock - 1) s_carry = run;
    __syncthreads();
  }
  if (b == 0 && t == 0) im.cnt[20] = s_carry;        // members in all clusters
  if (!valid) return;
  int pos = moff + before + (t - run0);
  pos = max(0, min(pos, N - 1));                     // in bounds whatever an aborted stage left behind
  const int tok = s_tok[t];
  im.members[pos] = make_int4(tok, c, moff, size);
  if (before == 0 && t == run0) {                    // first member of the cluster: the row's bookkeeping
    const int dst = im.vis_start + c;
    if (im.P_out) im.P_out[dst] = im.P[im.vis_start + min(max(im.cidx_ptr[c], 0), N - 1)];
    if (im.size_out) im.size_out[dst] = size;
    if (im.logw_out) im.logw_out[dst] = logf((float)size);   // Eq. 11: log of the token weight
  }
}

// ---- member records from finished labels ----------------------------------------------------------
// grid (ceil(maxN / 128), B), 128 threads.  The rows x centres pass on the tensor cores has already written
// the labels, the cluster sizes and cnt_cb (members of cluster c in token block b) as its groups of rows
// finished; what is left is the second part of k_lists: the member of cluster c that is token i of block b
// belongs at  member_off[c] + (members of c in the blocks before b) + (members of c before i in block b).
__global__ void __launch_bounds__(kListBlock) k_members(const __grid_constant__ Batch bt) {
  const ImgDesc &im = bt.img[blockIdx.y];
  TL_SCOPE(im, 8);
  // the number of clusters was final before the rows x centres pass began, and this kernel cannot start before
  // every CTA of that pass has begun: it may be read ahead of the wait
  const int C = min(ld_cg_i32(im.C_ptr), im.Np);
  pdl_wait();
  pdl_trigger();
  const int N = im.N;
  const int nblk = (N + kListBlock - 1) / kListBlock;
  const int b = blockIdx.x, t = threadIdx.x, lane = t & 31, w = t >> 5;
  if (b >= nblk) return;
  __shared__ __align__(16) int slab[kListBlock];
  __shared__ int excl[kScanTile];
  __shared__ int wsum[kListBlock / 32];
  __shared__ int s_carry;
  const int i = b * kListBlock + t;
  int c = -1;
  if (i < N) {
    if (C > 0) c = ld_cg_i32(&im.label[i]);
    else {                                           // no centre at all (a failed earlier stage): nothing was labelled
      im.label[i] = -1;
      if (im.label_user) im.label_user[i] = -1;
    }
    if (c >= C || c < -1) c = -1;
  }
  const bool valid = c >= 0;
  slab[t] = c;
  // in flight while the block is searched: the counts of the earlier blocks, the cluster's size, the sizes to scan
  constexpr int kCbRegs = 8;                         // rows of cnt_cb of up to 64 token blocks are read at once
  uint4 cb[kCbRegs];
  int size = 0;
  const uint4 *row = reinterpret_cast<const uint4 *>(im.cnt_cb + (size_t)(valid ? c : 0) * im.nbp);
#pragma unroll
  for (int v = 0; v < kCbRegs; ++v) cb[v] = (valid && v * 8 < b) ? __ldcg(row + v) : make_uint4(0u, 0u, 0u, 0u);
  if (valid) size = ld_cg_i32(&im.csize[c]);
  int v8[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int cc = t * 8 + k;
    v8[k] = cc < C ? ld_cg_i32(&im.csize[cc]) : 0;
  }
  __syncthreads();
  TL_POINT(im, 13);
  int place = 0;                                     // members of c before token i in this block
  if (valid) {
    const int4 *s4 = reinterpret_cast<const int4 *>(slab);
    const int full = t >> 2;
    for (int u = 0; u < full; ++u) {
      const int4 x = s4[u];
      place += (x.x == c) + (x.y == c) + (x.z == c) + (x.w == c);
    }
    const int4 x = s4[full];
    place += ((t & 3) > 0 && x.x == c) + ((t & 3) > 1 && x.y == c) + ((t & 3) > 2 && x.z == c);
  }
  int before = 0;
#pragma unroll
  for (int v = 0; v < kCbRegs; ++v) {
    const uint32_t xs[4] = {cb[v].x, cb[v].y, cb[v].z, cb[v].w};
#pragma unroll
    for (int k = 0; k < 8; ++k)
      if (v * 8 + k < b) before += (int)((xs[k >> 1] >> ((k & 1) * 16)) & 0xFFFFu);
  }
  if (valid)
    for (int v = kCbRegs; v * 8 < b; ++v) {          // more token blocks than that
      const uint4 x = __ldcg(row + v);
      const uint32_t xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
      for (int k = 0; k < 8; ++k)
        if (v * 8 + k < b) before += (int)((xs[k >> 1] >> ((k & 1) * 16)) & 0xFFFFu);
    }
  // member_off[c] = cluster sizes below c, scanned kScanTile at a time
  if (t == 0) s_carry = 0;
  __syncthreads();
  int moff = 0;
  for (int base = 0; base < C; base += kScanTile) {
    int s = 0;
    if (base > 0) {
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int cc = base + t * 8 + k;
        v8[k] = cc < C ? ld_cg_i32(&im.csize[cc]) : 0;
      }
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) s += v8[k];
    int x = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= o) x += y;
    }
    if (lane == 31) wsum[w] = x;
    __syncthreads();
    int off = s_carry;
    for (int k = 0; k < w; ++k) off += wsum[k];
    int run = off + x - s;
#pragma unroll
    for (int k = 0; k < 8; ++k) { excl[t * 8 + k] = run; run += v8[k]; }
    __syncthreads();
    if (valid && c >= base && c < base + kScanTile) moff = excl[c - base];
    if (t == kListBlock - 1) s_carry = run;
    __syncthreads();
  }
  if (b == 0 && t == 0) im.cnt[20] = s_carry;        // members in all clusters
  TL_POINT(im, 14);
  if (!valid) return;
  int pos = moff + before + place;
  pos = max(0, min(pos, N - 1));                     // in bounds whatever an aborted stage left behind
  im.members[pos] = make_int4(i, c, moff, size);
  if (before == 0 && place == 0) {                   // first member of the cluster: the row's bookkeeping
    const int dst = im.vis_start + c;
    if (im.P_out) im.P_out[dst] = im.P[im.vis_start + min(max(im.cidx_ptr[c], 0), N - 1)];
    if (im.size_out) im.size_out[dst] = size;
    if (im.logw_out) im.logw_out[dst] = logf((float)size);   // Eq. 11: log of the token weight
  }
}

// ---- Eq. 10 ------------------------------------------------------------------------------------------
// Grid (X, B), kMrgThreads threads, two CTAs per SM.  Work items are the member records in cluster order
// followed by the text rows; CTA x takes items [x per, (x + 1) per).  A thread owns VPL groups of 8 columns
// and adds the rows of the running cluster in float.  The rows arrive through a ring of DEPTH rows in shared
// memory filled with asynchronous 16-byte copies (every thread copies and later reads its own columns, so
// the ring needs no barrier): DEPTH rows are in flight per SM whatever the registers hold.  A cluster that
// lies inside the range is divided and stored when the next one begins.  A range boundary cuts at most two clusters per CTA: the one that began before the range (its
// sum is set aside when it ends) and the one that goes on after it.  Their sums go to scratch (slot 0 and
// slot 1 of the CTA) with a ticket each; the CTA that draws a cluster's last ticket adds the sums in range
// order and stores the row, so the result does not depend on which CTA that is.
constexpr int kMrgThreads = 512;
constexpr int kMrgTile = 256;                       // records staged in shared memory at a time
constexpr int kMrgCtasPerSm = 2;
constexpr int kMrgRingBytes = 160 * 1024 / kMrgCtasPerSm;   // rows in flight per CTA

template <typename T, typename O, int VPL, int DEPTH>
__global__ void __launch_bounds__(kMrgThreads, kMrgCtasPerSm) k_merge(const __grid_constant__ Batch bt) {
  const ImgDesc &im = bt.img[blockIdx.y];
  TL_SCOPE(im, 9);
  // final since the centre selection, which is complete before any kernel after it can start
  const int C = min(ld_cg_i32(im.C_ptr), im.Np);
  pdl_wait();
  pdl_trigger();
  const int t = threadIdx.x;
  __shared__ int4 s_rec[kMrgTile];                  // {row of H, cluster, first member position, size}
  __shared__ int s_dst[kMrgTile];                   // output row
  __shared__ float s_inv[kMrgTile];                 // 1 / size (1 for text rows and centre-only merging)
  __shared__ int s_last;
  const int n_text = im.n_total - im.N;
  const int d = bt.d, ng = d / 8;
  const bool center_only = (im.flags & PACT_FLAG_CENTER_ONLY) != 0;
  const T *H = reinterpret_cast<const T *>(im.H);
  O *Ho = reinterpret_cast<O *>(im.H_out);
  const int n_mem = center_only ? C : min(max(ld_cg_i32(&im.cnt[20]), 0), im.N);
  const int total = n_mem + n_text;
  const int X = gridDim.x, x = blockIdx.x;
  const int per = (total + X - 1) / X;
  const int lo = min(total, x * per), hi = min(total, lo + per);
  if (x == 0 && t == 0) im.cnt[PACT_CNT_N_OUT] = n_text + C;

  float acc[VPL][8];
  int cur_c = -1, cur_off = 0, cur_size = 0, cur_dst = 0;
  float cur_inv = 1.f;
  bool head_open = false;                           // the running cluster began before this range
#pragma unroll
  for (int v = 0; v < VPL; ++v)
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[v][e] = 0.f;

  auto store_row = [&](const float (&a)[VPL][8], float inv, int dst) {
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
      const int g = t + v * kMrgThreads;
      if (g < ng) {
        float y[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) y[e] = a[v][e] * inv;
        store_vec8<O>(Ho + (size_t)dst * im.ldHo + g * 8, y);
      }
    }
  };
  // a cluster cut by a range boundary: sum to scratch, ticket, and the last one adds the sums in range order
  auto cut = [&](float (&a)[VPL][8], int c, int off, int size, float inv, int dst, int slot) {
    float *part = im.mpart + ((size_t)x * 2 + slot) * d;
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
      const int g = t + v * kMrgThreads;
      if (g < ng) {
        reinterpret_cast<float4 *>(part + g * 8)[0] = make_float4(a[v][0], a[v][1], a[v][2], a[v][3]);
        reinterpret_cast<float4 *>(part + g * 8)[1] = make_float4(a[v][4], a[v][5], a[v][6], a[v][7]);
      }
    }
    const int x0 = off / per, x1 = (off + size - 1) / per;
    __threadfence();
    __syncthreads();
    if (t == 0) s_last = (atomicAdd(&im.cticket[c], 1) == x1 - x0);
    __syncthreads();
    const bool last = s_last != 0;
    __syncthreads();                                 // s_last may be rewritten by the second cut cluster
    if (!last) return;
    __threadfence();
#pragma unroll
    for (int v = 0; v < VPL; ++v)
#pragma unroll
      for (int e = 0; e < 8; ++e) a[v][e] = 0.f;
    for (int xx = x0; xx <= x1; ++xx) {
      const float *p = im.mpart + ((size_t)xx * 2 + (xx < x1 ? 1 : 0)) * d;
#pragma unroll
      for (int v = 0; v < VPL; ++v) {
        const int g = t + v * kMrgThreads;
        if (g < ng) {
          const float4 u = ld_cg_f4(p + g * 8), w = ld_cg_f4(p + g * 8 + 4);
          a[v][0] += u.x; a[v][1] += u.y; a[v][2] += u.z; a[v][3] += u.w;
          a[v][4] += w.x; a[v][5] += w.y; a[v][6] += w.z; a[v][7] += w.w;
        }
      }
    }
    if (t == 0) im.cticket[c] = 0;
    store_row(a, inv, dst);
  };

  constexpr int Q16 = (int)sizeof(T) * 8 / 16;        // 16-byte pieces of a group of 8 columns
  constexpr int kSlot = VPL * kMrgThreads * Q16;      // 16-byte pieces per ring slot
  extern __shared__ uint4 ring[];                     // [DEPTH][kSlot]
  auto issue = [&](int j, int tn) {                   // row j of the tile -> slot j % DEPTH; one group per call
    if (j < tn) {
      const T *row = H + (size_t)s_rec[j].x * im.ldH;
      uint4 *slot = ring + (size_t)(j % DEPTH) * kSlot;
#pragma unroll
      for (int v = 0; v < VPL; ++v) {
        const int g = t + v * kMrgThreads;
        if (g < ng) {
#pragma unroll
          for (int pc = 0; pc < Q16; ++pc) {
            const unsigned dsta = (unsigned)__cvta_generic_to_shared(slot + (size_t)g * Q16 + pc);
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dsta), "l"(row + g * 8 + pc * (16 / (int)sizeof(T))) : "memory");
          }
        }
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  auto consume = [&](int j) {
    asm volatile("cp.async.wait_group %0;" ::"n"(DEPTH - 1) : "memory");
    const int4 rec = s_rec[j];
    if (rec.y != cur_c) {                            // the next cluster begins (the same for all threads)
      if (cur_c >= 0) {
        if (head_open) {                               // the cluster that began before this range ends here
          cut(acc, cur_c, cur_off, cur_size, cur_inv, cur_dst, 0);
          head_open = false;
        } else {
          store_row(acc, cur_inv, cur_dst);
        }
      } else {
        head_open = rec.z < lo;
      }
#pragma unroll
      for (int v = 0; v < VPL; ++v)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[v][e] = 0.f;
      cur_c = rec.y; cur_off = rec.z; cur_size = rec.w;
      cur_dst = s_dst[j]; cur_inv = s_inv[j];
    }
    const uint4 *slot = ring + (size_t)(j % DEPTH) * kSlot;
#pragma unroll
    for (int v = 0; v < VPL; ++v) {
      const int g = t + v * kMrgThreads;
      if (g < ng) {
        Raw8<T> x;
        x.from_ring(slot + (size_t)g * Q16);
        x.add_to(acc[v]);
      }
    }
  };
  for (int t0 = lo; t0 < hi; t0 += kMrgTile) {
    const int tn = min(kMrgTile, hi - t0);
    __syncthreads();                                 // the previous tile's records are no longer needed
    if (t < tn) {
      const int g = t0 + t;
      int4 rec;
      int dst;
      float inv = 1.f;
      if (g < n_mem) {
        if (center_only) rec = make_int4(im.cidx_ptr[g], g, g, 1);
        else rec = __ldcg(im.members + g);
        // in bounds whatever an aborted earlier stage left in the records
        rec.x = min(max(rec.x, 0), im.N - 1) + im.vis_start;     // row of H
        rec.y = min(max(rec.y, 0), C - 1);
        rec.z = min(max(rec.z, 0), g);
        rec.w = min(max(rec.w, g - rec.z + 1), n_mem - rec.z);
        dst = im.vis_start + rec.y;
        if (!center_only) inv = 1.0f / (float)rec.w;
      } else {                                       // a text row: a cluster of its own, numbered after the real ones
        const int tr = g - n_mem;
        const int src = tr < im.vis_start ? tr : tr + im.N;
        dst = tr < im.vis_start ? tr : tr + C;
        rec = make_int4(src, C + tr, g, 1);
        im.P_out[dst] = im.P[src];
        im.size_out[dst] = 1;
        if (im.logw_out) im.logw_out[dst] = 0.f;
      }
      s_rec[t] = rec;
      s_dst[t] = dst;
      s_inv[t] = inv;
    }
    __syncthreads();
    TL_POINT(im, 15);
    for (int j = 0; j < DEPTH; ++j) issue(j, tn);
#pragma unroll 1
    for (int j = 0; j < tn; ++j) {
      consume(j);
      issue(j + DEPTH, tn);
    }
  }
  if (cur_c < 0) return;                             // an empty range
  const bool goes_on = cur_off + cur_size > hi;
  if (head_open) {                                   // one cluster covers the whole range
    cut(acc, cur_c, cur_off, cur_size, cur_inv, cur_dst, goes_on ? 1 : 0);
    return;
  }
  if (goes_on) cut(acc, cur_c, cur_off, cur_size, cur_inv, cur_dst, 1);
  else store_row(acc, cur_inv, cur_dst);
}

// ---- launchers -----------------------------------------------------------------------------------

namespace {
int g_lists_resident = 0;                            // CTAs of k_lists that fit on the device at once
}

template <typename T, bool FB>
static cudaError_t launch_lists_t(const Batch &bt, int maxN, int spin_limit, cudaStream_t st) {
  const dim3 grid((maxN + kListBlock - 1) / kListBlock, bt.B);
  if ((long long)grid.x * grid.y <= g_lists_resident) {
    return launch_coop(k_lists<T, FB>, grid, dim3(kListBlock), 0, st, true, bt, 0, spin_limit);
  }
  cudaError_t e = launch_k(k_lists<T, FB>, grid, dim3(kListBlock), 0, st, true, bt, 1, spin_limit);
  if (e != cudaSuccess) return e;
  return launch_k(k_lists<T, FB>, grid, dim3(kListBlock), 0, st, true, bt, 2, spin_limit);
}

cudaError_t launch_lists(const Batch &bt, int maxN, bool bf16, bool from_best, int spin_limit, cudaStream_t st) {
  if (from_best) {
    if (bf16) return launch_lists_t<__nv_bfloat16, true>(bt, maxN, spin_limit, st);
    return launch_lists_t<float, true>(bt, maxN, spin_limit, st);
  }
  return launch_lists_t<float, false>(bt, maxN, spin_limit, st);
}

cudaError_t launch_members(const Batch &bt, int maxN, cudaStream_t st) {
  const dim3 grid((maxN + kListBlock - 1) / kListBlock, bt.B);
  return launch_k(k_members, grid, dim3(kListBlock), 0, st, true, bt);
}

int lists_kernels(int maxN, int B) {
  return (long long)((maxN + kListBlock - 1) / kListBlock) * B <= g_lists_resident ? 1 : 2;
}

int merge_ctas(int sm_count, int B) {
  const int X = kMrgCtasPerSm * sm_count / B;
  return X < 1 ? 1 : X;
}

template <typename T, typename O, int VPL>
static cudaError_t launch_merge_v(const Batch &bt, dim3 grid, cudaStream_t st) {
  constexpr int kSlotBytes = VPL * kMrgThreads * 8 * (int)sizeof(T);
  constexpr int DEPTH = kMrgRingBytes / kSlotBytes;
  return launch_k(k_merge<T, O, VPL, DEPTH>, grid, dim3(kMrgThreads), (size_t)DEPTH * kSlotBytes, st, true, bt);
}

template <typename T, typename O>
static cudaError_t launch_merge_t(const Batch &bt, const ClusterCfg &cfg, cudaStream_t st) {
  dim3 grid(merge_ctas(cfg.sm_count, bt.B), bt.B);
  if (bt.d <= kMrgThreads * 8) return launch_merge_v<T, O, 1>(bt, grid, st);
  return launch_merge_v<T, O, kMergeMaxD / 8 / kMrgThreads>(bt, grid, st);
}

template <typename T, typename O, int VPL>
static cudaError_t merge_attr() {
  constexpr int kSlotBytes = VPL * kMrgThreads * 8 * (int)sizeof(T);
  constexpr int DEPTH = kMrgRingBytes / kSlotBytes;
  return cudaFuncSetAttribute(k_merge<T, O, VPL, DEPTH>, cudaFuncAttributeMaxDynamicSharedMemorySize, DEPTH * kSlotBytes);
}

cudaError_t merge_configure() {
  int dev = 0, sms = 0, per_sm = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_lists<__nv_bfloat16, true>, kListBlock, 0);
  if (e != cudaSuccess) return e;
  int m = per_sm;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_lists<float, true>, kListBlock, 0);
  if (e != cudaSuccess) return e;
  m = per_sm < m ? per_sm : m;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_lists<float, false>, kListBlock, 0);
  if (e != cudaSuccess) return e;
  m = per_sm < m ? per_sm : m;
  g_lists_resident = m * sms;
  constexpr int V2 = kMergeMaxD / 8 / kMrgThreads;
  e = merge_attr<__nv_bfloat16, __nv_bfloat16, 1>();
  if (e == cudaSuccess) e = merge_attr<__nv_bfloat16, __nv_bfloat16, V2>();
  if (e == cudaSuccess) e = merge_attr<__nv_bfloat16, float, 1>();
  if (e == cudaSuccess) e = merge_attr<__nv_bfloat16, float, V2>();
  if (e == cudaSuccess) e = merge_attr<float, __nv_bfloat16, 1>();
  if (e == cudaSuccess) e = merge_attr<float, __nv_bfloat16, V2>();
  if (e == cudaSuccess) e = merge_attr<float, float, 1>();
  if (e == cudaSuccess) e = merge_attr<float, float, V2>();
  return e;
}

cudaError_t launch_merge(const Batch &bt, bool in_bf16, bool out_bf16, const ClusterCfg &cfg, cudaStream_t st) {
  if (in_bf16) return out_bf16 ? launch_merge_t<__nv_bfloat16, __nv_bfloat16>(bt, cfg, st)
                               : launch_merge_t<__nv_bfloat16, float>(bt, cfg, st);
  return out_bf16 ? launch_merge_t<float, __nv_bfloat16>(bt, cfg, st) : launch_merge_t<float, float>(bt, cfg, st);
}

}  // namespace pact
