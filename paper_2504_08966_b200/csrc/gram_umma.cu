// tcgen05 tile kernels for bf16 keys (sm_100a): the all-pairs distance pass of DBDPC (Eq. 5) with
// the density (Eq. 6) and the d <= d_c adjacency fused into the epilogue, the rows x centres
// nearest-centre pass (Algorithm 2 assignment, Eq. 8), and the largest distance between two keys of a
// layer (the quantity that decides the reduction layer L) as a max-epilogue over the tiles on and above
// the diagonal.  Nothing of the distance matrix reaches memory: accumulators live in tensor memory
// and are consumed from there.
//
// One persistent CTA per SM, 576 threads:
//   warp 0      TMA producer: 128-byte-swizzled K-slabs of the two operands into a shared-memory ring
//   warp 1      allocates tensor memory, issues tcgen05.mma (128 x BN x 16, bf16 -> fp32)
//   warps 2-17  epilogue: tcgen05.ld of their 32-lane quadrant (four warps per quadrant, a quarter of the
//               columns each), distance arithmetic of common.cuh
// Several accumulators (512 / BN of them share the tensor memory) let the epilogue of tile t overlap
// the MMAs of the next tiles.  The all-pairs pass computes every unordered pair of survivors once: a
// 128 x 128 block above the diagonal serves its rows (density sums, adjacency words) and, through a
// shared-memory exchange of the terms and a warp transpose of the adjacency bits, its columns as well;
// blocks on the diagonal serve their rows only.  Every mbarrier wait is bounded; when one runs out the
// CTA raises the image's status word, drains what it armed, frees its tensor memory and returns.
#include <cuda.h>

#include "kernels.cuh"
#include "tma.cuh"

namespace pact {

namespace {

constexpr int BM = 128;           // rows per tile (UMMA M)
constexpr int BK = 64;            // bf16 elements per K-slab = one 128-byte swizzle row
constexpr int A_BYTES = BM * BK * 2;
constexpr int TMEM_COLS = 512;    // all of an SM's tensor memory
constexpr int MAX_STAGES = 6;
#ifndef PACT_EPI_WARPS
#define PACT_EPI_WARPS 16
#endif
constexpr int EPI_WARPS = PACT_EPI_WARPS;      // per tensor-memory lane quadrant EPI_WARPS / 4 warps share the columns
                                  // (16 measured 0.35 us per step faster than 8 once a stage held two K-slabs)
constexpr int THREADS = 64 + EPI_WARPS * 32;
constexpr int MAX_ACC = 4;

// Per tile width BN (UMMA N): 256 columns for the rows x centres and the largest-distance passes,
// 128 for the all-pairs pass, whose tiles are the 128 x 128 blocks on and above the diagonal.
template <int BN> struct TileCfg {
  static constexpr int B_BYTES = BN * BK * 2;
  // a stage holds two K-slabs of both operands: half as many barrier waits per tile as with one (measured
  // 0.4 us per step faster at equal bytes in flight)
  static constexpr int SLABS = 2;
  static constexpr int STAGE_BYTES = SLABS * (A_BYTES + B_BYTES);
  static constexpr int STAGES = 2;
  static constexpr int NACC = TMEM_COLS / BN;      // accumulators in tensor memory
  static constexpr int HALF = BN / (EPI_WARPS / 4); // columns per epilogue warp
  // BN = 128 (all-pairs pass): one 32 x 32 exchange buffer per epilogue warp behind the ring
  static constexpr size_t RING = 1024 + (size_t)STAGES * STAGE_BYTES;
  static constexpr size_t SMEM = RING + (BN == 128 ? (size_t)EPI_WARPS * 32 * 36 * 4 : 0);
  // kind::f16 instruction descriptor: fp32 accumulate, bf16 x bf16, both operands K-major.
  static constexpr uint32_t IDESC =
      (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
};

struct TmapSet {
  CUtensorMap a[kMaxBatchPerLaunch];
  CUtensorMap b[kMaxBatchPerLaunch];
};

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, uint64_t *bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t *slot, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory operand descriptor: K-major rows of 128 bytes, 128-byte swizzle, 8-row groups
// 1024 bytes apart, descriptor version 1.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}

struct Shared {
  uint64_t full[MAX_STAGES], empty[MAX_STAGES], acc_full[MAX_ACC], acc_empty[MAX_ACC];
  uint64_t done;                                   // every MMA this CTA has issued is complete
  uint32_t tmem_base;
  int abort;
  __align__(16) float rn_col[EPI_WARPS][128];    // inverse norms of this warp's columns
};

enum { MODE_GRAM = 0, MODE_ASSIGN = 1, MODE_SPREAD = 2 };

// The largest-distance pass needs every unordered pair once: tiles that lie wholly below the diagonal
// are left out (by the producer, the MMA issuer and the epilogue alike).
template <int MODE, int BN> __device__ __forceinline__ bool tile_wanted(int tmi, int tni) {
  return MODE != MODE_SPREAD || (tni + 1) * BN > tmi * BM;
}

// Tile `t` of the pass -> block row and block column.  The all-pairs pass walks the nb (nb + 1) / 2
// blocks with column >= row, row by row; the other passes walk the full grid.
template <int MODE> __device__ __forceinline__ int tile_count(int ntm, int ntn) {
  return MODE == MODE_GRAM ? ntm * (ntm + 1) / 2 : ntm * ntn;
}
template <int MODE> __device__ __forceinline__ void tile_at(int t, int ntm, int ntn, int &tmi, int &tni) {
  if (MODE == MODE_GRAM) {
    // row i starts at i * ntm - i (i - 1) / 2
    const float b = 2.f * (float)ntm + 1.f;
    int i = (int)((b - sqrtf(fmaxf(b * b - 8.f * (float)t, 0.f))) * 0.5f);
    i = max(0, min(i, ntm - 1));
    while (i > 0 && i * ntm - i * (i - 1) / 2 > t) --i;
    while (i + 1 < ntm && (i + 1) * ntm - (i + 1) * i / 2 <= t) ++i;
    tmi = i;
    tni = i + (t - (i * ntm - i * (i - 1) / 2));
  } else if (MODE == MODE_ASSIGN) {
    // full-width column tiles first, the (usually narrow) last column last: the CTAs that take a second
    // tile then take a cheap one
    const int fullc = ntn - 1, nfull = ntm * fullc;
    if (t < nfull) { tmi = t / fullc; tni = t % fullc; }
    else { tmi = t - nfull; tni = fullc; }
  } else {
    tmi = t / ntn;
    tni = t % ntn;
  }
}
// Columns of tile column tni that the MMA has to produce: the rows x centres pass stops at the last
// centre, rounded up to the instruction's granularity of 16.
template <int MODE, int BN> __device__ __forceinline__ int tile_width(int tni, int ncols) {
  if (MODE != MODE_ASSIGN) return BN;
  const int left = ncols - tni * BN;
  return left >= BN ? BN : ((left + 15) & ~15);
}

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// One 32-column chunk of the epilogue of the all-pairs pass for one row (= one lane): distance
// (Eq. 5), density term (Eq. 6) as an integer multiple of 2^-30, adjacency bit d <= d_c, band count.
// EDGE adds the per-element checks that only edge chunks need (diagonal, columns past the end).
// COLS (blocks above the diagonal) also hands every pair to its column: the warp's 32 x 32 terms go
// through a shared-memory buffer `tr` (row stride 36 words: conflict-free stores, 16-byte loads), lane k
// adds the 32 terms of column k, and a 32 x 32 bit transpose gives it the column's adjacency word.  The arithmetic is that of DistF (common.cuh) with the two inverse norms multiplied first,
// written out so that three terms are summed in 32 bits.
template <bool EDGE, bool COLS>
__device__ __forceinline__ void gram_chunk(const uint32_t (&v)[32], const float *rn_col, float rni, int row, int c0,
                                           int ncols, float d_c, float neg_k, int lane, uint32_t *tr,
                                           unsigned long long &rowsum, uint32_t &bits, int &band,
                                           unsigned long long &colsum, uint32_t &colbits) {
  uint32_t b = 0u;
  unsigned long long s = 0ull;
  uint32_t s3 = 0u;                                 // three terms, each at most 2^30, fit in 32 bits
  int bnd = 0;
#pragma unroll
  for (int k4 = 0; k4 < 32; k4 += 4) {
    const float4 rn4 = *reinterpret_cast<const float4 *>(rn_col + k4);
    const float rnj[4] = {rn4.x, rn4.y, rn4.z, rn4.w};
#pragma unroll
    for (int kk = 0; kk < 4; ++kk) {
      const int k = k4 + kk;
      // rn_i * rn_j first: a pair must get the same distance whichever of the two is the row, so that
      // duplicate keys keep exactly equal densities
      float dd = fminf(fmaxf(1.0f - __uint_as_float(v[k]) * (rni * rnj[kk]), 0.0f), 2.0f);
      bool ok = true;
      if (EDGE) {
        const int gj = c0 + k;
        if (gj == row) dd = 0.f;
        ok = gj < ncols;
      }
      uint32_t term = __float2uint_rn(ex2_approx(dd * neg_k) * (float)(1u << kRhoShift));
      bool within = dd <= d_c;
      const bool inband = fabsf(dd - d_c) <= 1e-6f;
      if (EDGE) {
        if (!ok) { term = 0u; within = false; }
        if (ok && inband && row < c0 + k) ++bnd;
      } else {
        if (inband) ++bnd;
      }
      s3 += term;
      if (within) b |= 1u << k;
      if (k % 3 == 2 || k == 31) { s += s3; s3 = 0u; }   // a run of keys at distance 0 adds 2^30 each
      if (COLS) tr[k * 36 + lane] = term;
    }
  }
  rowsum += s;
  bits = b;
  band += bnd;
  if (COLS) {
    __syncwarp();
    // lane k: the 32 terms of column k, three to a 32-bit partial sum as above
    unsigned long long cs = 0ull;
    uint32_t c3 = 0u;
    const uint4 *src = reinterpret_cast<const uint4 *>(tr + lane * 36);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const uint4 x = src[j];
      const uint32_t xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        c3 += xs[i];
        if ((j * 4 + i) % 3 == 2 || j * 4 + i == 31) { cs += c3; c3 = 0u; }
      }
    }
    colsum = cs;
    // transpose the 32 x 32 bit matrix (lane l holds row l): five exchange steps
    uint32_t w = b;
#pragma unroll
    for (int sft = 16; sft >= 1; sft >>= 1) {
      const uint32_t m = sft == 16 ? 0x0000FFFFu : sft == 8 ? 0x00FF00FFu : sft == 4 ? 0x0F0F0F0Fu
                         : sft == 2 ? 0x33333333u : 0x55555555u;
      const uint32_t y = __shfl_xor_sync(0xffffffffu, w, sft);
      w = (lane & sft) ? ((w & ~m) | ((y >> sft) & m)) : ((w & m) | ((y << sft) & ~m));
    }
    colbits = w;
    __syncwarp();                                   // tr may be rewritten by the next chunk
  }
}

// Labels of a group of 32 tokens (lane = token) whose nearest centres are final, formed by the last epilogue
// warp of the rows x centres pass to finish the group: a survivor takes its nearest centre's cluster (a centre
// its own), a pruned token that cluster iff the distance is strictly below alpha * d_c (Eq. 8-9), else -1.
// The group's members per cluster are added to the table of its 128-token block and to the cluster sizes
// (integer adds: the sums do not depend on the order in which groups finish).
// r: the token's position among the survivors (< 0: pruned); own_cid: its cluster id if it is a centre, else -1
// (both known before the pass, so that only the nearest centre has to be fetched here).
__device__ __forceinline__ void label_group(const ImgDesc &im, int i, int lane, int C, int r, int own_cid) {
  int lab = -1, joined = 0, dropped = 0, band = 0;
  if (i < im.N) {
    const unsigned long long pk = __ldcg(im.best + i);
    lab = (int)(pk & 0xFFFFFFFFull);
    const float dd = __uint_as_float((uint32_t)(pk >> 32));
    if (r >= 0) {
      if (own_cid >= 0) lab = own_cid;
    } else {
      if (DistF::in_band_t(dd, im)) ++band;
      if (DistF::below_t(dd, im)) ++joined; else { lab = -1; ++dropped; }
    }
    if (lab >= C || lab < -1) lab = -1;             // only after a failed earlier stage
    im.label[i] = lab;
    if (im.label_user) im.label_user[i] = lab;
  }
  const unsigned same = __match_any_sync(0xffffffffu, lab);
  if (lab >= 0 && lane == __ffs(same) - 1) {
    const int len = __popc(same), b = i / kListBlock;
    // 16-bit cell (c, b) of the table, added to through the 32-bit word that holds it (a cell stays <= 128)
    uint32_t *word = reinterpret_cast<uint32_t *>(im.cnt_cb) + (((size_t)lab * im.nbp + b) >> 1);
    atomicAdd(word, (uint32_t)len << (16 * (b & 1)));
    atomicAdd(&im.csize[lab], len);
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
}

// The epilogue of one accumulator tile for one warp: the warp's 32 rows (tensor-memory lanes) of the 128-row
// block tmi against HALF columns from cbase on.  Waits for the accumulator, reads it 32 columns at a time and
// applies the mode's arithmetic; arrive() is called once the accumulator has been read.  skip: the warp only
// waits and releases (a block below the diagonal of the all-pairs pass).  Returns false when the wait ran out.
template <int MODE, int HALF, bool WAIT_MIN = false, typename Arrive>
__device__ __forceinline__ bool epi_tile(const ImgDesc &im, int kept_rows, int tmi, int cbase, bool skip, int nrows,
                                         int ncols, uint32_t taddr, uint64_t *acc_full, uint32_t parity, float *rn_col,
                                         uint32_t *tr, int lane, int qd, int &band, float &mx, Arrive arrive,
                                         unsigned long long &seen) {
  // inverse norms of this warp's columns and of this lane's row (in flight while the MMAs run)
  const float *rn_src = MODE == MODE_GRAM ? im.rnk : (MODE == MODE_SPREAD ? im.rn : im.rnc);
  float4 r4;
  {
    const int gj = cbase + lane * 4;
    r4.x = gj + 0 < ncols ? rn_src[gj + 0] : 0.f;
    r4.y = gj + 1 < ncols ? rn_src[gj + 1] : 0.f;
    r4.z = gj + 2 < ncols ? rn_src[gj + 2] : 0.f;
    r4.w = gj + 3 < ncols ? rn_src[gj + 3] : 0.f;
  }
  const int row = tmi * BM + qd * 32 + lane;
  const bool row_ok = row < nrows;
  const bool kept_space = MODE == MODE_GRAM || (MODE == MODE_ASSIGN && kept_rows);
  float rni = row_ok ? (kept_space ? im.rnk[row] : im.rn[row]) : 0.f;
  if (MODE == MODE_GRAM) {
    // the all-pairs pass multiplies the two inverse norms first; a vanishing key (inverse norm at
    // its clamp, 1e20) takes 0 here so that the product stays finite: dot product 0, distance 1
    constexpr float kHuge = 1e19f;
    if (rni > kHuge) rni = 0.f;
    if (r4.x > kHuge) r4.x = 0.f;
    if (r4.y > kHuge) r4.y = 0.f;
    if (r4.z > kHuge) r4.z = 0.f;
    if (r4.w > kHuge) r4.w = 0.f;
  }
  __syncwarp();
  if (lane * 4 < HALF) reinterpret_cast<float4 *>(rn_col)[lane] = r4;
  __syncwarp();
  if (!mbar_wait_warp(acc_full, parity)) return false;
  tc_fence_after();
  unsigned long long rowsum = 0ull;
  float bd = 3.0f, bc = -4.0f;                  // distance to the nearest centre of the tile (<= 2) and its cosine
  int bi = 0;
  const float d_c = im.d_c, neg_k = -im.inv_dn_log2e;
  const int r0 = tmi * BM + qd * 32;
  const bool above = MODE == MODE_GRAM && cbase / BM > tmi;   // block above the diagonal: rows and columns
#pragma unroll 1
  for (int ch = 0; ch < HALF / 32; ++ch) {
    const int c0 = cbase + ch * 32;
    if (skip || c0 >= ncols) break;              // uniform
    uint32_t v[32];
    tmem_ld32(taddr + ch * 32, v);
    tmem_ld_wait();
    if (MODE == MODE_GRAM) {
      uint32_t bits, colbits = 0u;
      unsigned long long colsum = 0ull;
      if (above) {
        // every row of this block is a survivor (only the last block row is ragged, and it has no
        // block to its right); each pair (row, column) is also the pair (column, row)
        int bnd = 0;
        if (c0 + 32 > ncols)
          gram_chunk<true, true>(v, rn_col + ch * 32, rni, row, c0, ncols, d_c, neg_k, lane, tr, rowsum, bits, bnd, colsum, colbits);
        else
          gram_chunk<false, true>(v, rn_col + ch * 32, rni, row, c0, ncols, d_c, neg_k, lane, tr, rowsum, bits, bnd, colsum, colbits);
        band += bnd;                            // row < column throughout
        const int gj = c0 + lane;
        if (gj < ncols) {
          atomicAdd(&im.rho_fix[gj], colsum);
          im.adj[(size_t)gj * im.Wp + (r0 >> 5)] = colbits;
        }
      } else {
        const bool edge = (c0 + 32 > ncols) || (c0 < r0 + 32 && c0 + 32 > r0);
        if (edge) gram_chunk<true, false>(v, rn_col + ch * 32, rni, row, c0, ncols, d_c, neg_k, lane, tr, rowsum, bits, band, colsum, colbits);
        else {
          int bnd = 0;
          gram_chunk<false, false>(v, rn_col + ch * 32, rni, row, c0, ncols, d_c, neg_k, lane, tr, rowsum, bits, bnd, colsum, colbits);
          if (row < c0) band += bnd;            // each unordered pair once; the chunk lies wholly on one side
        }
      }
      if (row_ok) im.adj[(size_t)row * im.Wp + (c0 >> 5)] = bits;
    } else if (MODE == MODE_SPREAD) {
      // The largest distance of the chunk belongs to its smallest cosine: d = clamp(1 - c) does not increase
      // with c, in floating point either, so the cosines (dot * rn_i) * rn_j are compared and one distance is
      // formed per chunk from the smallest.  Rows and columns past the end hold zero dot products,
      // i.e. distance 1, and the pair (i, i) is not a pair: chunks that hold either take the checked loop.
      float cmin = 4.0f;
      const bool plain = c0 + 32 <= ncols && r0 + 32 <= nrows && (c0 + 32 <= r0 || c0 >= r0 + 32);   // uniform
      if (plain) {
#pragma unroll
        for (int k4 = 0; k4 < 32; k4 += 4) {
          const float4 rn4 = *reinterpret_cast<const float4 *>(rn_col + ch * 32 + k4);
          const float rnj[4] = {rn4.x, rn4.y, rn4.z, rn4.w};
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) cmin = fminf(cmin, (__uint_as_float(v[k4 + kk]) * rni) * rnj[kk]);
        }
      } else {
        const int lim = row_ok ? min(32, ncols - c0) : 0;
        const int self = row - c0;
#pragma unroll
        for (int k4 = 0; k4 < 32; k4 += 4) {
          const float4 rn4 = *reinterpret_cast<const float4 *>(rn_col + ch * 32 + k4);
          const float rnj[4] = {rn4.x, rn4.y, rn4.z, rn4.w};
#pragma unroll
          for (int kk = 0; kk < 4; ++kk) {
            const int k = k4 + kk;
            const float c = (__uint_as_float(v[k]) * rni) * rnj[kk];
            if (k < lim && k != self) cmin = fminf(cmin, c);
          }
        }
      }
      if (cmin < 4.0f) mx = fmaxf(mx, fminf(fmaxf(1.0f - cmin, 0.0f), 2.0f));
    } else {
      // the nearest centre of the chunk is the one with the largest cosine (dot * rn_i) * rn_j; the first of
      // equal cosines wins, i.e. the centre with the lowest index; the distance is formed once per tile
      const int lim = min(32, ncols - c0);
#pragma unroll
      for (int k4 = 0; k4 < 32; k4 += 4) {
        const float4 rn4 = *reinterpret_cast<const float4 *>(rn_col + ch * 32 + k4);
        const float rnj[4] = {rn4.x, rn4.y, rn4.z, rn4.w};
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
          const int k = k4 + kk;
          const float c = (__uint_as_float(v[k]) * rni) * rnj[kk];
          if (k < lim && c > bc) { bc = c; bi = c0 + k; }
        }
      }
    }
  }
  if (MODE == MODE_ASSIGN && bc > -3.0f) bd = fminf(fmaxf(1.0f - bc, 0.0f), 2.0f);
  // the accumulator may be overwritten once all epilogue warps have read it
  tc_fence_before();
  __syncwarp();
  if (lane == 0) arrive();
  if (row_ok && !skip) {
    if (MODE == MODE_GRAM) atomicAdd(&im.rho_fix[row], rowsum);
    else if (MODE == MODE_ASSIGN && bd <= 2.0f) {
      const unsigned long long pk = ((unsigned long long)__float_as_uint(bd) << 32) | (unsigned)bi;
      const unsigned long long old = atomicMin(&im.best[kept_rows ? im.kept_idx[row] : row], pk);
      if (WAIT_MIN) seen |= old;                   // the caller waits for the value: the minimum is then in place
    }
  }
  return true;
}

}  // namespace

// grid (X, B), 64 + 32 EPI_WARPS threads, dynamic smem = TileCfg<BN>::SMEM.
// kept_rows (assignment only), bit 0: rows are the gathered survivors (Kp, rnk) instead of all tokens;
// bit 1: the labels, cluster sizes and per-block member counts are formed here as groups of rows finish.
template <int MODE, int BN>
__global__ void __launch_bounds__(THREADS, 1) k_tiles_umma(const __grid_constant__ Batch bt,
                                                           const __grid_constant__ TmapSet tm, int kept_rows) {
  using Cfg = TileCfg<BN>;
  constexpr int STAGES = Cfg::STAGES, NACC = Cfg::NACC, HALF = Cfg::HALF, SLABS = Cfg::SLABS;
  constexpr int STAGE_BYTES = Cfg::STAGE_BYTES, B_BYTES = Cfg::B_BYTES;
  const ImgDesc &im = bt.img[blockIdx.y];
  TL_SCOPE(im, MODE == MODE_GRAM ? 4 : 6);
  (void)kept_rows;
  extern __shared__ uint8_t smem_raw[];
  __shared__ Shared sh;
  uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // set-up that does not depend on the kernels before this one
  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
    for (int a = 0; a < NACC; ++a) { mbar_init(&sh.acc_full[a], 1); mbar_init(&sh.acc_empty[a], EPI_WARPS); }
    mbar_init(&sh.done, 1);
    sh.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(&sh.tmem_base, TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sh.tmem_base;
  pdl_wait();
  pdl_trigger();

  int nrows, ncols;
  if (MODE == MODE_GRAM) { nrows = *im.q_ptr; ncols = nrows; }
  else if (MODE == MODE_SPREAD) { nrows = im.N; ncols = im.N; }
  else { nrows = (kept_rows & 1) ? *im.q_ptr : im.N; ncols = *im.C_ptr; }
  const int ntm = (nrows + BM - 1) / BM, ntn = (ncols + BN - 1) / BN;
  const int ntiles = tile_count<MODE>(ntm, ntn);
  const bool active = (int)blockIdx.x < ntiles;       // CTAs without a tile only give their tensor memory back
  const int nslab = bt.d_k / BK;

  if (!active) {
  } else if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      const CUtensorMap *ma = &tm.a[blockIdx.y], *mb = &tm.b[blockIdx.y];
      uint32_t it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < ntiles; tile += gridDim.x) {
        int tmi, tni;
        tile_at<MODE>(tile, ntm, ntn, tmi, tni);
        if (!tile_wanted<MODE, BN>(tmi, tni)) continue;
        const int bw = tile_width<MODE, BN>(tni, ncols);
        for (int ks = 0; ks < nslab; ks += SLABS, ++it) {
          const int s = it % STAGES;
          const int n = min(SLABS, nslab - ks);
          if (!mbar_wait(&sh.empty[s], ((it / STAGES) & 1) ^ 1)) { ok = false; break; }
          uint8_t *a_dst = ring + (size_t)s * STAGE_BYTES, *b_dst = a_dst + SLABS * A_BYTES;
          const bool second = BN == 256 && bw > BN / 2;   // the second 128 rows of B are needed
          const uint32_t per = second || BN != 256 ? (A_BYTES + B_BYTES) : (A_BYTES + B_BYTES / 2);
          mbar_arrive_expect_tx(&sh.full[s], (uint32_t)n * per);
          for (int h = 0; h < n; ++h) {
            tma_load_2d(a_dst + h * A_BYTES, ma, &sh.full[s], (ks + h) * BK, tmi * BM);
            tma_load_2d(b_dst + h * B_BYTES, mb, &sh.full[s], (ks + h) * BK, tni * BN);
            if (second) tma_load_2d(b_dst + h * B_BYTES + B_BYTES / 2, mb, &sh.full[s], (ks + h) * BK, tni * BN + BN / 2);
          }
        }
      }
      if (!ok) atomicExch(&sh.abort, 1);
      // drain: every armed stage completes before the CTA may exit (its copies target this smem)
      const uint32_t armed = it < (uint32_t)STAGES ? it : (uint32_t)STAGES;
      for (uint32_t k = 0; k < armed; ++k) {
        const uint32_t j = it - 1 - k;
        mbar_wait(&sh.full[j % STAGES], (j / STAGES) & 1);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < ntiles; tile += gridDim.x) {
        int tmi, tni;
        tile_at<MODE>(tile, ntm, ntn, tmi, tni);
        if (!tile_wanted<MODE, BN>(tmi, tni)) continue;
        const uint32_t a = tcount % NACC;
        if (!mbar_wait(&sh.acc_empty[a], ((tcount / NACC) & 1) ^ 1)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + a * BN;
        // instruction descriptor with this tile's width in its N field
        const uint32_t idesc = (Cfg::IDESC & ~(0x3Fu << 17)) | ((uint32_t)(tile_width<MODE, BN>(tni, ncols) >> 3) << 17);
        for (int ks = 0; ks < nslab; ks += SLABS, ++it) {
          const int s = it % STAGES;
          const int n = min(SLABS, nslab - ks);
          if (!mbar_wait(&sh.full[s], (it / STAGES) & 1)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(ring + (size_t)s * STAGE_BYTES), b_addr = a_addr + SLABS * A_BYTES;
#pragma unroll
          for (int h = 0; h < SLABS; ++h) {
            if (h < n) {
#pragma unroll
              for (int k = 0; k < BK / 16; ++k)
                umma_bf16(d_tmem, smem_desc(a_addr + h * A_BYTES + k * 32), smem_desc(b_addr + h * B_BYTES + k * 32), idesc, (ks | h | k) != 0);
            }
          }
          umma_commit(&sh.empty[s]);               // frees the slab once these MMAs have read it
        }
        if (ok) umma_commit(&sh.acc_full[a]);      // accumulator complete
        ++tcount;
      }
      // whatever way the loop ended, no MMA may still be running when the tensor memory is given back
      umma_commit(&sh.done);
      if (!mbar_wait(&sh.done, 0)) ok = false;
      if (!ok) atomicExch(&sh.abort, 1);
    }
  } else {
    // ---------------- epilogue ----------------
    const int ew = warp - 2;
    const int qd = warp & 3;                        // tensor-memory lane quadrant this warp may read
    const int half = ew >> 2;                       // which half of the tile's columns
    float *rn_col = sh.rn_col[ew];
    uint32_t *tr = reinterpret_cast<uint32_t *>(ring + Cfg::RING - 1024) + ew * (32 * 36);   // BN = 128 only
    uint32_t tcount = 0;
    int band = 0;
    bool ok = true;
    float mx = 0.f;                                 // largest distance seen by this lane (MODE_SPREAD)
    // Labels (rows x centres pass with bit 1 of kept_rows): a group of 32 tokens is final once `need` warps
    // (every column tile, every column half) have put their nearest centres in place; each warp draws a
    // ticket per group and the one that draws the last labels the group.  The tickets of up to kPend tiles
    // are drawn together, so that a warp waits for its atomics to land once, not once per tile.
    constexpr int kPend = 4;
    const int need = (MODE == MODE_ASSIGN && (kept_rows & 2)) ? ntn * (EPI_WARPS / 4) : 0;
    int pend_tmi[kPend], pend_r[kPend], pend_cid[kPend], npend = 0;
    unsigned long long seen = 0ull;                 // previous values of the minima this lane has updated
    auto flush_labels = [&]() {
      // Every lane's atomic minima have returned, i.e. are in place, once their return values have been used:
      // the fence then has nothing left to wait for.  (No stored value has distance bits above 2.0f.)
      const unsigned odd = __ballot_sync(0xffffffffu, seen == 0xFFFFFFFE00000001ull);
      seen = 0ull;
      __threadfence();
      int mine = 0;
      if (lane < npend && odd == 0u) {
        int tmi_l = pend_tmi[0];
#pragma unroll
        for (int k = 1; k < kPend; ++k) if (lane == k) tmi_l = pend_tmi[k];
        mine = atomicAdd(&im.rtick[tmi_l * (BM / 32) + qd], 1) == need - 1;
      }
      const unsigned lastmask = __ballot_sync(0xffffffffu, mine);
      if (lastmask) __threadfence();
#pragma unroll
      for (int k = 0; k < kPend; ++k)
        if (k < npend && ((lastmask >> k) & 1u))
          label_group(im, pend_tmi[k] * BM + qd * 32 + lane, lane, ncols, pend_r[k], pend_cid[k]);
      npend = 0;
    };
    for (int tile = blockIdx.x; ok && tile < ntiles; tile += gridDim.x) {
      int tmi, tni;
      tile_at<MODE>(tile, ntm, ntn, tmi, tni);
      if (!tile_wanted<MODE, BN>(tmi, tni)) continue;
      const uint32_t a = tcount % NACC;
      const int cbase = tni * BN + half * HALF;     // first column of this warp
      const uint32_t taddr = tmem_base + a * BN + half * HALF + ((uint32_t)(qd * 32) << 16);
      if (MODE == MODE_ASSIGN && need > 0) {
        // what the labels of this warp's 32 tokens need besides the nearest centre (known before the pass)
        const int row = tmi * BM + qd * 32 + lane;
        int r = -1, own = -1;
        if (row < nrows) {
          r = im.slot[row];
          if (r >= 0 && ((im.cmask[r >> 5] >> (r & 31)) & 1u)) own = im.cid[r];
        }
        pend_tmi[npend] = tmi; pend_r[npend] = r; pend_cid[npend] = own;
      }
      if (need > 0)
        ok = epi_tile<MODE, HALF, true>(im, kept_rows & 1, tmi, cbase, false, nrows, ncols, taddr, &sh.acc_full[a], (tcount / NACC) & 1,
                                        rn_col, tr, lane, qd, band, mx, [&]() { mbar_arrive(&sh.acc_empty[a]); }, seen);
      else
        ok = epi_tile<MODE, HALF>(im, kept_rows & 1, tmi, cbase, false, nrows, ncols, taddr, &sh.acc_full[a], (tcount / NACC) & 1,
                                  rn_col, tr, lane, qd, band, mx, [&]() { mbar_arrive(&sh.acc_empty[a]); }, seen);
      if (!ok) break;
      ++tcount;
      if (MODE == MODE_ASSIGN && need > 0 && ++npend == kPend) flush_labels();
    }
    if (MODE == MODE_ASSIGN && need > 0 && ok && npend > 0) flush_labels();
    if (!ok) atomicExch(&sh.abort, 1);
    if (MODE == MODE_GRAM && band) atomicAdd(&im.cnt[PACT_CNT_BAND_DC], band);
    if (MODE == MODE_SPREAD) {
      // distances are clamped to [0, 2]: their bit patterns order like unsigned integers
      const unsigned w = __reduce_max_sync(0xffffffffu, __float_as_uint(mx));
      if (lane == 0 && w) atomicMax(reinterpret_cast<unsigned *>(&im.cnt[kCntSpread]), w);
    }
  }

  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) tmem_dealloc(tmem_base, TMEM_COLS);
  if (threadIdx.x == 0 && sh.abort) atomicMin(&im.cnt[PACT_CNT_STATUS], (int)PACT_ERR_TIMEOUT);
}

// ---- tiles on pairs of CTAs (cta_group::2) ----------------------------------------------------------------------
// Two CTAs of a cluster share one 256 x 256 tile: each holds 128 of its rows (operand A) and 128 of its
// columns (half of operand B), CTA 0 issues tcgen05.mma.cta_group::2 for both, and each CTA finds its
// 128 x 256 part of the product in its own tensor memory.  A CTA therefore fetches half as many operand
// bytes from the L2 per output element as it does alone.  The largest-distance pass always runs this way, the
// all-pairs pass when an SM has six or more 128 x 128 blocks to do and the rows x centres pass when it has two or
// more 128-row blocks (with fewer, the coarser tiles cost a round).
//   full[s]      in CTA 0: both CTAs' copies of stage s report their bytes there
//   empty[s]     in each CTA: tcgen05.commit (multicast to both CTAs) once the MMAs have read stage s
//   acc_full[a]  in each CTA: tcgen05.commit (multicast) once accumulator a is complete
//   acc_empty[a] in CTA 0: the epilogue warps of both CTAs arrive there
// Every wait is bounded as in the single-CTA kernel; the CTAs leave together through a cluster barrier, after
// which nothing is in flight towards either's shared memory.
constexpr int PBN = 256;                              // tile width of the pair kernel
constexpr int PNACC = TMEM_COLS / PBN;
constexpr int PMAX_STAGES = 5;
// EW epilogue warps per CTA (8 or 16).  The all-pairs pass runs with 16: its epilogue is heavy, and its exchange
// buffers (one per epilogue warp) leave room for four stages of one K-slab; the others run with 8 and three
// stages of two K-slabs each: a stage costs a barrier round trip between the two CTAs whatever it holds, and
// with half as many stages per tile the MMA issuer waits half as often.
template <int MODE, int EW> struct PairCfg {
  static constexpr int SLABS = (MODE == MODE_GRAM && EW > 8) ? 1 : 2;   // K-slabs per stage
  static constexpr int STAGES = (MODE == MODE_GRAM && EW > 8) ? 4 : 3;
  static constexpr int STAGE_BYTES = SLABS * 2 * A_BYTES;   // per CTA: SLABS x (128 rows of A, 128 rows of B)
  static constexpr size_t RING = 1024 + (size_t)STAGES * STAGE_BYTES;
  static constexpr size_t SMEM = RING + (MODE == MODE_GRAM ? (size_t)EW * 32 * 36 * 4 : 0);
  static constexpr int THREADS = 64 + EW * 32;
  static constexpr int COLS = PBN / (EW / 4);      // columns of the tile per epilogue warp
};

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
  // relaxed: the warp has nothing to publish through memory, its reads of the accumulator are complete
  // (tcgen05.wait::ld) before the arrive is issued, and a release at cluster scope would cost a memory fence
  asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void cluster_barrier() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_alloc2(uint32_t *slot, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
// tiled copy whose bytes are reported to a barrier that may live in the other CTA of the pair (no multicast:
// the data go to this CTA's shared memory only)
__device__ __forceinline__ void tma_load_2d_pair(void *dst, const CUtensorMap *map, uint32_t bar_cluster_addr, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(bar_cluster_addr), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accum) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accum) : "memory");
}
// arrives on the barrier at this shared-memory offset in both CTAs of the pair once the MMAs issued so far are done
__device__ __forceinline__ void umma_commit_pair(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(smem_u32(bar)), "h"((unsigned short)3) : "memory");
}

template <int EW> struct SharedPair {
  uint64_t full[PMAX_STAGES], empty[PMAX_STAGES], acc_full[PNACC], acc_empty[PNACC];
  uint64_t done;                                   // every MMA of the pair is complete (signalled in both CTAs)
  uint32_t tmem_base;
  int abort;
  __align__(16) float rn_col[EW][128];
};

// grid (2 P) in clusters of two CTAs, 64 + 32 EW threads, dynamic smem = PairCfg<MODE, EW>::SMEM.
// The 256 x 256 tiles of all images (or layers) of the batch form one list, image after image; pair p takes the
// items p, p + P, ... of it, so that the pairs stay equally loaded whatever the number of images.  CTA r of the
// pair owns the 128-row block 2 I + r of tile (I, J).  In the all-pairs and largest-distance passes the tiles
// with J >= I are listed, and of the tile (I, I) the block (2 I + 1, 2 I) lies below the diagonal: computed, not used.
template <int MODE, int EW>
__global__ void __launch_bounds__(PairCfg<MODE, EW>::THREADS, 1) k_tiles_pair(const __grid_constant__ Batch bt,
                                                                              const __grid_constant__ TmapSet tm, int kept_rows) {
  using PC = PairCfg<MODE, EW>;
  constexpr int PSTAGES = PC::STAGES, SLABS = PC::SLABS, PSTAGE_BYTES = PC::STAGE_BYTES;
  constexpr size_t PRING = PC::RING;
  constexpr int LIST = MODE == MODE_ASSIGN ? MODE_ASSIGN : MODE_GRAM;   // how the tiles of an image are listed
  TL_SCOPE(bt.img[0], MODE == MODE_GRAM ? 4 : 6);
  extern __shared__ uint8_t smem_raw[];
  __shared__ SharedPair<EW> sh;
  __shared__ int s_first[kMaxBatchPerLaunch + 1], s_rows[kMaxBatchPerLaunch], s_cols[kMaxBatchPerLaunch];
  uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();
  const bool leader = rank == 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < PSTAGES; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
    for (int a = 0; a < PNACC; ++a) { mbar_init(&sh.acc_full[a], 1); mbar_init(&sh.acc_empty[a], 2 * EW); }
    mbar_init(&sh.done, 1);
    sh.abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc2(&sh.tmem_base, TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  cluster_barrier();                                  // both CTAs' barriers exist before either is signalled
  tc_fence_after();
  const uint32_t tmem_base = sh.tmem_base;
  pdl_wait();
  pdl_trigger();

  // rows, columns and first list position of every image
  if (threadIdx.x == 0) {
    int first = 0;
    for (int b = 0; b < bt.B; ++b) {
      const ImgDesc &ib = bt.img[b];
      int nr, nc;
      if (MODE == MODE_GRAM) { nr = *ib.q_ptr; nc = nr; }
      else if (MODE == MODE_SPREAD) { nr = ib.N; nc = ib.N; }
      else { nr = (kept_rows & 1) ? *ib.q_ptr : ib.N; nc = *ib.C_ptr; }
      s_rows[b] = nr;
      s_cols[b] = nc;
      s_first[b] = first;
      first += tile_count<LIST>((nr + 2 * BM - 1) / (2 * BM), (nc + PBN - 1) / PBN);
    }
    s_first[bt.B] = first;
  }
  __syncthreads();
  const int total = s_first[bt.B];
  const int P = gridDim.x >> 1, pr = blockIdx.x >> 1;
  const int nslab = bt.d_k / BK;
  // item -> image b (items only grow, so b only moves forward), tile (I, J), rows and columns of the image
  auto locate = [&](int item, int &b, int &I, int &J, int &nrows, int &ncols) {
    while (item >= s_first[b + 1]) ++b;
    nrows = s_rows[b];
    ncols = s_cols[b];
    tile_at<LIST>(item - s_first[b], (nrows + 2 * BM - 1) / (2 * BM), (ncols + PBN - 1) / PBN, I, J);
  };
  // columns the MMA has to produce: the rows x centres pass stops at the last centre, in steps of 32
  auto width = [&](int J, int ncols) {
    if (MODE != MODE_ASSIGN) return PBN;
    const int left = ncols - J * PBN;
    return left >= PBN ? PBN : ((left + 31) & ~31);
  };

  if (pr >= total) {
  } else if (warp == 0) {
    // ---------------- TMA producer (each CTA for its own shared memory) ----------------
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      int b = 0;
      for (int item = pr; ok && item < total; item += P) {
        int I, J, nrows, ncols;
        locate(item, b, I, J, nrows, ncols);
        const CUtensorMap *ma = &tm.a[b], *mb = &tm.b[b];
        const int bw = width(J, ncols);
        for (int ks = 0; ks < nslab; ks += SLABS, ++it) {
          const int s = it % PSTAGES;
          const int n = min(SLABS, nslab - ks);      // K-slabs of this stage
          if (!mbar_wait(&sh.empty[s], ((it / PSTAGES) & 1) ^ 1)) { ok = false; break; }
          uint8_t *a_dst = ring + (size_t)s * PSTAGE_BYTES, *b_dst = a_dst + SLABS * A_BYTES;
          if (leader) mbar_arrive_expect_tx(&sh.full[s], (uint32_t)n * 4u * A_BYTES);   // the bytes of both CTAs
          const uint32_t bar = map_to_rank(smem_u32(&sh.full[s]), 0);
          for (int h = 0; h < n; ++h) {
            tma_load_2d_pair(a_dst + h * A_BYTES, ma, bar, (ks + h) * BK, (2 * I + (int)rank) * BM);
            tma_load_2d_pair(b_dst + h * A_BYTES, mb, bar, (ks + h) * BK, J * PBN + (int)rank * (bw >> 1));
          }
        }
      }
      if (!ok) atomicExch(&sh.abort, 1);
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (CTA 0 for both) ----------------
    if (lane == 0 && leader) {
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      int b = 0;
      for (int item = pr; ok && item < total; item += P) {
        int I, J, nrows, ncols;
        locate(item, b, I, J, nrows, ncols);
        const uint32_t a = tcount % PNACC;
        if (!mbar_wait(&sh.acc_empty[a], ((tcount / PNACC) & 1) ^ 1)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + a * PBN;
        // kind::f16, fp32 accumulate, bf16 x bf16, both operands K-major, M = 256 over the pair, N = this tile's width
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(width(J, ncols) >> 3) << 17) | ((uint32_t)((2 * BM) >> 4) << 24);
        for (int ks = 0; ks < nslab; ks += SLABS, ++it) {
          const int s = it % PSTAGES;
          const int n = min(SLABS, nslab - ks);
          if (!mbar_wait(&sh.full[s], (it / PSTAGES) & 1)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(ring + (size_t)s * PSTAGE_BYTES), b_addr = a_addr + SLABS * A_BYTES;
#pragma unroll
          for (int h = 0; h < SLABS; ++h) {
            if (h < n) {
#pragma unroll
              for (int k = 0; k < BK / 16; ++k)
                umma_bf16_pair(d_tmem, smem_desc(a_addr + h * A_BYTES + k * 32), smem_desc(b_addr + h * A_BYTES + k * 32), idesc,
                               (ks | h | k) != 0);
            }
          }
          umma_commit_pair(&sh.empty[s]);          // frees the stage in both CTAs once these MMAs have read it
        }
        if (ok) umma_commit_pair(&sh.acc_full[a]); // accumulator complete, in both CTAs
        ++tcount;
      }
      umma_commit_pair(&sh.done);                  // both CTAs learn that no MMA is running any more
      if (!ok) atomicExch(&sh.abort, 1);
    }
    // whatever way the loop ended, no MMA may still be running when the tensor memory is given back
    if (lane == 0 && !mbar_wait(&sh.done, 0)) atomicExch(&sh.abort, 1);
  } else {
    // ---------------- epilogue (each CTA for its 128 rows) ----------------
    const int ew = warp - 2;
    const int qd = warp & 3;                        // tensor-memory lane quadrant this warp may read
    const int half = ew >> 2;                       // which part of the tile's columns
    float *rn_col = sh.rn_col[ew];
    uint32_t *tr = reinterpret_cast<uint32_t *>(ring + PRING - 1024) + ew * (32 * 36);   // all-pairs pass only
    uint32_t tcount = 0;
    bool ok = true;
    float mx = 0.f;                                 // largest distance of the current image (layer)
    int b = 0, b_mx = 0;
    unsigned long long unused_seen = 0ull;
    auto flush_mx = [&](int bb) {
      const unsigned w = __reduce_max_sync(0xffffffffu, __float_as_uint(mx));
      if (lane == 0 && w) atomicMax(reinterpret_cast<unsigned *>(&bt.img[bb].cnt[kCntSpread]), w);
      mx = 0.f;
    };
    for (int item = pr; ok && item < total; item += P) {
      int I, J, nrows, ncols;
      locate(item, b, I, J, nrows, ncols);
      if (MODE == MODE_SPREAD && b != b_mx) { flush_mx(b_mx); b_mx = b; }
      const ImgDesc &im = bt.img[b];
      const uint32_t a = tcount % PNACC;
      const int R = 2 * I + (int)rank;              // this CTA's 128-row block
      const int cbase = J * PBN + half * PC::COLS;  // this warp's columns
      const bool skip = MODE != MODE_ASSIGN && cbase / BM < R;   // below the diagonal
      const uint32_t taddr = tmem_base + a * PBN + half * PC::COLS + ((uint32_t)(qd * 32) << 16);
      const uint32_t rel = map_to_rank(smem_u32(&sh.acc_empty[a]), 0);
      int band = 0;
      ok = epi_tile<MODE, PC::COLS>(im, kept_rows, R, cbase, skip, nrows, ncols, taddr, &sh.acc_full[a], (tcount / PNACC) & 1,
                                    rn_col, tr, lane, qd, band, mx, [&]() { mbar_arrive_remote(rel); }, unused_seen);
      if (MODE == MODE_GRAM && band) atomicAdd(&im.cnt[PACT_CNT_BAND_DC], band);
      if (!ok) break;
      ++tcount;
    }
    if (!ok) atomicExch(&sh.abort, 1);
    if (MODE == MODE_SPREAD) flush_mx(b_mx);
  }

  tc_fence_before();
  __syncthreads();
  cluster_barrier();                                  // nothing is in flight towards the other CTA any more
  tc_fence_after();
  if (warp == 1) tmem_dealloc2(tmem_base, TMEM_COLS);
  if (threadIdx.x == 0 && sh.abort)
    for (int b = 0; b < bt.B; ++b) atomicMin(&bt.img[b].cnt[PACT_CNT_STATUS], (int)PACT_ERR_TIMEOUT);
}

// ---- host side -----------------------------------------------------------------------------------

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn g_encode = nullptr;

bool encode_rows(CUtensorMap *map, const void *base, long long rows, long long ld_elems, int d_k) {
  const cuuint64_t dims[2] = {(cuuint64_t)d_k, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ld_elems * 2};
  const cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)BM};
  const cuuint32_t estr[2] = {1, 1};
  return g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kGramBN = 128, kWideBN = 256;

}  // namespace

bool umma_supported(int d_k) { return g_encode != nullptr && d_k % BK == 0; }

namespace {
bool g_pair_ok = false;                               // clusters of two CTAs of the pair kernel can be launched
bool g_pair_gram_ok = false;                          // ... of its all-pairs form with 16 epilogue warps
bool g_pair_assign_ok = false;                        // ... of its rows x centres form

template <int MODE, int EW>
cudaError_t launch_pair(const Batch &bt, const TmapSet &tm, long long tiles, int kept_rows, const ClusterCfg &cfg, bool pdl,
                        cudaStream_t st) {
  using PC = PairCfg<MODE, EW>;
  long long P = cfg.sm_count / 2;                     // one pair per two SMs
  if (P > tiles * bt.B) P = tiles * bt.B;
  if (P < 1) P = 1;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3((unsigned)(2 * P));
  lc.blockDim = dim3(PC::THREADS);
  lc.dynamicSmemBytes = PC::SMEM;
  lc.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr;
  lc.numAttrs = pdl ? 2 : 1;
  return cudaLaunchKernelEx(&lc, k_tiles_pair<MODE, EW>, bt, tm, kept_rows);
}

// can clusters of two CTAs of this kernel be launched at all?
template <int MODE, int EW> cudaError_t pair_configure(bool &ok) {
  using PC = PairCfg<MODE, EW>;
  ok = false;
  cudaError_t e = cudaFuncSetAttribute(k_tiles_pair<MODE, EW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)PC::SMEM);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(2);
  lc.blockDim = dim3(PC::THREADS);
  lc.dynamicSmemBytes = PC::SMEM;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  lc.attrs = attr;
  lc.numAttrs = 1;
  int n = 0;
  e = cudaOccupancyMaxActiveClusters(&n, k_tiles_pair<MODE, EW>, &lc);
  if (e != cudaSuccess || n < 1) (void)cudaGetLastError();
  else ok = true;
  return cudaSuccess;
}
}  // namespace

cudaError_t umma_configure() {
  void *fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess) return e;
  if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
  g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  e = cudaFuncSetAttribute(k_tiles_umma<MODE_GRAM, kGramBN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)TileCfg<kGramBN>::SMEM);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(k_tiles_umma<MODE_SPREAD, kWideBN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)TileCfg<kWideBN>::SMEM);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(k_tiles_umma<MODE_ASSIGN, kWideBN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)TileCfg<kWideBN>::SMEM);
  if (e != cudaSuccess) return e;
  e = pair_configure<MODE_ASSIGN, 8>(g_pair_assign_ok);
  if (e != cudaSuccess) return e;
  e = pair_configure<MODE_GRAM, 16>(g_pair_gram_ok);
  if (e != cudaSuccess) return e;
  return pair_configure<MODE_SPREAD, 8>(g_pair_ok);
}

static int umma_grid_x(long long tiles, int B, int sms) {
  long long x = sms / B;                            // one CTA per SM: all CTAs of the batch run at once
  if (x < 1) x = 1;
  if (x > tiles) x = tiles;
  return (int)(x < 1 ? 1 : x);
}

cudaError_t launch_gram_umma(const Batch &bt, int maxN, const ClusterCfg &cfg, cudaStream_t st, int est_rows) {
  TmapSet tm;
  for (int b = 0; b < bt.B; ++b) {
    const ImgDesc &im = bt.img[b];
    if (!encode_rows(&tm.a[b], im.Kp, im.Np, bt.d_k, bt.d_k)) return cudaErrorInvalidValue;
    tm.b[b] = tm.a[b];
  }
  // With many blocks per SM (batches, long images) pairs of CTAs on 256 x 256 tiles with 16 epilogue warps each are
  // faster: half the operand bytes per pair of blocks and a shorter epilogue.  With few (three per SM on one
  // 7290-token image) the coarser tiles cost a round, and single CTAs on 128 x 128 blocks are.
  if (est_rows < 1 || est_rows > maxN) est_rows = maxN;
  const long long nq = (est_rows + BM - 1) / BM;
  if (g_pair_gram_ok && nq * (nq + 1) / 2 * bt.B >= 6LL * cfg.sm_count) {
    const long long n2 = (maxN + 2 * BM - 1) / (2 * BM);
    return launch_pair<MODE_GRAM, 16>(bt, tm, n2 * (n2 + 1) / 2, 0, cfg, true, st);
  }
  const long long nb = (maxN + BM - 1) / BM;
  dim3 grid(umma_grid_x(nb * (nb + 1) / 2, bt.B, cfg.sm_count), bt.B);
  return launch_k(k_tiles_umma<MODE_GRAM, kGramBN>, grid, dim3(THREADS), TileCfg<kGramBN>::SMEM, st, true, bt, tm, 0);
}

bool umma_pairs_for_assign(int maxN, int B, const ClusterCfg &cfg) {
  // with two or more 128-row blocks per SM (batches, long images) pairs of CTAs on 256 x 256 tiles are faster:
  // the pass is bound by operand bytes from the L2, and a pair fetches two thirds of them
  return g_pair_assign_ok && (long long)((maxN + BM - 1) / BM) * B >= 2LL * cfg.sm_count;
}

// labels: the single-CTA kernel also forms labels and member counts (all-token rows only); pairs: the pair kernel
// (all-token rows, no labels)
cudaError_t launch_assign_umma(const Batch &bt, int maxN, bool kept_rows, const ClusterCfg &cfg, cudaStream_t st, bool labels,
                               bool pairs) {
  TmapSet tm;
  for (int b = 0; b < bt.B; ++b) {
    const ImgDesc &im = bt.img[b];
    if (kept_rows) {
      if (!encode_rows(&tm.a[b], im.Kp, im.Np, bt.d_k, bt.d_k)) return cudaErrorInvalidValue;
    } else if (!encode_rows(&tm.a[b], im.Kc, im.N, im.ldKc, bt.d_k)) return cudaErrorInvalidValue;
    if (!encode_rows(&tm.b[b], im.Kcen, im.Np, bt.d_k, bt.d_k)) return cudaErrorInvalidValue;
  }
  if (pairs && !kept_rows && g_pair_assign_ok) {
    const long long pt = (long long)((maxN + 2 * BM - 1) / (2 * BM)) * ((maxN + PBN - 1) / PBN);
    return launch_pair<MODE_ASSIGN, 8>(bt, tm, pt, 0, cfg, true, st);
  }
  const long long tiles = (long long)((maxN + BM - 1) / BM) * ((maxN + kWideBN - 1) / kWideBN);
  dim3 grid(umma_grid_x(tiles, bt.B, cfg.sm_count), bt.B);
  return launch_k(k_tiles_umma<MODE_ASSIGN, kWideBN>, grid, dim3(THREADS), TileCfg<kWideBN>::SMEM, st, true, bt, tm, (kept_rows ? 1 : 0) | (labels && !kept_rows ? 2 : 0));
}

// every layer of the batch is one "image": rows and columns are all N keys of K_clu
cudaError_t launch_spread_umma(const Batch &bt, int maxN, const ClusterCfg &cfg, cudaStream_t st) {
  TmapSet tm;
  for (int b = 0; b < bt.B; ++b) {
    const ImgDesc &im = bt.img[b];
    if (!encode_rows(&tm.a[b], im.Kc, im.N, im.ldKc, bt.d_k)) return cudaErrorInvalidValue;
    tm.b[b] = tm.a[b];
  }
  if (g_pair_ok) {
    const long long ptiles = (long long)((maxN + 2 * BM - 1) / (2 * BM)) * ((maxN + PBN - 1) / PBN);
    return launch_pair<MODE_SPREAD, 8>(bt, tm, ptiles, 0, cfg, false, st);
  }
  const long long tiles = (long long)((maxN + BM - 1) / BM) * ((maxN + kWideBN - 1) / kWideBN);
  dim3 grid(umma_grid_x(tiles, bt.B, cfg.sm_count), bt.B);
  return launch_k(k_tiles_umma<MODE_SPREAD, kWideBN>, grid, dim3(THREADS), TileCfg<kWideBN>::SMEM, st, false, bt, tm, 0);
}

}  // namespace pact
