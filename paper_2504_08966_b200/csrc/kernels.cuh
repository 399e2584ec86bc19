// Launchers of the PACT kernels (host side); one translation unit per stage group.
#pragma once
#include "common.cuh"

namespace pact {

// Launches a kernel; pdl: with the programmatic-serialization attribute (it may start before its predecessor in
// the stream has finished and must call pdl_wait() before it reads what the predecessor wrote).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl,
                            Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

constexpr int kMergeMaxD = 256 * 4 * 8;   // widest hidden state the merge kernel holds in registers

// how a kernel finds its rows
enum RowMode { ROWS_ALL = 0, ROWS_KEPT_LIST = 1, ROWS_PRUNED_LIST = 2 };

// euti.cu
constexpr int kQPartRows = 32;            // most row blocks the column sums of Q are split into
constexpr int kHistBits = 12;             // key bits of the first-level histogram of the threshold selection
constexpr int kHistShift = 32 - kHistBits; // a key's bin in that histogram is key >> kHistShift
// Cooperative launch (every CTA resident at once), optionally with the programmatic-serialization attribute too.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_coop(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl,
                               Args &&...args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Algorithm 1.  mode 0: scores, threshold, lists, survivor keys (four kernels; the first also clears what later
// kernels accumulate into); mode 1: scores only (three kernels).
// mark (optional) is called between the kernels of the group (the per-kernel timing of a profiled call)
typedef cudaError_t (*StageMark)(void *);
cudaError_t launch_euti(const Batch &bt, int maxN, bool bf16, int mode, cudaStream_t st, StageMark mark = nullptr,
                        void *mark_arg = nullptr);
int euti_kernels(int mode);
// threshold + ordered compaction; gather: also copy the survivor keys and clear the accumulators
void launch_select_gather(const Batch &bt, int maxN, bool bf16, bool gather, cudaStream_t st);
cudaError_t euti_configure(int n_qcols, int n_qh);
cudaError_t select_configure();            // what launch_select_gather needs, once per device

// cluster.cu
struct ClusterCfg {
  int sm_count;
  int centers_smem_max; // most dynamic shared memory the centre-selection kernel may ask for
};
cudaError_t cluster_configure(ClusterCfg *cfg);
// gathers survivor keys and inverse norms; all_tokens: also every token's inverse norm
void launch_keynorm_gather(const Batch &bt, int maxN, bool bf16, bool all_tokens, cudaStream_t st);
void launch_center_key_gather(const Batch &bt, int maxN, bool bf16, cudaStream_t st);
void launch_gram(const Batch &bt, int maxN, bool bf16, const ClusterCfg &cfg, cudaStream_t st);
// density order, centre selection, cluster ids and centre keys in one cooperative kernel
// maxQ: estimate of the largest number of survivors of an image (sizes the staging buffer only)
cudaError_t launch_centers(const Batch &bt, int maxQ, bool bf16, const ClusterCfg &cfg, int spin_limit, cudaStream_t st);
void launch_assign(const Batch &bt, int maxN, bool bf16, RowMode mode, const ClusterCfg &cfg, cudaStream_t st);
void launch_label(const Batch &bt, int maxN, bool bf16, RowMode mode, cudaStream_t st);
// layer choice: inverse norms of all keys of every layer, largest pair distance (any dtype), result
void launch_key_rnorm(const Batch &bt, int maxN, bool bf16, cudaStream_t st);
void launch_spread(const Batch &bt, int maxN, bool bf16, const ClusterCfg &cfg, cudaStream_t st);
void launch_spread_finish(const Batch &bt, float *max_dist, int32_t *layer_out, int layer_base, float threshold,
                          cudaStream_t st);

// gram_umma.cu: tcgen05 versions of the two tile passes for bf16 keys whose width is a multiple of 64
cudaError_t umma_configure();
bool umma_supported(int d_k);
// est_rows: an upper estimate of the survivors per image when the host has one (0: maxN)
cudaError_t launch_gram_umma(const Batch &bt, int maxN, const ClusterCfg &cfg, cudaStream_t st, int est_rows = 0);
cudaError_t launch_assign_umma(const Batch &bt, int maxN, bool kept_rows, const ClusterCfg &cfg, cudaStream_t st, bool labels = false,
                               bool pairs = false);
bool umma_pairs_for_assign(int maxN, int B, const ClusterCfg &cfg);
cudaError_t launch_members(const Batch &bt, int maxN, cudaStream_t st);
cudaError_t launch_spread_umma(const Batch &bt, int maxN, const ClusterCfg &cfg, cudaStream_t st);

// merge.cu
// member records in cluster order from label[] (from_best: labels are first formed from the nearest-centre
// pass, all tokens); csize, cticket and cnt_cb must be zero.  spin_limit bounds the wait of its barrier.
cudaError_t launch_lists(const Batch &bt, int maxN, bool bf16, bool from_best, int spin_limit, cudaStream_t st);
int lists_kernels(int maxN, int B);        // kernels launch_lists launches (1, or 2 when the grid cannot be resident at once)
cudaError_t launch_merge(const Batch &bt, bool in_bf16, bool out_bf16, const ClusterCfg &cfg, cudaStream_t st);
cudaError_t merge_configure();
int merge_ctas(int sm_count, int B);       // CTAs per image of k_merge (sizes its scratch)

}  // namespace pact
