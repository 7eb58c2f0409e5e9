// Internal declarations shared by the translation units of libks (not part of the ABI).
#pragma once

#include <cuda_runtime.h>

#include <cstddef>
#include <cstdint>

#include "ks.h"

namespace ks {

// Top-level nodes of the quantised trees as kernel-parameter constants (constant bank):
// x = row offset in the byte tile, y = (threshold index + 1) replicated into the four bytes.
constexpr int kFastTopPairs = 3584;
struct FastTopParams {
  uint2 w[kFastTopPairs];
};

// Constants of the tensor-core MLP path that travel as a kernel parameter (constant bank):
// folded standardisation per K position, biases, the last layer's weights widened to fp32.
struct alignas(16) MlpTcParams {
  float scale[64], shift[64];
  float b1[256], b2[256], w3[256];
  float b3;
  // one-hot input form: the problem-only inputs (11 columns + 7 level indicators) are folded
  // into a per-CTA bias, the 7 candidate-side level indicators are formed from the record
  int onehot;
  uint16_t ind0[8], ind1[8];           // bf16 of an indicator's standardised value when 0 / 1 (kernel sched 0..3, epilogue sched 0..2)
  float p_scale[18], p_shift[18];      // standardisation of the folded inputs
  const float* w1_prob;                // device, [18][256]: first-layer weights of the folded inputs
  int wait_limit;                      // tries a barrier wait may take (set at every launch)
  int starve;                          // test hook: the weight image is never copied, so the first wait runs out
};

// Linear scorer (one weight layer) in a form the fused ridge kernel consumes: per feature column
// the weight and the standardisation, per expanded categorical field (one-hot input form) the
// contribution of every level, and the bias. Passed by value at every launch.
struct RidgeParams {
  float w[64], mu[64], sigma[64];  // by feature column; w = 0 for a column that is expanded
  float lut5[4], lut9[4], lut17[4], lut18[4];  // one-hot form: contribution of each level (else 0)
  float bias;
};

// Generic device form of a tree node: 8 bytes, children tree-relative.
struct DevNode {
  float v;        // threshold, or the leaf value
  uint16_t feat;  // 0xFFFF = leaf
  uint16_t left;  // left child (right = left + 1)
};

// Rows and thresholds of one feature column in the quantised form: its sorted distinct
// thresholds are thr[thr0 .. thr0 + nthr), cut into nslice rows of at most 127, followed by
// nrank rank rows (categorical columns with partition splits; rank[r][level] = rank of the level
// in the row's ordering).
struct FeatQ {
  uint32_t thr0;
  uint16_t nthr, row0, nslice, nrank;
  uint8_t rank[3][4];
};

// Probe budget of the quantised kernel's chunk waits (0: the default) and the test hook that
// starves a wait (the barrier is armed for more bytes than its copy brings).
struct FastWait {
  int limit;
  int starve;
};

struct GbdtModel {
  int n_trees = 0;
  int max_depth = 0;
  int64_t n_nodes = 0;
  float base = 0.0f;
  DevNode* d_nodes = nullptr;  // all trees back to back
  int* d_roots = nullptr;      // [n_trees + 1] offsets into d_nodes
  // quantised fast form (complete trees, chunked level-order layout), see ks_gbdt_fast.cu
  bool fast = false;
  int fast_depth = 0;          // every tree padded to this depth
  int fast_threads = 0;        // tile geometry: threads per CTA (512 or 1,024) ...
  int block_cands = 0;         // ... and candidates per CTA = bytes per tile row (1,024 or 512)
  int buf_bytes = 0;           // size of one of the two chunk buffers in shared memory
  int ctas_per_sm = 1;         // CTAs of this geometry that share an SM
  int n_qrows = 0;             // quantised feature rows (127-threshold slices and rank rows)
  int n_qthr = 0, thr_cand0 = 0, thr_prob0 = 0;  // thresholds in all; first of the candidate-only / problem-only features
  int n_pair_rows = 0, n_cand_rows = 0, n_prob_rows = 0;  // rows by what their feature depends on
  int top_levels = 0;          // levels whose nodes also live in h_top
  bool top_compact = false;    // h_top holds one 32-bit word per node instead of a pair
  FastTopParams* h_top = nullptr;  // host copy, passed by value at every launch
  int tpc = 0;                 // trees per chunk
  int n_chunks = 0;
  int chunk_bytes = 0;
  uint32_t* d_qnodes = nullptr;  // [n_chunks][chunk_bytes / 4]
  float* d_qthr = nullptr;       // [n_qthr] sorted thresholds, feature after feature
  FeatQ* d_qfeat = nullptr;      // [64] rows and thresholds of each feature column
};

struct MlpModel {
  int n_layers = 0;
  int widths[KS_MLP_MAX_LAYERS + 1] = {0};
  int max_width = 0;
  uint16_t* d_w[KS_MLP_MAX_LAYERS] = {nullptr};  // bf16 [out, in] row-major
  float* d_b[KS_MLP_MAX_LAYERS] = {nullptr};
  float* d_mu = nullptr;
  float* d_sigma = nullptr;
  // one weight layer (the linear ridge scorer): fused kernel without a feature tile
  RidgeParams* h_ridge = nullptr;
  // tensor-core path (shape 64-256-256-1 only), see ks_mlp_tc.cu
  bool tc = false;
  uint16_t* d_tc_image = nullptr;      // W1 and W2 in the shared-memory operand layout
  float* d_w1_prob = nullptr;          // one-hot form: first-layer weights of the folded inputs
  MlpTcParams* h_tc_params = nullptr;  // host copy, passed by value at every launch
};

// kernel-side view of an MLP (passed by value)
struct MlpView {
  int n_layers;
  int widths[KS_MLP_MAX_LAYERS + 1];
  const uint16_t* w[KS_MLP_MAX_LAYERS];
  const float* b[KS_MLP_MAX_LAYERS];
  const float* mu;
  const float* sigma;
};

}  // namespace ks

struct ks_ctx {
  int device = 0;
  ks_gpu_desc desc{};
  void* ws = nullptr;  // device workspace (partial top-k lists, staging)
  size_t ws_bytes = 0;
  void* pinned = nullptr;  // host staging for ks_select_one results
  size_t pinned_bytes = 0;
  int* d_counters = nullptr;  // [kMaxSliceBlocks + 1] arrival counters of the slice mode, zero between calls
  int32_t* d_pinned_idx = nullptr;  // device aliases of `pinned` (mapped host memory)
  float* d_pinned_score = nullptr;
  int* h_status = nullptr;  // status word (mapped pinned host memory) set by kernels whose
  int* d_status = nullptr;  // bounded waits give up; d_status is its device alias
  int64_t launches = 0;
  int select_one_seq = 0;  // sequence number of the last single-problem call
  ks::FastWait wait{0, 0};  // probe budget of bounded device waits (0: default) and the starve hook (tests)
  char err[256] = {0};
  // optional timing of the dominant kernel of the last ks_select* call (ks_profile_enable)
  bool profile = false;
  bool profile_valid = false;
  cudaEvent_t ev_begin = nullptr, ev_end = nullptr;
};

// A candidate catalogue prepared for single-problem calls with one model (ks_catalogue_prepare).
struct ks_catalogue {
  ks_ctx* ctx = nullptr;
  const ks_model* model = nullptr;
  const ks_candidate* d_c = nullptr;
  int C = 0;
  int device = 0;
  bool prepared = false;   // false: calls go through ks_select_one
  int nblk = 0, slices = 1, max_k = KS_MAX_K;
  void* d_mem = nullptr;   // one block: rows | memo | partial lists | partial-score planes | similarity order
  size_t off_memo = 0, off_part = 0, off_scores = 0, off_order = 0;
};

struct ks_model {
  ks_ctx* ctx = nullptr;
  int device = 0;  // the context's device (kept here: the model may outlive the context)
  int kind = 0;  // 0 tree ensemble, 1 MLP, 2 static sampling score
  ks::GbdtModel gbdt;
  ks::MlpModel mlp;
};

namespace ks {

constexpr int kBlock = 256;            // threads per block of the pair kernels
constexpr int kSubTilesMax = 8;        // sub-tiles of kBlock rows one block ranks
constexpr int kFastMaxDepth = 10;
constexpr int kFastMaxProbRows = 256;  // rows of problem-only features
constexpr int kFastMaxCandRec = 256;   // rows of candidate-only features (bytes of a per-call record)
constexpr int kFastMaxPairRec = 256;   // rows of per-pair features a memoised model may have
constexpr size_t kMemoTableBytes = size_t(256) << 20;  // per-(problem, class) records held at a time
constexpr int kFastWaitLimit = 1 << 17;  // probes of a chunk wait (a sleep ends early, ~0.2 us measured): tens of ms
constexpr int kMlpThreads = 512;        // threads per block of the tensor-core MLP kernel
constexpr int kMaxSliceBlocks = 1024;  // candidate blocks the slice mode supports

// Levels of the categorical field held by feature column `col` (0: not a level-code column):
// layout flags, operand type, bias flag, activation, kernel / epilogue schedule, tile scheduler.
inline int categorical_levels(int col) {
  switch (col) {
    case 3: case 4: case 8: case 19: return 2;
    case 9: case 18: return 3;
    case 5: case 17: return 4;
    default: return 0;
  }
}

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) costs a driver call; remembers, per kernel and
// device, the largest size already granted (ks_api.cu).
cudaError_t ensure_dynamic_smem(const void* kernel, size_t bytes);
// A descriptor every entry point accepts: no zero capacity or rate, reserved word zero.
bool valid_desc(const ks_gpu_desc& d);

// Builds the quantised fast form of a validated ensemble when it qualifies (m.fast).
cudaError_t build_fast_gbdt(GbdtModel& m, int n_trees, const int64_t* h_tree_offsets,
                            const ks_node_host* h_nodes);

// Slice mode of the quantised tree kernel (single-problem latency call).
struct FastSlice {
  int n_slices;
  long long pairs;   // rows of one partial-score plane
  float* scores;     // [n_slices][pairs]
  int* counters;     // [blocks + 1], zero between calls
  int32_t* out_idx;  // single-problem form: [k], device-visible; else null (a merge kernel follows)
  float* out_score;
  uint8_t* tiles;    // single-problem form: scratch for the prepared tiles [blocks][rows][block_cands], or null
  int* out_seq;      // single-problem form: device-visible word that receives `seq` after the results
  int seq;
};

// What a prepared catalogue hands to the quantised tree kernel instead of per-call work.
struct FastPrepared {
  const uint8_t* cand_rows;  // [16 type combinations][C][record] candidate-only rows
  void* memo_mem;            // class tables and ids of every combination + one problem's record table, or null
};

// Similarity order of a catalogue (ks_order.cu): positions sorted so that neighbours differ in as
// few knobs as possible; written to the front of `scratch` as C int32.
constexpr int kOrderMinProblems = 16;  // batches of at least this many problems are ranked in similarity order
size_t order_scratch_bytes(int C);
cudaError_t launch_catalogue_order(const ks_candidate* d_c, int C, void* scratch, cudaStream_t stream,
                                   int64_t* launches);

// Search-space enumeration and validity filtering (ks_catalogue.cu).
cudaError_t launch_enumerate(long long first, long long count, ks_candidate* d_out, cudaStream_t stream,
                             int64_t* launches);
size_t valid_catalogue_scratch_bytes(int C);
cudaError_t launch_valid_catalogue(const ks_gpu_desc& desc, const ks_problem& p, unsigned flags,
                                   const ks_candidate* d_c, int C, void* d_scratch, ks_candidate* d_out,
                                   int32_t* d_out_index, int32_t* d_count, cudaStream_t stream,
                                   int64_t* launches);
cudaError_t launch_remap_indices(int32_t* d_idx, long long n, const int32_t* d_map, int map_len,
                                 cudaStream_t stream, int64_t* launches);

// Quantised tree path: blocks per problem for `per_problem` rows, and the launch itself.
void fast_tiling(const GbdtModel& g, int P, int64_t per_problem, int* nblk, int* rows_per_cta);
size_t fast_scratch_bytes(const GbdtModel& g, int C);  // per-call table of candidate-only rows
size_t fast_memo_bytes(const GbdtModel& g, int P, int C);  // memo of the per-pair rows (0: not used)
void free_fast_gbdt(GbdtModel& m);
cudaError_t launch_select_fast(const ks_gpu_desc& desc, const GbdtModel& g, const ks_problem* d_p,
                               const ks_problem* p_by_value, int P, const ks_candidate* d_c, int C,
                               int nblk, int rows_per_cta, const int64_t* seg_off, const int32_t* seg_idx,
                               int k, unsigned long long* partial, void* scratch, int* status,
                               cudaStream_t stream, int64_t* launches, cudaEvent_t ev_begin,
                               const FastSlice* slice = nullptr, void* memo_mem = nullptr,
                               const FastWait* wait = nullptr, const FastPrepared* prep = nullptr,
                               const int32_t* perm = nullptr);
// Prepared catalogue (single-problem calls against a fixed catalogue and model).
size_t fast_prepared_rows_bytes(const GbdtModel& g, int C);
size_t fast_prepared_memo_bytes(const GbdtModel& g, int C);  // 0: the model's per-pair rows do not fit a record
cudaError_t fast_prepare(const ks_gpu_desc& desc, const GbdtModel& g, const ks_candidate* d_c, int C, void* d_rows,
                         void* memo_mem, cudaStream_t stream, int64_t* launches);
int fast_slices(const GbdtModel& g, int64_t blocks);
// ks_score with a qualifying ensemble: tiles quantised from the feature rows, then the same walk.
size_t score_fast_scratch_bytes(const GbdtModel& g, int64_t rows);
cudaError_t launch_score_fast(const ks_gpu_desc& desc, const GbdtModel& g, const float* d_feat, int64_t rows,
                              float* d_scores, void* scratch, int* status, cudaStream_t stream,
                              int64_t* launches, const FastWait* wait = nullptr, int floor_repeat = 0);
// checked build (KS_DEBUG_BOUNDS): source line of the first index found out of range (0: none;
// -1: not a checked build), and its reset
int fast_bounds_line();
void fast_bounds_clear();

// Tensor-core MLP path.
cudaError_t build_fast_mlp(MlpModel& m, const uint16_t* const* h_w, const float* const* h_b, const float* h_mu,
                           const float* h_sigma);
void free_fast_mlp(MlpModel& m);
// Linear scorer: fills m.h_ridge when the model has one weight layer.
cudaError_t build_ridge(MlpModel& m, const uint16_t* h_w, const float* h_b, const float* h_mu,
                        const float* h_sigma);
void free_ridge(MlpModel& m);
size_t ridge_scratch_bytes(int C);
int mlp_tc_blocks_per_problem(int P, int64_t per_problem);
size_t mlp_tc_scratch_bytes(int C);
// ks_score on the tensor-core kernel (ordinal input form only): the given rows are the input.
bool score_mlp_tc_ok(const MlpModel& m);
cudaError_t launch_score_mlp_tc(const ks_gpu_desc& desc, const MlpModel& m, const float* d_feat, int64_t rows,
                                float* d_scores, int* status, cudaStream_t stream, int64_t* launches,
                                const FastWait* wait = nullptr);
constexpr int kMlpWaitLimit = 1 << 14;  // tries of a barrier wait of the tensor-core kernel (each blocks for up to a few microseconds): tens of ms
cudaError_t launch_select_mlp_tc(const ks_gpu_desc& desc, const MlpModel& m, const ks_problem* d_p,
                                 const ks_problem* p_by_value, int P, const ks_candidate* d_c, int C, int nblk,
                                 const int64_t* seg_off, const int32_t* seg_idx, int k,
                                 unsigned long long* partial, void* scratch, int* status, cudaStream_t stream,
                                 int64_t* launches, cudaEvent_t ev_begin, const FastWait* wait = nullptr);

// k-way merge of gathered partial lists (multi-GPU candidate split).
cudaError_t launch_merge_lists(const int32_t* d_idx, const float* d_score, int P, int n, int k, int32_t* d_out_idx,
                               float* d_out_score, cudaStream_t stream, int64_t* launches);

// ---- launchers (each enqueues on `stream`, returns the cudaError of the launch) -----------
cudaError_t launch_featurize(const ks_gpu_desc& desc, const ks_problem* d_p, int P,
                             const ks_candidate* d_c, int C, const int64_t* d_seg_off,
                             const int32_t* d_seg_idx, int64_t pairs, float* d_out, void* scratch,
                             cudaStream_t stream, int64_t* launches);
size_t featurize_scratch_bytes(int P);  // table of problem terms for the dense form

cudaError_t launch_score_gbdt(const GbdtModel& m, const float* d_feat, int64_t rows, float* d_scores,
                              uint16_t* d_leaf_idx, cudaStream_t stream, int64_t* launches);

cudaError_t launch_score_mlp(const MlpModel& m, const float* d_feat, int64_t rows, float* d_scores,
                             cudaStream_t stream, int64_t* launches);

// Fused featurize + score + top-k. `p_by_value` non-null selects the single-problem form.
// d_partial: workspace for the per-block partial lists and per-call tables, at least
// select_partial_bytes().
size_t select_partial_bytes(const ks_model& model, int P, int C, int64_t pairs, bool segmented, int k);
cudaError_t launch_select(const ks_gpu_desc& desc, const ks_model& model, const ks_problem* d_p,
                          const ks_problem* p_by_value, int P, const ks_candidate* d_c, int C,
                          const int64_t* d_seg_off, const int32_t* d_seg_idx, int64_t pairs, int k,
                          void* d_partial, int32_t* d_topk_idx, float* d_topk_score,
                          cudaStream_t stream, int64_t* launches, int* d_status,
                          cudaEvent_t ev_begin = nullptr, cudaEvent_t ev_end = nullptr, int* d_counters = nullptr,
                          const FastWait* wait = nullptr);

}  // namespace ks
