/*
 * ks.h -- C ABI of libks: execution-free CUTLASS kernel selection on one sm_100a GPU.
 *
 * The library evaluates, for every (GEMM problem p, candidate configuration c) pair, the
 * statically computable hardware-aware feature map x = phi(p, c, h) of the paper's section
 * "From CUTLASS Candidates to Hardware-Aware Features" (Table "Feature groups" and the
 * sub-sections Structural Core, Work Decomposition and Wave Quantization, Memory Behavior,
 * Resource Pressure and Occupancy, Pipeline Balance), scores x with a learned ranker
 * f_theta (section "Learning to Rank Candidates": Model A, an additive tree ensemble, or
 * Model B, a feed-forward ranker) and returns, per problem, the k best candidates -- the
 * decision rule c^(p) = argmax_{c in C(p)} f_theta(x(p, c, h)) (Eq. "selection"), widened
 * from the single argmax to a top-k shortlist.
 *
 * Conventions
 *   - Every call returns a ks_status (KS_OK == 0). Nothing aborts, throws or prints.
 *   - Pointers named d_* are DEVICE pointers on the context's CUDA device, h_* are HOST
 *     pointers; the caller owns every data buffer, the library owns only ks_ctx / ks_model.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream). Batch
 *     calls only enqueue work on that stream; they do not synchronise.
 *   - A context is bound to one device and is not thread-safe: use one per host thread.
 *   - Every batch call of a context (ks_featurize, ks_score, ks_select, ks_valid_catalogue, ...)
 *     uses the context's one device workspace, which is grown on demand: calls on one context
 *     must go on one stream, or be serialised by the caller.
 *   - A kernel whose bounded device-side wait gives up sets the context's status word and the
 *     call's results are void. ks_select_one and ks_select_host report it themselves
 *     (KS_ERR_TIMEOUT); after an asynchronous call, ks_device_status reports and clears it, and
 *     must be called before the context's next call once a failure is suspected.
 *   - All structs are plain little-endian PODs with exactly the fields shown.
 */
#ifndef KS_H_
#define KS_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define KS_F 63          /* number of features (columns 0..62 of a feature row)            */
#define KS_F_PAD 64      /* a feature row is 64 fp32; column 63 is always 0                */
#define KS_F_ONEHOT 80   /* input width of the ranker's one-hot form */
#define KS_MAX_K 32      /* largest k accepted by ks_select / ks_select_one                */
#define KS_MAX_DEPTH 15  /* deepest tree accepted (a leaf index must fit 16 bits)          */
#define KS_MAX_DIM (1u << 19) /* largest M, N or K for which all int64 products are exact  */
#define KS_MLP_MAX_LAYERS 6
#define KS_MLP_MAX_WIDTH 1024

typedef int ks_status;
enum {
  KS_OK = 0,
  KS_ERR_INVALID_ARG = 1, /* null pointer, size out of range, malformed model              */
  KS_ERR_UNSUPPORTED = 2, /* valid request this build has no kernel for                    */
  KS_ERR_CUDA = 3,        /* a CUDA runtime call failed; see ks_last_cuda_error            */
  KS_ERR_TIMEOUT = 4,     /* a bounded device-side wait gave up (status word set)          */
  KS_ERR_OOM = 5          /* device or host allocation failed                              */
};

/* GEMM instance p = (M, N, K, layout) (section "Problem and Candidate Sets"), extended with
 * the operand / output types and the epilogue-fusion kind of the transfer studies. */
typedef struct {
  uint32_t m, n, k;   /* 1 .. KS_MAX_DIM                                                   */
  uint8_t layout;     /* 0 TN, 1 TT, 2 NN, 3 NT (order of Table "Configuration knobs")     */
  uint8_t dtype_ab;   /* 0 fp16, 1 bf16, 2 fp8_e4m3, 3 tf32                                */
  uint8_t dtype_d;    /* 0 fp16, 1 bf16, 2 fp8_e4m3, 3 fp32                                */
  uint8_t epi_flags;  /* bit0 bias; bits1-2 activation: 0 none, 1 ReLU, 2 GELU             */
} ks_problem;         /* 16 bytes, 16-byte aligned in arrays                               */

/* One CUTLASS configuration c (Table "Configuration knobs"). All extents >= 1. */
typedef struct {
  uint16_t tile_m, tile_n, tile_k; /* thread-block tile T_M x T_N x T_K                    */
  uint16_t instr_n;                /* instruction tile N extent                            */
  uint8_t stages;                  /* mainloop pipeline stages S                           */
  uint8_t cluster_m, cluster_n;    /* cluster shape c_M x c_N                              */
  uint8_t kernel_sched;            /* 0 WS, 1 Pingpong, 2 Cooperative, 3 TMA-basic         */
  uint8_t epi_sched;               /* 0 NoSmem, 1 TMA, 2 TMA-Cooperative                   */
  uint8_t tile_sched;              /* 0 Persistent, 1 Stream-K                             */
  uint8_t instr_m, instr_k;        /* instruction tile M and K extents                     */
} ks_candidate;                    /* 16 bytes, 16-byte aligned in arrays                  */

/* Hardware descriptor h (section "Structural Core": SM count, shared-memory and register
 * capacities, LLC capacity, memory bandwidth, compute-engine peak). Plain data: the values
 * describe the target the candidates would run on, not the GPU libks itself runs on. */
typedef struct {
  uint32_t num_sms;            /* S_SM                                                     */
  uint32_t smem_per_sm;        /* C_smem, bytes                                            */
  uint32_t smem_per_cta_max;   /* largest footprint one CTA may request, bytes             */
  uint32_t smem_reserved;      /* bytes added to every footprint                           */
  uint32_t regs_per_sm;        /* C_reg, 32-bit registers                                  */
  uint32_t max_threads_per_sm;
  uint32_t max_ctas_per_sm;
  uint32_t reserved0;          /* must be 0                                                */
  uint64_t l2_bytes;           /* LLC capacity                                             */
  uint64_t tma_bytes_per_us;   /* aggregate load bandwidth BW_TMA, bytes per microsecond   */
  uint64_t tc_flops_per_us_per_sm[4]; /* per-SM tensor rate by dtype_ab, flop per us       */
} ks_gpu_desc;                 /* 80 bytes                                                 */

/* Interchange form of one tree node. Node 0 of a tree is its root. An internal node sends
 * a row to `left` when x[feat] < thr (strict, fp32) and to `left + 1` otherwise; a leaf has
 * feat == 0xFFFF and carries its value in thr_or_leaf. Indices are relative to the tree.
 * kind == KS_NODE_PARTITION marks a partition split on a categorical field (section "Model A":
 * native categorical handling with a fixed level ordering): feat must be one of the columns
 * that hold a level code (layout flags 3, 4; operand type 5; bias flag 8; activation 9; kernel
 * schedule 17; epilogue schedule 18; tile scheduler 19), the bit pattern of thr_or_leaf is a
 * non-zero membership mask over the field's level codes (bit c = level c), and a row whose
 * level is in the set goes to `left + 1`, any other row to `left`. Feature rows given to
 * ks_score must hold one of the field's level codes in such a column; which way any other
 * value (not a level, NaN, infinite) goes at a partition split is unspecified. At a numeric
 * split a NaN goes to `left + 1`, as x < thr is false. */
#define KS_NODE_NUMERIC 0
#define KS_NODE_PARTITION 1
typedef struct {
  float thr_or_leaf;
  uint16_t feat;   /* 0 .. KS_F-1, or 0xFFFF for a leaf                                    */
  uint16_t kind;   /* KS_NODE_NUMERIC or KS_NODE_PARTITION; 0 for a leaf                   */
  int32_t left;    /* index of the left child (right child = left + 1); 0 for a leaf       */
} ks_node_host;    /* 12 bytes                                                             */

/* Device form of a tree node, for ks_select_trees_static only (models created through
 * ks_model_create_gbdt are repacked by the library). 8 bytes. */
typedef struct {
  float thr_or_leaf; /* threshold of an internal node, value of a leaf                    */
  uint16_t feat;     /* 0 .. KS_F-1 (| 0x8000: partition split, thr_or_leaf = level mask), */
                     /* or 0xFFFF for a leaf                                               */
  uint16_t left;     /* tree-relative index of the left child (right child = left + 1)     */
} ks_node_dev;

#define KS_STATIC_MAX_KEYS 524288 /* partial top-k entries ks_select_trees_static can hold  */

typedef struct ks_ctx ks_ctx;
typedef struct ks_model ks_model;
typedef struct ks_catalogue ks_catalogue;

/* ---- context ------------------------------------------------------------------------- */

/* Create a context on CUDA device `cuda_device` for the target described by *desc (copied).
 * Fails with KS_ERR_INVALID_ARG on a null pointer or a descriptor with a zero capacity or
 * rate, KS_ERR_CUDA / KS_ERR_OOM if the device cannot be used. */
ks_status ks_create(ks_ctx** out_ctx, int cuda_device, const ks_gpu_desc* desc);
ks_status ks_destroy(ks_ctx* ctx);
/* Text of the last CUDA error seen by this context ("" if none). Owned by the context. */
const char* ks_last_cuda_error(const ks_ctx* ctx);

/* ---- models -------------------------------------------------------------------------- */

/* Model A (section "Model A (gradient-boosted ranker)"): f(x) = base_score + sum_m h_m(x).
 * h_nodes holds the trees back to back, tree t in [h_tree_offsets[t], h_tree_offsets[t+1]).
 * All structural validation happens here, on the host: feature ids < KS_F, children inside
 * the tree and after their parent, finite thresholds and leaves, partition splits only on
 * level-code columns with a non-zero mask inside the field's levels, depth <= KS_MAX_DEPTH,
 * every node reachable exactly once. The trees are repacked into a private device layout;
 * the host arrays may be freed on return. Synchronous. */
ks_status ks_model_create_gbdt(ks_ctx* ctx, int n_trees, const int64_t* h_tree_offsets,
                               const ks_node_host* h_nodes, float base_score,
                               ks_model** out_model);

/* Model B (section "Model B (feed-forward ranker)") with the standardisation folded in:
 * x'_j = (x_j - mu_j) / sigma_j for j < 63 with a non-finite x_j replaced by 0 first,
 * x'_63 = 0, rounded to bf16; every hidden layer is h = ReLU(W h_prev + b) with fp32
 * accumulation, rounded to bf16; the last layer (width 1) is s = w . h + b in fp32.
 * h_widths = {64, w_1, ..., w_{L-1}, 1} (n_layers = L weight matrices, 1 <= L <=
 * KS_MLP_MAX_LAYERS; hidden widths multiples of 64, <= KS_MLP_MAX_WIDTH). L = 1 is the linear
 * scorer w . x' + b of section "Linear Ridge Baseline". h_w_bf16[l] is
 * row-major [out, in] bf16 bit patterns, h_bias[l] is [out] fp32; h_mu / h_sigma are
 * [h_widths[0]] fp32 with sigma != 0. Synchronous.
 * h_widths[0] = KS_F_ONEHOT selects the one-hot input form (section "Model B": categorical
 * fields one-hot encoded): positions 0..58 are the feature columns other than 5, 9, 17, 18 in
 * ascending order; 59..62, 63..65, 66..69, 70..72 are the level indicators (0 / 1) of operand
 * type (column 5), activation (9), kernel schedule (17) and epilogue schedule (18); 73..79 are
 * zero. mu / sigma apply position by position (indicators included). */
ks_status ks_model_create_mlp(ks_ctx* ctx, int n_layers, const int* h_widths,
                              const uint16_t* const* h_w_bf16, const float* const* h_bias,
                              const float* h_mu, const float* h_sigma, ks_model** out_model);

/* The static sampling score of the paper's data-collection policy as a scorer with no learned
 * parameters: with n_c = ceil(M / (c_M T_M)) * ceil(N / (c_N T_N)) clusters and
 * W = ceil(n_c / S_SM) cluster waves, s = n_c / (W S_SM c_M c_N) * S * sqrt(T_M T_N T_K)
 * (S_SM read as the SM count). Usable with ks_select / ks_select_one / ks_select_host (ranking
 * by it is the paper's "static top-B" policy); ks_score returns KS_ERR_UNSUPPORTED because the
 * score is a function of (p, c), not of the feature row. */
ks_status ks_model_create_static(ks_ctx* ctx, ks_model** out_model);

/* Frees the model's device buffers. A model may be destroyed before or after its context, but
 * must not be used in a call once the context is gone. */
ks_status ks_model_destroy(ks_model* model);

/* ---- search space and validity (the steps in front of the path) --------------------------- */

/* Combinations per layout of the searched knobs (Table "Configuration knobs"):
 * 4 tile_m * 9 tile_n * 5 tile_k * 11 stages * 15 cluster shapes * 3 kernel schedules *
 * 3 epilogue schedules * 2 tile schedulers. */
#define KS_CATALOGUE_SIZE 534600

/* ks_valid_catalogue flags. KS_VALID_COUPLED adds the two couplings between epilogue and
 * mainloop schedule that the schedule names imply but the paper's table does not list
 * (TMA-Cooperative epilogue <=> cooperative mainloop; TMA epilogue => non-cooperative mainloop).
 * KS_VALID_WASTEFUL adds the rule of section "Validity Constraints" that drops candidates with
 * T_N > 2M or T_N > 2N. KS_VALID_PRINTED_CAPACITY applies the capacity rule exactly as Table
 * "Static validity constraints" prints it, mainloop + epilogue + reserve <= capacity for every
 * schedule; without it the schedule-specific footprint of feature column 49 is compared
 * (warp-specialised mainloops reuse their buffers for the epilogue), the reading that
 * reproduces the paper's between-layout count differences. */
#define KS_VALID_COUPLED 1u
#define KS_VALID_WASTEFUL 2u
#define KS_VALID_PRINTED_CAPACITY 4u

/* Writes the candidates with linear ids first .. first+count-1 of the search space to
 * d_out[0..count) (device, 16-byte aligned, caller-owned). The id is a mixed-radix number whose
 * digits follow the rows of Table "Configuration knobs", first row slowest: tile_m
 * {64,128,192,256}, tile_n {16,32,48,64,80,96,128,192,256}, tile_k {32,64,128,256,512}, stages
 * 2..12, cluster shape (the 15 pairs of {1,2,4,8,16} with c_M c_N <= 16, c_M slowest),
 * kernel_sched {0 WS, 1 Pingpong, 2 Cooperative}, epi_sched {0 NoSmem, 1 TMA, 2 TMA-Cooperative},
 * tile_sched {0 Persistent, 1 Stream-K}; instruction shape 64 x tile_n x 16. Asynchronous on
 * `stream`. KS_ERR_INVALID_ARG unless 0 <= first, 0 <= count, first + count <=
 * KS_CATALOGUE_SIZE. */
ks_status ks_enumerate(ks_ctx* ctx, int64_t first, int64_t count, ks_candidate* d_out, void* stream);

/* Static validity filter (Table "Static validity constraints") with order-preserving
 * compaction. The rules: Stream-K => cooperative mainloop; cooperative mainloop => T_M = 0 mod
 * 128; shared-memory footprint of one CTA (feature column smem_total, which includes the
 * descriptor's reserve) <= smem_per_cta_max; A column-major => T_K <= 256 C_N; B row-major =>
 * T_K <= 256 C_M; plus the rules `flags` selects.
 *   problem       host pointer, one record: its layout and element types decide; m and n are
 *                 read only under KS_VALID_WASTEFUL
 *   d_candidates  device, [C] records, 16-byte aligned; NULL = the search space's ids 0..C-1
 *                 generated on the fly (then C <= KS_CATALOGUE_SIZE)
 *   d_out         device, capacity C records, 16-byte aligned, or NULL: the valid candidates in
 *                 input order
 *   d_out_index   device, capacity C, or NULL: their positions in the input (= ids)
 *   d_count       device, one int32: how many are valid
 *   h_count       host, or NULL; when given the call copies the count there and waits for the
 *                 stream, otherwise it is asynchronous on `stream`
 * Entries of d_out / d_out_index past the count are left untouched. Uses the context's
 * workspace (calls on one context must not overlap). */
ks_status ks_valid_catalogue(ks_ctx* ctx, const ks_problem* problem, unsigned flags,
                             const ks_candidate* d_candidates, int C, ks_candidate* d_out,
                             int32_t* d_out_index, int32_t* d_count, int32_t* h_count, void* stream);

/* d_idx[i] <- d_map[d_idx[i]] for 0 <= d_idx[i] < map_len, else -1: turns top-k positions in a
 * compacted catalogue (ks_select on ks_valid_catalogue's d_out) back into positions of the
 * unfiltered one (d_map = its d_out_index). In place, asynchronous on `stream`. */
ks_status ks_remap_indices(ks_ctx* ctx, int32_t* d_idx, int64_t n, const int32_t* d_map, int map_len,
                           void* stream);

/* ---- the three calls of the selection path -------------------------------------------- */

/* Candidate sets: with d_seg_offsets == NULL every problem is ranked against the whole pool
 * d_c[0..C) (dense P x C; pairs = P*C, pair (i, j) is row i*C + j). Otherwise problem i is
 * ranked against d_c[d_seg_index[j]] for j in [d_seg_offsets[i], d_seg_offsets[i+1])
 * (d_seg_offsets has P+1 non-decreasing entries starting at 0; row j belongs to pair j).
 * A problem's candidate set is a set: the indices of one segment must be distinct (for the
 * ranking calls; an index listed twice is reported once by some kernels and twice by others). */

/* x = phi(p, c, h) for every pair (Table "Feature groups"; the column list is
 * ks_feature_name). Writes pairs x 64 fp32, row-major. `pairs` must equal P*C or
 * seg_offsets[P] (the caller states it so that no device read is needed on the host). */
ks_status ks_featurize(ks_ctx* ctx, const ks_problem* d_p, int P, const ks_candidate* d_c,
                       int C, const int64_t* d_seg_offsets, const int32_t* d_seg_index,
                       int64_t pairs, float* d_features, void* stream);

/* s = f_theta(x) for `rows` feature rows (row-major [rows, 64] fp32). For a tree model,
 * d_leaf_idx (nullable, [rows, n_trees] uint16) receives the tree-relative node index of
 * the leaf each tree ends in. Must be NULL for an MLP. Without leaf indices, an ensemble that
 * qualifies for the quantised walk of ks_select is scored by that walk on the given rows (the
 * leaf values are then added in that kernel's order, not tree by tree; same tolerance); the
 * call may grow the context's workspace, so it orders after earlier work like ks_select does.
 * An MLP that the tensor-core kernel of ks_select serves (input width 64, one or two hidden
 * layers of at most 256 units) is scored by that kernel on the given rows. Non-finite inputs
 * of an MLP count as 0 before standardisation. */
ks_status ks_score(ks_ctx* ctx, const float* d_features, int64_t rows, const ks_model* model,
                   float* d_scores, uint16_t* d_leaf_idx, void* stream);

/* Fused featurize + score + per-problem top-k (Eq. "selection" as a shortlist): for problem
 * i the k best pairs of its candidate set ordered by (score descending, pool index
 * ascending). d_topk_idx [P, k] receives pool indices (-1 where the set has fewer than k
 * members), d_topk_score [P, k] the scores (-inf there). 1 <= k <= KS_MAX_K. The feature
 * matrix and the scores are never written to memory. `pairs` as in ks_featurize. The call
 * sizes the context's workspace (owned by the context, grown on demand, which synchronises the
 * device when it happens): partial lists, a per-call table of 16 x C records of at most 256
 * bytes, and, for a tree model on a batch of 32 problems or more, at most 256 MiB for the
 * tables of per-pair tile rows (larger batches are served in several launches that reuse it);
 * KS_ERR_OOM if the workspace cannot be had. d_p and d_c must be 16-byte aligned (each record
 * is fetched with one 128-bit load), else KS_ERR_INVALID_ARG. */
ks_status ks_select(ks_ctx* ctx, const ks_problem* d_p, int P, const ks_candidate* d_c, int C,
                    const int64_t* d_seg_offsets, const int32_t* d_seg_index, int64_t pairs,
                    const ks_model* model, int k, int32_t* d_topk_idx, float* d_topk_score,
                    void* stream);

/* Latency form of ks_select for one problem passed by value against the dense pool
 * d_c[0..C): h_topk_idx / h_topk_score ([k], host memory, pinned for best latency) are
 * valid when the call returns (it synchronises `stream`). */
ks_status ks_select_one(ks_ctx* ctx, ks_problem p, const ks_candidate* d_c, int C,
                        const ks_model* model, int k, int32_t* h_topk_idx,
                        float* h_topk_score, void* stream);

/* A candidate catalogue prepared for a stream of single-problem calls with one model (the
 * dynamic-selection setting: problems arrive one at a time, the catalogue and the ranker stay).
 * Everything about a call that depends only on (catalogue, model) is computed here, once: for a
 * tree ensemble on the quantised path, every candidate's quantised candidate-only columns under
 * each of the 16 element-type combinations and the classes of candidates that look alike to
 * the per-pair columns. ks_select_one_prepared then evaluates the per-pair columns once per class
 * for the problem at hand and runs the fused walk + top-k: two launches per call instead of
 * building the candidates' tiles anew. The handle owns its device memory (a few hundred bytes
 * per candidate), refers to d_c and the model (both must outlive it and stay unchanged) and
 * belongs to the context. For models the quantised path does not serve, the handle is a plain
 * reference and ks_select_one_prepared is ks_select_one. Synchronises `stream`. */
ks_status ks_catalogue_prepare(ks_ctx* ctx, const ks_candidate* d_c, int C, const ks_model* model,
                               ks_catalogue** out_catalogue, void* stream);
ks_status ks_catalogue_destroy(ks_catalogue* catalogue);
/* ks_select_one against a prepared catalogue: same results, same conventions. */
ks_status ks_select_one_prepared(ks_ctx* ctx, const ks_catalogue* catalogue, ks_problem p, int k,
                                 int32_t* h_topk_idx, float* h_topk_score, void* stream);

/* ks_select for callers whose inputs live in HOST memory: copies problems, candidates and
 * segment arrays to the device, runs ks_select, copies the [P, k] results back and
 * synchronises. Device staging comes from the context's workspace (grown on demand). */
ks_status ks_select_host(ks_ctx* ctx, const ks_problem* h_p, int P, const ks_candidate* h_c,
                         int C, const int64_t* h_seg_offsets, const int32_t* h_seg_index,
                         int64_t pairs, const ks_model* model, int k, int32_t* h_topk_idx,
                         float* h_topk_score, void* stream);

/* Merge of partial top-k lists (Eq. "selection" over a candidate set that was split: the best k
 * of a union are among the best k of its parts). For each of P problems, d_idx / d_score hold n
 * gathered (pool index, score) entries, row-major [P, n], an index of -1 marking an empty
 * entry; d_topk_idx / d_topk_score [P, k] receive the k best by (score descending, index
 * ascending), padded with -1 / -inf. This is the one exchange step of the multi-GPU forms: ranks
 * that each ranked a share of the candidates gather their lists and merge them here.
 * Asynchronous on `stream`. */
ks_status ks_merge_topk(ks_ctx* ctx, const int32_t* d_idx, const float* d_score, int P, int n, int k,
                        int32_t* d_topk_idx, float* d_topk_score, void* stream);

/* ---- selection without any allocation ------------------------------------------------------- */

/* (The paper has no counterpart: this entry point exists for deployment reasons only.)
 * The dense form of ks_select for a tree ensemble, for callers that cannot allocate device
 * memory at all: processes whose own pool already owns the whole GPU, code running between
 * cudaStreamBeginCapture and EndCapture or inside a stream-ordered pipeline that a
 * synchronising cudaMalloc / cudaFree would stall, hosts that forbid driver allocations after
 * start-up. Such callers cannot create a ks_ctx or ks_model (both own device buffers), so
 * everything arrives as plain device pointers on device `cuda_device`:
 *   d_nodes / d_tree_offsets  the ensemble as ks_node_dev records, tree t occupying
 *                             [d_tree_offsets[t], d_tree_offsets[t+1]) (n_trees + 1 int32 offsets),
 *                             node 0 of a tree its root. The arrays are NOT validated (they are
 *                             device memory): child indices must stay inside their tree, feature
 *                             ids below KS_F, depth at most KS_MAX_DEPTH.
 *   d_p[P], d_c[C]            problems and the candidate pool; every problem is ranked against
 *                             the whole pool.
 *   d_topk_idx / d_topk_score [P, k] results as for ks_select.
 * The call launches the same fused kernels as ks_select's generic tree path, asynchronously on
 * `stream`, and calls no cudaMalloc, cudaFree or other allocating routine. The only scratch the
 * kernels need, the per-block partial top-k lists, lives in a fixed 4 MiB array inside the
 * library image (every GPU that loads libks holds it until the process exits). Limits and rules:
 *   - P * B * k must not exceed KS_STATIC_MAX_KEYS, where B <= ceil(C / 256) is the number of
 *     candidate blocks per problem the launcher picks; P * ceil(C / 256) * k <=
 *     KS_STATIC_MAX_KEYS is always sufficient. Larger requests return KS_ERR_UNSUPPORTED and
 *     launch nothing.
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress);
 *     make that first call outside any stream capture. With CUDA's lazy module loading that
 *     first call is also what places the kernels' code and the 4 MiB array on the device: a
 *     caller whose own pool takes all remaining memory must make it BEFORE the pool does.
 *   - All calls share the one array, which keeps the previous call's contents. The kernels
 *     write every entry they later read, so nothing has to be cleared, but two calls whose
 *     kernels overlap on the GPU (different streams, or different host threads) race on it:
 *     serialise them.
 * Returns KS_OK, KS_ERR_INVALID_ARG, KS_ERR_UNSUPPORTED or KS_ERR_CUDA. */
ks_status ks_select_trees_static(int cuda_device, const ks_gpu_desc* desc, const ks_problem* d_p, int P,
                                 const ks_candidate* d_c, int C, const ks_node_dev* d_nodes,
                                 const int32_t* d_tree_offsets, int n_trees, float base_score, int k,
                                 int32_t* d_topk_idx, float* d_topk_score, void* stream);

/* ---- introspection -------------------------------------------------------------------- */

const char* ks_status_string(ks_status s);
int ks_feature_count(void);             /* KS_F                                            */
const char* ks_feature_name(int index); /* NULL if index is outside 0..KS_F-1              */
/* Number of kernels libks launched on behalf of this context since creation. */
int64_t ks_launch_count(const ks_ctx* ctx);
/* Waits for all work of the context's device and reports (then clears) the status word that
 * kernels set when one of their bounded device-side waits gave up: KS_OK or KS_ERR_TIMEOUT.
 * ks_select_one and ks_select_host perform this check themselves. */
ks_status ks_device_status(ks_ctx* ctx);
/* Measurement aid (the paper has no counterpart): with profiling on, every ks_select records a
 * CUDA event on the caller's stream before and after its dominant kernel (the fused
 * featurize + score + partial top-k kernel, excluding the small merge that follows).
 * ks_profile_last_ms waits for the last such kernel and returns its duration. */
ks_status ks_profile_enable(ks_ctx* ctx, int on);
ks_status ks_profile_last_ms(ks_ctx* ctx, float* out_ms);
/* One line naming the fused kernel that ks_select runs for this model and, for a tree
 * ensemble on the quantised path, its tile geometry (threads per CTA x candidates per CTA),
 * rows and distinct thresholds. Written to buf (at most len bytes, always terminated). */
ks_status ks_model_describe(const ks_model* model, char* buf, int len);

/* ---- test hooks (the paper has no counterpart) ------------------------------------------- */

/* Bounded device-side waits of this context's kernels: `probe_limit` > 0 replaces the number
 * of probes a wait may take before it gives up (0 restores the default, tens of milliseconds);
 * `starve` != 0 makes the tree kernel arm each chunk barrier for 16 bytes more than its copy
 * brings, and the tensor-core kernel skip the copy of its weight image, so that the first wait
 * runs out, the kernel sets the status word and returns, and the call reports KS_ERR_TIMEOUT
 * without any fault: the failure path can be tested on a healthy GPU. */
ks_status ks_debug_set_wait(ks_ctx* ctx, int probe_limit, int starve);
/* Measurement aid, no counterpart in the paper: the tree walk of ks_score stripped of everything
 * but its gather and instruction stream, to measure the floor that stream sets for the tree
 * kernel. Tiles are built from the `rows` feature rows (device, [rows][64] floats) exactly as
 * ks_score builds them; every CTA then copies the first chunks of the ensemble once (two per
 * tree group: the CTA's threads / 256 groups deal the chunks among themselves, group g taking
 * chunks g, g + G, ...) and every group walks its two resident chunks as often as `repeat` passes
 * over the whole ensemble would make it walk chunks, without waiting for, releasing or refilling
 * a chunk buffer; the sums go to d_scores (device, [rows]; with one group, c0 and c1 the sums of
 * the two chunks' leaves for a
 * row and n = repeat x n_chunks: base + ceil(n / 2) c0 + floor(n / 2) c1). The time of a pass is
 * the difference of two calls with different `repeat`, divided by the difference. Tree models on
 * the quantised kernel with 1,024-candidate tiles, three word-wise and five path levels only
 * (the benchmark's ensemble); anything else returns KS_ERR_UNSUPPORTED. 1 <= repeat <= 4096.
 * Asynchronous on `stream`; uses the context's workspace like ks_score. */
ks_status ks_debug_walk_floor(ks_ctx* ctx, const float* d_features, int64_t rows, const ks_model* model,
                              int repeat, float* d_scores, void* stream);
/* Checked build only (libks_debug.so, compiled with KS_DEBUG_BOUNDS): the kernels compare
 * every index they form from data with its range and, instead of touching memory out of range,
 * record the source line of the first violation. Returns that line, 0 when there was none,
 * -1 in a regular build; ks_debug_bounds_clear resets it. Both synchronise the device. */
int ks_debug_bounds_line(void);
void ks_debug_bounds_clear(void);

#ifdef __cplusplus
}
#endif
#endif /* KS_H_ */
