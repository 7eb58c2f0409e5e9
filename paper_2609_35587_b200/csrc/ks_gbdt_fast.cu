// Quantised fast path of the fused select kernel for tree ensembles (Model A).
//
// Repack (host, at model-create time)
//   A split "x[f] < thr" only needs to know how many of feature f's distinct thresholds are
//   <= x. With the thresholds of f sorted, bin(x) = #{j : thr_j <= x}, and
//   x < thr_j  <=>  bin(x) <= j  exactly. A feature's thresholds are cut into slices of 127; a
//   "row" is one slice, a pair's byte in that row the number of the slice's thresholds that are
//   <= x (0..127), and a node one 32-bit word (row offset, index within the slice). A feature
//   with thousands of distinct thresholds (an ensemble trained by exact greedy splitting) simply
//   owns more rows; the tile geometry follows the row count (see FastGeom). Trees are padded to
//   complete trees of the ensemble's depth D and stored in chunks, each chunk laid out level by
//   level ([level][tree][node]) followed by its leaves, so that a chunk is one contiguous block
//   a CTA copies into shared memory with one bulk async copy. The nodes of the top levels are
//   also kept as (row offset, replicated threshold) pairs that travel as a kernel parameter,
//   i.e. through the constant bank.
//   A partition split on a categorical field ("level in S goes right") joins the same scheme
//   through rank rows: a row whose byte is the rank of the pair's level in a fixed ordering of
//   the field's levels, chosen so that S or its complement is the set of ranks >= c; the node
//   then is the ordinary "bin <= c - 1 goes left", with its children exchanged for a complement.
//
// Hoisting
//   Rows are grouped by what their feature depends on. Candidate-only rows (given the
//   problem's element types) are quantised once per call by cand_rows_kernel into a table
//   indexed by (type combination, candidate); problem-only rows once per CTA; only the
//   per-pair rows are computed and searched for every pair - or, in a batch of problems, once
//   per (problem, class of candidates that look alike to the per-pair columns) and copied
//   (see MemoView).
//
// Other entries into the same walk
//   single-problem call: the trees are split over several CTAs per candidate block (slices),
//   the tiles are built once by tile_one_kernel; scoring call (ks_score): tiles are quantised
//   from given feature rows by tile_rows_kernel and the scores are stored instead of ranked.
//
// Kernel (an item = one problem x up to NC candidates; a CTA of THREADS threads serves one item,
// or - batch form of the geometries with one CTA per SM - a run of items: one candidate block
// for problem after problem, whose candidate-only rows it keeps in the tile)
//   phase A  fill the [row][candidate] byte tile. A 32-bit word of a row holds the four
//            candidates that share a lane slot, so a warp's byte loads of any mix of rows
//            touch 32 distinct banks and one word load serves four candidates;
//   phase B  stream the ensemble through rings of two shared-memory buffers (cp.async.bulk +
//            mbarrier, bounded waits). Thread (w, g) owns the four candidates of word w and
//            walks group g's share of the trees: the chunks of its ring (see ring_count), and of
//            those the trees that fall to it when two groups share a ring. The top levels are evaluated for all four
//            candidates at once, node by node, with byte-parallel arithmetic on whole words;
//            below that each candidate follows its own path: a' = 2 a + k0 (+ 4 to go right), a
//            multiply-add plus a predicated add;
//   phase C  add the groups' partial scores, rank the block's keys, write a partial top-k list.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <limits>
#include <new>
#include <vector>

#include "ks_features.cuh"
#include "ks_internal.h"
#include "ks_memo.cuh"
#include "ks_topk.cuh"

namespace ks {

namespace {

constexpr int kBufBytes = 16 * 1024;   // one tree-chunk buffer (twice that where the shared memory allows)
constexpr int kSlice = 127;            // thresholds per row: a byte is 0x80 | (0..127)
constexpr unsigned kSleepNs = 1200;    // asked-for sleep between two probes of a chunk barrier (400 to 2500 measured alike)
constexpr int kCombos = 16;            // dtype_ab x dtype_d

constexpr int kSmCount = 148;           // SMs of the one device this library is built for (sm_100a)
// Chunk rings of a CTA with G tree groups: every ring has kNBuf buffers and serves G / rings groups,
// which share out the trees of its chunks; ring r takes the chunks r, r + rings, ... A ring of
// its own per group means that only the group's warps meet at a buffer's release, for the same
// shared memory and the same trees per thread and chunk (config 1, two groups: 55.3 -> 54.4 ms);
// four groups do best with two rings (config 2: 132.4 ms with four rings, 131.6 with one, 129.3 with two).
__host__ __device__ constexpr int ring_count(int groups) { return groups <= 2 ? groups : 2; }
constexpr int kNBuf = 2;                // buffers of a ring (four of 8 KB and three of 12 KB measured slower)
// shared memory map (byte offsets from the dynamic shared base): the rings' chunk buffers, then the tile
constexpr int kOffBuf0 = 0;

#ifdef KS_DEBUG_BOUNDS
// Checked build: every index formed from data (tile byte, node, chunk, record, partial list) is
// compared with its range; a violation records its source line in this word and uses element 0.
__device__ int g_bounds_line;
__device__ __forceinline__ long long checked_index(long long i, long long n, int line) {
  if (i < 0 || i >= n) {
    atomicCAS(&g_bounds_line, 0, line);
    return 0;
  }
  return i;
}
#define KS_IDX(i, n) checked_index(static_cast<long long>(i), static_cast<long long>(n), __LINE__)
#else
#define KS_IDX(i, n) (i)
#endif

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: one probe, then sleep-and-probe (measured faster than the blocking try_wait with
// or without a time hint); gives up after `limit` probes, or as soon as another warp of the CTA
// has given up (`fail`), and reports false.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, int limit, volatile int* fail) {
  if (mbar_test_wait(bar, parity)) return true;
  for (int i = 0; i < limit; ++i) {
    __nanosleep(kSleepNs);
    if (mbar_test_wait(bar, parity)) return true;
    if ((i & 63) == 63 && *fail) return false;
  }
  return false;
}
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ float lds_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
  return v;
}

// Raised by a CTA whose bounded wait ran out, so that the CTAs after it leave at once; cleared by
// the per-call table kernel that precedes every launch of the select kernel.
__device__ int g_fast_abort;

// #{j < n : T[j] <= v} over n sorted thresholds.
__device__ __forceinline__ int count_le(const float* T, int n, float v) {
  int pos = 0;
  for (int s = n > 0 ? 1 << (31 - __clz(n)) : 0; s >= 1; s >>= 1) {
    const int np = pos + s;
    if (np <= n && T[np - 1] <= v) pos = np;
  }
  return pos;
}

// Tile bytes of one feature value: slice s of the feature's thresholds gets the number of its
// thresholds that are <= v, i.e. the overall count less 127 s clamped to 0..127; a rank row gets
// the rank of the level code v. `T` is the feature's own sorted threshold array. With
// `nan_right` a NaN takes the last bin of every slice (x < t is false: it goes right).
// `pos` is the count of the feature's thresholds that are <= v (unused for a feature without slices).
template <typename Put>
__device__ __forceinline__ void emit_rows(const FeatQ& q, int pos, float v, Put put) {
  if (q.nslice) {
    for (int s = 0; s < q.nslice; ++s) {
      int b = pos - kSlice * s;
      b = b < 0 ? 0 : (b > kSlice ? kSlice : b);
      put(q.row0 + s, static_cast<uint8_t>(0x80 | b));
    }
  }
  if (q.nrank) {
    const int code = __float2int_rz(v);
    for (int r = 0; r < q.nrank; ++r)
      put(q.row0 + q.nslice + r, static_cast<uint8_t>(0x80 | ((code >= 0 && code < 4) ? q.rank[r][code] : 0)));
  }
}
template <typename Put>
__device__ __forceinline__ void quantise(const FeatQ& q, const float* T, float v, bool nan_right, Put put) {
  const int pos = q.nslice ? ((nan_right && v != v) ? q.nthr : count_le(T, q.nthr, v)) : 0;
  emit_rows(q, pos, v, put);
}

// The per-pair columns (class 2 of feat_class) in ascending order, and a column's place among them.
constexpr int kPairCols = 21;
__host__ __device__ constexpr int pair_slot(int col) {
  return col <= 36 ? col - 23 : (col == 39 ? 14 : (col <= 44 ? col - 26 : col - 41));
}
__host__ __device__ constexpr int pair_col(int slot) {
  return slot <= 13 ? slot + 23 : (slot == 14 ? 39 : (slot <= 18 ? slot + 26 : slot + 41));
}
constexpr bool pair_slots_match_classes() {
  int n = 0;
  for (int c = 0; c < KS_F; ++c)
    if (feat_class(c) == 2) {
      if (pair_slot(c) != n || pair_col(n) != c) return false;
      ++n;
    }
  return n == kPairCols;
}
static_assert(pair_slots_match_classes(), "per-pair columns");

// All per-pair columns of one pair at once: the binary searches advance in step (one probe of
// every column per round), so that a thread has 21 independent loads in flight instead of one
// dependent chain after the other. `T` is the staged (or global) array of per-pair thresholds.
template <typename Put>
__device__ __forceinline__ void quantise_pair_columns(const FeatQ* s_fq, const float* T, const float (&v)[kPairCols],
                                                      int max_thr, Put put) {
  int pos[kPairCols];
#pragma unroll
  for (int i = 0; i < kPairCols; ++i) pos[i] = 0;
  for (int s = max_thr > 0 ? 1 << (31 - __clz(max_thr)) : 0; s >= 1; s >>= 1) {
#pragma unroll
    for (int i = 0; i < kPairCols; ++i) {
      const FeatQ& q = s_fq[pair_col(i)];
      const int np = pos[i] + s;
      if (np <= q.nthr && T[q.thr0 + np - 1] <= v[i]) pos[i] = np;
    }
  }
#pragma unroll
  for (int i = 0; i < kPairCols; ++i) emit_rows(s_fq[pair_col(i)], pos[i], v[i], put);
}

// Byte of row i (0 .. 4 W - 1) of a block within one tile row of W words: the four rows of a
// word are consecutive, so that in a catalogue ranked in similarity order a thread's four
// candidates are near-duplicates.
__device__ __forceinline__ int tile_byte(int i, int) { return i; }

// Slice mode (single-problem latency call): the trees are split over n_slices CTAs per
// candidate block. Every CTA stores its partial scores; the last CTA to arrive for a block
// (atomic counter, nobody waits) adds the slices in a fixed order and ranks the block; the
// last block overall merges the lists and writes the final result.
struct SliceArgs {
  int n_slices;            // 1 = every CTA walks the whole ensemble
  long long pairs;         // rows of the partial-score planes
  float* scores;           // [n_slices][pairs] partial scores
  int* counters;           // [P * nblk + 1], zero on entry; every counter is reset by its last user
  int32_t* out_idx;        // single-problem form only: [k] final result (device-visible, may be
  float* out_score;        // mapped host memory); null when a merge kernel follows
  const uint8_t* tiles;    // prepared tiles [blocks][rows][NC] (tile_one_kernel), or null
  int* out_seq;            // single-problem form: receives `seq` once the k results are written
  int seq;
  float* score_out;        // scoring call (ks_score): the scores of the block's rows go here, no ranking
  int repeat;              // floor measurement only: passes over the resident chunks
};

struct FastView {
  int n_rows, n_pair_rows, n_cand_rows, n_prob_rows;  // rows are ordered pair, candidate, problem
  int depth, n_chunks, chunk_bytes, tpc;
  int n_thr, thr_cand0, thr_prob0;  // thresholds in all, and where the candidate-only / problem-only features' begin
  int cand_rec, pair_rec;           // bytes per record of the per-call tables (multiples of 16)
  int wait_limit, starve;           // probes a chunk wait may take; test hook: arm the barrier for bytes that never come
  int buf_bytes;                    // size of one chunk buffer in shared memory
  float base;
  const uint32_t* chunks;      // [n_chunks][chunk_bytes / 4]
  const float* thr;            // [n_thr] sorted thresholds, feature after feature (per-pair features first)
  const FeatQ* feat;           // [64] rows and thresholds of each feature column
  const uint8_t* cand_rows;    // [kCombos][C][cand_rec] quantised candidate-only rows
  const unsigned* pair_class;  // [kCombos][C] class of every candidate, or null (no memo)
  const uint8_t* pair_tab;     // [P][kMemoCap][pair_rec] per-pair tile bytes of every (problem, class)
  const uint8_t* prob_tab;     // [P][kProbRec] tile bytes of the problem-only rows and the problem's terms, or null
};

// ------------------------------------------------------------------------------------------
// candidate-only rows, once per call
// ------------------------------------------------------------------------------------------

__global__ void combo_mask_kernel(const ks_problem* __restrict__ p, int P, unsigned* __restrict__ mask) {
  unsigned m = 0;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < P; i += gridDim.x * blockDim.x) {
    const ks_problem pr = load_problem(p + i);
    m |= 1u << ((pr.dtype_ab & 3) * 4 + (pr.dtype_d & 3));
  }
  m = __reduce_or_sync(0xFFFFFFFFu, m);
  if ((threadIdx.x & 31) == 0 && m) atomicOr(mask, m);
}

// Thresholds of a range of features into shared memory when they fit `cap` floats, else the
// global array is searched in place. Returns the pointer that stands for fv.thr + first.
__device__ __forceinline__ const float* stage_thresholds(const FastView& fv, int first, int count, float* s_thr,
                                                         int cap) {
  if (count > cap) return fv.thr + first;
  const int vec = (first & 3) == 0 ? count / 4 : 0;  // whole 16-byte words when the source is aligned like s_thr
  for (int i = threadIdx.x; i < vec; i += blockDim.x)
    reinterpret_cast<float4*>(s_thr)[i] = __ldg(reinterpret_cast<const float4*>(fv.thr + first) + i);
  for (int i = 4 * vec + threadIdx.x; i < count; i += blockDim.x) s_thr[i] = __ldg(fv.thr + first + i);
  return s_thr;
}

__global__ void __launch_bounds__(256)
cand_rows_kernel(ks_gpu_desc desc, const ks_candidate* __restrict__ c, int C, const unsigned* mask_ptr,
                 unsigned mask_value, FastView fv, uint8_t* __restrict__ out, MemoView memo, int thr_cap) {
  extern __shared__ float s_cthr[];  // thresholds of the candidate-only features
  __shared__ FeatQ s_fq[64];
  const int combo = blockIdx.y;
  if (blockIdx.x == 0 && combo == 0 && threadIdx.x == 0) g_fast_abort = 0;
  const unsigned mask = mask_ptr ? *mask_ptr : mask_value;
  if (!((mask >> combo) & 1u)) return;
  const float* T = stage_thresholds(fv, fv.thr_cand0, fv.thr_prob0 - fv.thr_cand0, s_cthr, thr_cap) - fv.thr_cand0;
  if (threadIdx.x < 64) s_fq[threadIdx.x] = fv.feat[threadIdx.x];
  __syncthreads();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= C) return;
  ks_problem fake{};
  fake.m = fake.n = fake.k = 1;
  fake.dtype_ab = static_cast<uint8_t>(combo >> 2);
  fake.dtype_d = static_cast<uint8_t>(combo & 3);
  ProblemTerms t;
  problem_terms(fake, desc, t);
  const ks_candidate cand = load_candidate(c + i);
  uint8_t* rec = out + (static_cast<size_t>(combo) * C + i) * fv.cand_rec;
  const int first = fv.n_pair_rows;
  featurize_pair(t, cand, desc, [&](int col, float v) {
    if (feat_class(col) != 1) return;
    const FeatQ& q = s_fq[col];
    quantise(q, T + q.thr0, v, false, [&](int row, uint8_t b) { rec[KS_IDX(row - first, fv.cand_rec)] = b; });
  });
  if (memo.keys)
    memo.cls[static_cast<size_t>(combo) * C + i] = memo_assign(memo, combo, i, cand, resources(t, cand, desc).b_eff);
}

// Packs the occupied slots of every type combination's table (one block per combination), so
// that the per-problem kernel runs full warps over classes only.
__global__ void __launch_bounds__(1024)
memo_compact_kernel(MemoView memo) {
  __shared__ int s_n;
  const int combo = blockIdx.x;
  if (threadIdx.x == 0) s_n = 0;
  __syncthreads();
  for (int slot = threadIdx.x; slot < kMemoCap; slot += 1024)
    if (memo.keys[static_cast<size_t>(combo) * kMemoCap + slot] != 0ull)
      memo.dense[static_cast<size_t>(combo) * kMemoCap + atomicAdd(&s_n, 1)] = slot;
  __syncthreads();
  if (threadIdx.x == 0) memo.count[combo] = s_n;
}

// Per problem: the tile bytes of the per-pair rows of every class, from the class's member, plus
// (last block of a row) the problem's own terms and the tile bytes of its problem-only rows.
// grid (kMemoCap / 256, problem lanes): block (x, y) serves classes 256 x .. 256 x + 255 of the
// problems y, y + gridDim.y, ... of the batch, so the thresholds are staged once per block.
// `p` points at the batch's first problem; record (problem within the batch, slot) is written.
// Dynamic shared memory: the staged thresholds (thr_cap floats), then 256 records.
constexpr int kProbRec = kFastMaxProbRows + 128;  // problem-only rows, then the ProblemTerms
static_assert(sizeof(ProblemTerms) <= 128, "problem record");

__global__ void __launch_bounds__(256)
pair_table_kernel(ks_gpu_desc desc, const ks_problem* __restrict__ p, ks_problem p_value, int use_value, int n_prob,
                  const ks_candidate* __restrict__ c, FastView fv, MemoView memo, int thr_cap) {
  extern __shared__ __align__(16) float s_pthr[];  // thresholds of the per-pair features, then the records
  __shared__ ProblemTerms s_pt;
  __shared__ FeatQ s_fq[64];
  __shared__ float s_pf[64];
  const int tid = threadIdx.x;
  // the select kernel that follows may start its own set-up now (it waits for this grid to finish
  // before it reads the tables)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (blockIdx.x == 0 && tid == 0) g_fast_abort = 0;  // (also) precedes the select kernel
  int most = 0;
  for (int q = 0; q < kMemoCombos; ++q) most = max(most, memo.count[q]);
  // An item is (block of 256 classes, problem); the blocks of the grid deal the items among
  // themselves, so that the work is even whatever the number of classes. The item of class
  // block 0 also writes its problem's own record (problem-only rows and terms).
  const int class_blocks = most > 0 ? (most + 255) / 256 : 1;
  const int n_items = class_blocks * n_prob;
  if (static_cast<int>(blockIdx.x) >= n_items) return;
  const float* T = stage_thresholds(fv, 0, fv.thr_cand0, s_pthr, thr_cap);
  uint8_t* my_rec = reinterpret_cast<uint8_t*>(s_pthr + (thr_cap > 0 ? (thr_cap + 3) / 4 * 4 : 0)) +
                    static_cast<size_t>(tid) * fv.pair_rec;
  if (tid < 64) s_fq[tid] = fv.feat[tid];
  int max_thr = -1;  // the longest threshold list among the per-pair columns (found after the first barrier)
  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
    const int prob = item / class_blocks, j = (item % class_blocks) * 256 + tid;
    const bool first_block = item % class_blocks == 0;
    const ks_problem pr = use_value ? p_value : load_problem(p + prob);
    const int combo = (pr.dtype_ab & 3) * 4 + (pr.dtype_d & 3);
    const int n_classes = memo.count[combo];
    __syncthreads();  // the previous item's terms are no longer read (and the staging is complete)
    if (tid == 0) {
      problem_terms(pr, desc, s_pt);
      if (first_block) problem_columns(s_pt, [&](int col, float v) { s_pf[col] = v; });
    }
    __syncthreads();
    if (first_block) {
      // once per problem, for all its CTAs: the problem-only rows and the problem's terms
      uint8_t* out = const_cast<uint8_t*>(fv.prob_tab) + static_cast<size_t>(prob) * kProbRec;
      if (tid < KS_F && feat_class(tid) == 0) {
        const FeatQ& q = s_fq[tid];
        const int first = fv.n_pair_rows + fv.n_cand_rows;
        quantise(q, fv.thr + q.thr0, s_pf[tid], false,
                 [&](int row, uint8_t b) { out[KS_IDX(row - first, kFastMaxProbRows)] = b; });
      }
      if (tid < static_cast<int>(sizeof(ProblemTerms) / 4))
        reinterpret_cast<uint32_t*>(out + kFastMaxProbRows)[tid] = reinterpret_cast<const uint32_t*>(&s_pt)[tid];
    }
    if (j >= n_classes) continue;
    if (max_thr < 0) {
      max_thr = 0;
#pragma unroll
      for (int i = 0; i < kPairCols; ++i) max_thr = max(max_thr, static_cast<int>(s_fq[pair_col(i)].nthr));
    }
    const int slot = memo.dense[static_cast<size_t>(combo) * kMemoCap + j];
    const ks_candidate cand = load_candidate(c + memo.reps[static_cast<size_t>(combo) * kMemoCap + slot]);
    const long long b_eff = resources(s_pt, cand, desc).b_eff;
    float vals[kPairCols];
    pair_columns<true>(s_pt, cand, desc, b_eff, [&](int col, float v) { vals[pair_slot(col)] = v; });
    quantise_pair_columns(s_fq, T, vals, max_thr, [&](int row, uint8_t b) { my_rec[KS_IDX(row, fv.pair_rec)] = b; });
    // the record leaves as whole 16-byte words (it is a multiple of 16 bytes, and so is its place)
    uint4* dst = reinterpret_cast<uint4*>(static_cast<uint8_t*>(memo.tab) +
                                          (static_cast<size_t>(prob) * kMemoCap + slot) * fv.pair_rec);
    const uint4* src = reinterpret_cast<const uint4*>(my_rec);
    for (int q = 0; q < fv.pair_rec / 16; ++q) dst[q] = src[q];
  }
}

// ------------------------------------------------------------------------------------------
// single-problem call: the whole tile of every candidate block, once per call
// ------------------------------------------------------------------------------------------

// One thread per tile slot writes all rows of its candidate's tile column, in the layout phase A
// would produce, for the one problem of the call. The CTAs that share a candidate block in slice
// mode then copy the block's tile instead of each rebuilding it. Slots past the catalogue get the
// neutral byte. Also clears the abort flag (this kernel precedes the select kernel).
template <bool kPairRows>  // true: the per-pair rows; false: the candidate-only and problem-only rows
__device__ __forceinline__ void tile_one_rows(const ks_gpu_desc& desc, const ks_problem& p_value,
                                              const ks_candidate* __restrict__ c, int C, const FastView& fv,
                                              int NC, uint8_t* __restrict__ tiles, float* s_thr, int thr_cap) {
  __shared__ ProblemTerms s_pt;
  __shared__ FeatQ s_fq[64];
  const int tid = threadIdx.x;
  if (blockIdx.x == 0 && tid == 0) g_fast_abort = 0;
  // rows and thresholds are ordered per-pair, candidate-only, problem-only
  const int first = kPairRows ? 0 : fv.n_pair_rows;
  const int count = kPairRows ? fv.n_pair_rows : fv.n_rows - fv.n_pair_rows;
  const int t_first = kPairRows ? 0 : fv.thr_cand0;
  const int t_count = kPairRows ? fv.thr_cand0 : fv.n_thr - fv.thr_cand0;
  const float* T = stage_thresholds(fv, t_first, t_count, s_thr, thr_cap) - t_first;
  if (tid < 64) s_fq[tid] = fv.feat[tid];
  if (tid == 0) problem_terms(p_value, desc, s_pt);
  __syncthreads();
  const int slot = blockIdx.x * blockDim.x + tid;
  const int blk = slot / NC, in = slot % NC;
  uint8_t* my = tiles + static_cast<size_t>(blk) * fv.n_rows * NC + tile_byte(in, NC / 4);
  if (slot >= C) {
    for (int q = first; q < first + count; ++q) my[static_cast<size_t>(q) * NC] = 0x80;
    return;
  }
  const ks_candidate cand = load_candidate(c + slot);
  featurize_pair(s_pt, cand, desc, [&](int col, float v) {
    if (col >= KS_F || (feat_class(col) == 2) != kPairRows) return;
    const FeatQ& q = s_fq[col];
    quantise(q, T + q.thr0, v, false, [&](int row, uint8_t b) { my[static_cast<size_t>(KS_IDX(row, fv.n_rows)) * NC] = b; });
  });
}

// blockIdx.y picks the role, so that both halves of the work are in flight together
__global__ void __launch_bounds__(256)
tile_one_kernel(ks_gpu_desc desc, ks_problem p_value, const ks_candidate* __restrict__ c, int C, FastView fv,
                int NC, uint8_t* __restrict__ tiles, int thr_cap) {
  extern __shared__ float s_thr[];  // thresholds of this role's features
  if (blockIdx.y == 0) tile_one_rows<true>(desc, p_value, c, C, fv, NC, tiles, s_thr, thr_cap);
  else tile_one_rows<false>(desc, p_value, c, C, fv, NC, tiles, s_thr, thr_cap);
}

// ------------------------------------------------------------------------------------------
// scoring call: tiles from feature rows
// ------------------------------------------------------------------------------------------

// ks_score with a qualifying ensemble: one thread per tile word quantises all columns of the
// word's four feature rows into the tile layout of phase A and stores whole words, so that a
// warp's stores are full lines; the walk kernel then copies the tiles as in the single-problem
// call and writes the scores instead of ranking. A NaN goes right at every numeric split (x < t is
// false), like +inf: the last bin. Slots past the last row get the neutral byte. Also clears
// the abort flag. Launched with one thread per word of a row (NC / 4).
__global__ void __launch_bounds__(256)
tile_rows_kernel(const float* __restrict__ feat, int64_t rows, FastView fv, uint8_t* __restrict__ tiles,
                 int thr_cap) {
  extern __shared__ float s_thr[];  // thresholds of every feature
  __shared__ FeatQ s_fq[64];
  const int W = blockDim.x, NC = 4 * W;
  const int word = threadIdx.x;
  if (blockIdx.x == 0 && word == 0) g_fast_abort = 0;
  const float* T = stage_thresholds(fv, 0, fv.n_thr, s_thr, thr_cap);
  if (word < 64) s_fq[word] = fv.feat[word];
  __syncthreads();
  // byte b of the word is row 4 word + b of the block
  const int64_t base = static_cast<int64_t>(blockIdx.x) * NC;
  const float4* src[4];
  bool live[4];
#pragma unroll
  for (int b = 0; b < 4; ++b) {
    const int64_t slot = base + 4 * word + b;
    live[b] = slot < rows;
    src[b] = reinterpret_cast<const float4*>(feat + (live[b] ? slot : 0) * KS_F_PAD);
  }
  uint32_t* out = reinterpret_cast<uint32_t*>(tiles + static_cast<size_t>(blockIdx.x) * fv.n_rows * NC) + word;
#pragma unroll 2
  for (int q4 = 0; q4 < KS_F_PAD / 4; ++q4) {
    float v[4][4];
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const float4 t = __ldg(src[b] + q4);
      v[b][0] = t.x; v[b][1] = t.y; v[b][2] = t.z; v[b][3] = t.w;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int col = 4 * q4 + j;
      if (col >= KS_F) continue;
      const FeatQ& q = s_fq[col];
      int pos[4], code[4];
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const float x = v[b][j];
        pos[b] = !live[b] ? 0 : ((x != x) ? q.nthr : count_le(T + q.thr0, q.nthr, x));
        code[b] = live[b] ? __float2int_rz(x) : -1;
      }
      for (int s = 0; s < q.nslice; ++s) {
        uint32_t w = 0;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          int bin = pos[b] - kSlice * s;
          bin = bin < 0 ? 0 : (bin > kSlice ? kSlice : bin);
          w |= static_cast<uint32_t>(0x80 | bin) << (8 * b);
        }
        out[static_cast<size_t>(KS_IDX(q.row0 + s, fv.n_rows)) * W] = w;
      }
      for (int r = 0; r < q.nrank; ++r) {
        uint32_t w = 0;
#pragma unroll
        for (int b = 0; b < 4; ++b)
          w |= static_cast<uint32_t>(0x80 | ((code[b] >= 0 && code[b] < 4) ? q.rank[r][code[b]] : 0)) << (8 * b);
        out[static_cast<size_t>(KS_IDX(q.row0 + q.nslice + r, fv.n_rows)) * W] = w;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// phase A
// ------------------------------------------------------------------------------------------

// Sixteen rows of four neighbouring candidates: q[r] holds candidate r's bytes of rows row0 ..
// row0 + 15 (a 16-byte vector of its record). Byte r of a tile word is candidate r, so every
// group of four rows is a 4 x 4 byte transpose (eight byte permutes) and four word stores.
__device__ __forceinline__ void scatter_vectors(const uint4 (&q)[4], int row0, int n, unsigned char* word0, int NC) {
  const uint32_t w[4][4] = {{q[0].x, q[0].y, q[0].z, q[0].w},
                            {q[1].x, q[1].y, q[1].z, q[1].w},
                            {q[2].x, q[2].y, q[2].z, q[2].w},
                            {q[3].x, q[3].y, q[3].z, q[3].w}};
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    const int row = row0 + 4 * g;
    if (row >= n) break;
    const uint32_t lo_ab = __byte_perm(w[0][g], w[1][g], 0x5140u), lo_cd = __byte_perm(w[2][g], w[3][g], 0x5140u);
    const uint32_t hi_ab = __byte_perm(w[0][g], w[1][g], 0x7362u), hi_cd = __byte_perm(w[2][g], w[3][g], 0x7362u);
    const uint32_t out[4] = {__byte_perm(lo_ab, lo_cd, 0x5410u), __byte_perm(lo_ab, lo_cd, 0x7632u),
                             __byte_perm(hi_ab, hi_cd, 0x5410u), __byte_perm(hi_ab, hi_cd, 0x7632u)};
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (row + j < n) *reinterpret_cast<uint32_t*>(word0 + static_cast<size_t>(row + j) * NC) = out[j];
  }
}

// Fills the tile: candidate-only rows from the per-call table, problem-only rows from s_pbin,
// per-pair rows from the memo record of the candidate's class or computed here. Slots past the
// end of the segment get a neutral byte so that word-wise arithmetic on the tile never borrows
// across bytes. A thread serves the four candidates of one tile word (byte r of the word is
// candidate r): it fetches their records sixteen rows at a time and stores whole words; the
// THREADS / (NC / 4) threads that share a word deal the records' vectors among themselves.
template <int THREADS, int NC>
__device__ __noinline__ void fill_tile(const ks_gpu_desc& desc, const ProblemTerms& pt,
                                       const ks_candidate* __restrict__ c, const FastView& fv,
                                       const int64_t* __restrict__ seg_off, const int32_t* __restrict__ seg_idx,
                                       int C, int64_t lo, int64_t start, int64_t stop, const float* T,
                                       const FeatQ* s_fq, const uint8_t* s_pbin, unsigned char* tile, int prob,
                                       unsigned* s_cid, bool reuse) {
  constexpr int W = NC / 4, PARTS = THREADS / W;
  const int tid = threadIdx.x;
  const int combo = pt.dtype_ab * 4 + pt.dtype_d;
  // `reuse`: the tile still holds the candidate-only rows of these very candidates (the CTA's last
  // item was the same candidate block under the same element types), and s_cid their classes.
  // problem-only rows: one byte for the whole row
  {
    unsigned char* dst = tile + static_cast<size_t>(fv.n_pair_rows + fv.n_cand_rows) * NC;
    for (int i = tid; i < fv.n_prob_rows * (NC / 16); i += THREADS) {
      const uint32_t b = s_pbin[i / (NC / 16)] * 0x01010101u;
      reinterpret_cast<uint4*>(dst)[i] = make_uint4(b, b, b, b);
    }
  }
  const int word = tid % W, part = tid / W;
  unsigned char* word0 = tile + 4 * word;
  int ci[4];
  unsigned cid[4];
  bool lone = false;  // one of this word's candidates has no record of per-pair rows
  if (reuse) {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      ci[r] = start + 4 * word + r < stop ? 0 : -1;  // (the pool index itself is not needed again)
      cid[r] = s_cid[4 * word + r];
      lone |= ci[r] >= 0 && cid[r] == kNoClass;
    }
  } else {
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int64_t row = start + 4 * word + r;
      ci[r] = row < stop ? (seg_idx ? seg_idx[lo + row] : static_cast<int>(row)) : -1;
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      cid[r] = (ci[r] >= 0 && fv.pair_class) ? __ldg(fv.pair_class + static_cast<size_t>(combo) * C + ci[r]) : kNoClass;
      lone |= ci[r] >= 0 && cid[r] == kNoClass;
      if (s_cid && part == 0) s_cid[4 * word + r] = cid[r];
    }
  }
  const uint4 neutral = make_uint4(0x80808080u, 0x80808080u, 0x80808080u, 0x80808080u);
  const int cand_vecs = (fv.n_cand_rows + 15) / 16, pair_vecs = (fv.n_pair_rows + 15) / 16;
  const uint8_t* cand_rec[4];
  const uint8_t* pair_rec[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    cand_rec[r] = ci[r] >= 0 ? fv.cand_rows + (static_cast<size_t>(combo) * C + KS_IDX(ci[r], C)) * fv.cand_rec : nullptr;
    pair_rec[r] = cid[r] != kNoClass
                      ? fv.pair_tab + (static_cast<size_t>(prob) * kMemoCap + KS_IDX(cid[r], kMemoCap)) * fv.pair_rec
                      : nullptr;
  }
  // kBatch vectors of the four candidates are fetched before the first is stored, so that a thread
  // waits for the memory once per batch, not once per vector
  constexpr int kBatch = 1;
#pragma unroll 1
  for (int v0 = (reuse ? cand_vecs : 0) + part; v0 < cand_vecs + pair_vecs; v0 += kBatch * PARTS) {
    uint4 q[kBatch][4];
#pragma unroll
    for (int j = 0; j < kBatch; ++j) {
      const int v = v0 + j * PARTS;
      if (v >= cand_vecs + pair_vecs) break;
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const uint8_t* rec = v < cand_vecs ? cand_rec[r] : pair_rec[r];
        q[j][r] = rec ? __ldg(reinterpret_cast<const uint4*>(rec) + (v < cand_vecs ? v : v - cand_vecs)) : neutral;
      }
    }
#pragma unroll
    for (int j = 0; j < kBatch; ++j) {
      const int v = v0 + j * PARTS;
      if (v >= cand_vecs + pair_vecs) break;
      if (v < cand_vecs) scatter_vectors(q[j], 16 * v, fv.n_cand_rows, word0 + static_cast<size_t>(fv.n_pair_rows) * NC, NC);
      else scatter_vectors(q[j], 16 * (v - cand_vecs), fv.n_pair_rows, word0, NC);
    }
  }
  // candidates without a record (no memo in this call, or a class table that was full): their
  // per-pair columns are computed here, after the word stores that cover their bytes
  if (!__syncthreads_or(lone)) return;
  if (!lone) return;
#pragma unroll 1
  for (int r = part % 4; r < 4; r += (PARTS < 4 ? PARTS : 4)) {
    if (ci[r] < 0 || cid[r] != kNoClass) continue;
    unsigned char* my = word0 + r;
    const int64_t row = start + 4 * word + r;
    const ks_candidate cand = load_candidate(c + (seg_idx ? seg_idx[lo + row] : static_cast<int>(row)));
    pair_columns<true>(pt, cand, desc, resources(pt, cand, desc).b_eff, [&](int col, float v) {
      const FeatQ& q = s_fq[col];
      quantise(q, T + q.thr0, v, false, [&](int row, uint8_t b) { my[KS_IDX(row, fv.n_pair_rows) * NC] = b; });
    });
  }
}

// ------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------

// bytes of `a` where the top bit of the matching byte of `m` is set, else bytes of `b`
__device__ __forceinline__ uint32_t byte_select(uint32_t m, uint32_t a, uint32_t b) {
  const uint32_t f = __byte_perm(m, 0u, 0xBA98u);  // top bit of every byte replicated over the byte
  return (a & f) | (b & ~f);
}

// one path step of one walk: fetch the node, fetch the candidate's byte, move to the child:
// next = 2 a + k0 (+ 4 when the candidate goes right)
#ifndef KS_DEBUG_BOUNDS
__device__ __forceinline__ uint32_t path_step(uint32_t a, uint32_t cb_r, uint32_t k0, uint32_t, uint32_t, uint32_t) {
  uint32_t nx;
  asm volatile(
      "{\n"
      " .reg .u32 n, x, m;\n"
      " .reg .pred p;\n"
      " ld.shared.u32 n, [%1];\n"
      " shr.u32 m, n, 8;\n"
      " add.u32 m, m, %2;\n"
      " ld.shared.u8 x, [m];\n"
      " and.b32 n, n, 255;\n"
      " setp.gt.u32 p, x, n;\n"
      " mad.lo.u32 %0, %1, 2, %3;\n"
      " @p add.u32 %0, %0, 4;\n"
      "}\n"
      : "=r"(nx)
      : "r"(a), "r"(cb_r), "r"(k0));
  return nx;
}
#else
// checked build: the node address must lie in the chunk buffer, the byte address in the tile
__device__ __forceinline__ uint32_t path_step(uint32_t a, uint32_t cb_r, uint32_t k0, uint32_t buf,
                                              uint32_t tile0, uint32_t tile_bytes) {
  a = buf + static_cast<uint32_t>(KS_IDX((a - buf) >> 2, 2 * kBufBytes / 4)) * 4u;
  const uint32_t n = lds_u32(a);
  uint32_t m = (n >> 8) + cb_r;
  m = tile0 + static_cast<uint32_t>(KS_IDX(m - tile0, tile_bytes));
  uint32_t x;
  asm volatile("ld.shared.u8 %0, [%1];" : "=r"(x) : "r"(m));
  return 2u * a + k0 + (x > (n & 255u) ? 4u : 0u);
}
#endif

// L levels evaluated word-wise; NP path levels unrolled (-1: runtime count); kCompact: the top
// levels' constants travel as one 32-bit word per node (row offset << 8 | j + 1) instead of a
// (row offset, replicated j + 1) pair, so that twice as many trees keep their word-wise levels.
// THREADS threads rank NC candidates: NC / 4 words times THREADS / (NC / 4) tree groups.
// kFloor (measurement only): the walk without its chunk rings. Every tree group's first kNBuf
// chunks are copied once and stay resident; the group walks them again and again (sl.repeat
// times as many chunk walks as it has chunks), never waits, releases or refills, so the time per
// pass is that of the gather and instruction stream of the walk alone, at the occupancy and tile
// size of the real kernel.
template <int L, int NP, bool kCompact, int THREADS, int NC, bool kFloor = false>
__global__ void __launch_bounds__(THREADS, THREADS <= 256 ? 2 : 1)
select_fast_kernel(ks_gpu_desc desc, const ks_problem* __restrict__ p, ks_problem p_value, int use_value,
                   const ks_candidate* __restrict__ c, int P, int C, int nblk, int rows_per_cta,
                   const int64_t* __restrict__ seg_off, const int32_t* __restrict__ seg_idx, FastView fv,
                   int k, unsigned long long* __restrict__ partial, int* __restrict__ status,
                   SliceArgs sl, int n_items, const __grid_constant__ FastTopParams top) {
  constexpr int W = NC / 4;        // words per tile row = lane slots
  constexpr int G = THREADS / W;   // tree groups
  constexpr int RG = ring_count(G);  // chunk rings
  constexpr int GPR = G / RG;        // groups that share a ring (and split the trees of its chunks)
  static_assert(THREADS % W == 0 && W % 32 == 0 && G >= 1, "tile geometry");
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ ProblemTerms s_pt;
  __shared__ unsigned long long s_warp[THREADS / 32 * KS_MAX_K];
  __shared__ unsigned long long s_list[KS_MAX_K];
  __shared__ __align__(8) unsigned long long s_bar[kNBuf * RG];  // [ring][buffer]
  __shared__ FeatQ s_fq[64];
  __shared__ uint8_t s_pbin[kFastMaxProbRows];
  __shared__ float s_pfeat[64];
  __shared__ int s_fail, s_last, s_done[kNBuf * RG], s_abort, s_pending[kNBuf * RG];
  // the classes of the candidates whose candidate-only rows the tile holds (one-CTA forms only:
  // there a CTA serves one candidate block for many problems in a row, see below)
  __shared__ unsigned s_cid[THREADS > 256 && NC == 1024 ? NC : 1];

  const int tid = threadIdx.x;
  const int kOffTile = kNBuf * RG * fv.buf_bytes;  // every ring has kNBuf buffers
  const int S = sl.n_slices;
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bar0 = smem_u32(&s_bar[0]);  // barrier of buffer b: bar0 + 8 b
  const bool tiles_given = sl.tiles != nullptr;  // the tiles were built in front: no feature work here
  if (tid == 0) {
    for (int b = 0; b < kNBuf * RG; ++b) mbar_init(bar0 + 8u * b, 1);
    s_fail = 0;
    for (int b = 0; b < kNBuf * RG; ++b) s_done[b] = s_pending[b] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < 64) s_fq[tid] = fv.feat[tid];
  __syncthreads();
  // everything above is independent of the kernel in front (the per-problem tables): when this
  // grid was launched as its programmatic dependent, wait for that grid here
  asm volatile("griddepcontrol.wait;" ::: "memory");
  uint32_t phases = 0;  // bit b: parity of buffer b's barrier
  const int word = tid % W, grp = tid / W;
  volatile int* v_fail = &s_fail;

  // An item is one (problem, candidate block, tree slice). The batch form of a geometry that holds one CTA per SM is
  // launched with one CTA per SM, so that a CTA's set-up and the gap between two CTAs are paid
  // once, not per item; everything else (two CTAs per SM, which hide each other's gaps; tree
  // slices and scoring, which leave an item early) is launched with one CTA per item.
  // A CTA (of the 1,024-candidate forms) that serves many items of a dense batch takes a run of
  // consecutive items in the order (candidate block, problem): successive items then are the same
  // candidates for another problem, and while the element types stay the same their
  // candidate-only rows (and classes) stay in place. (The 512-candidate form serves segmented
  // batches in the benchmark; compiled with this path it ran them 2 % slower, so it keeps the
  // plain order.)
  const int grid = static_cast<int>(gridDim.x), cta = static_cast<int>(blockIdx.x);
  const bool block_major = NC == 1024 && grid < n_items && !seg_off && S == 1;
  const int per_cta = (n_items + grid - 1) / grid;
  const int first_item = block_major ? cta * per_cta : cta, item_step = block_major ? 1 : grid;
  const int last_item = block_major ? (first_item + per_cta < n_items ? first_item + per_cta : n_items) : n_items;
  int held_chunk = -1, held_combo = -1;  // what the tile's candidate-only rows belong to
#pragma unroll 1
  for (int item = first_item; item < last_item; item += item_step) {
  const int prob = block_major ? item % P : item / (nblk * S);
  const int chunk = block_major ? item / P : (item / S) % nblk, slice = item % S;
  // rows of this problem: lo = where its scores sit in per-row arrays; lo_idx = where its pool
  // indices start in seg_idx (per-problem segments, or - without offsets - one ranking order of
  // the whole catalogue shared by every problem)
  int64_t lo, len, lo_idx;
  if (seg_off) {
    lo = lo_idx = seg_off[prob];
    len = seg_off[prob + 1] - lo;
  } else {
    lo = static_cast<int64_t>(prob) * C;
    lo_idx = 0;
    len = C;
  }
  // chunks of the ensemble this CTA walks
  const int ch_begin = static_cast<int>(static_cast<int64_t>(fv.n_chunks) * slice / S);
  const int ch_end = static_cast<int>(static_cast<int64_t>(fv.n_chunks) * (slice + 1) / S);
  __syncthreads();  // the item before this one is finished with the shared state
  if (tid == 0) {
    if (!tiles_given && !fv.prob_tab) {
      problem_terms(use_value ? p_value : load_problem(p + prob), desc, s_pt);
      problem_columns(s_pt, [&](int col, float v) { s_pfeat[col] = v; });
    }
    s_abort = *reinterpret_cast<volatile int*>(&g_fast_abort);
  }
  if (tid < KS_MAX_K) s_list[tid] = 0ull;
  if (!tiles_given && fv.prob_tab) {
    const uint8_t* rec = fv.prob_tab + static_cast<size_t>(prob) * kProbRec;
    for (int i = tid; i < fv.n_prob_rows; i += THREADS) s_pbin[i] = __ldcg(rec + i);
    if (tid < static_cast<int>(sizeof(ProblemTerms) / 4))
      reinterpret_cast<uint32_t*>(&s_pt)[tid] = __ldcg(reinterpret_cast<const uint32_t*>(rec + kFastMaxProbRows) + tid);
  }
  __syncthreads();
  if (s_abort) {  // a wait ran out in an earlier CTA of this launch: the call fails, leave at once
    if (tid < k && slice == 0 && partial) partial[(static_cast<size_t>(prob) * nblk + chunk) * k + tid] = 0ull;
    return;
  }
  if (!tiles_given && !fv.prob_tab && tid < KS_F && feat_class(tid) == 0) {
    const int first = fv.n_pair_rows + fv.n_cand_rows;
    const FeatQ& q = s_fq[tid];
    quantise(q, fv.thr + q.thr0, s_pfeat[tid], false,
             [&](int row, uint8_t b) { s_pbin[KS_IDX(row - first, kFastMaxProbRows)] = b; });
  }

  for (int64_t start = static_cast<int64_t>(chunk) * rows_per_cta; start < len;
       start += static_cast<int64_t>(nblk) * rows_per_cta) {
    const int64_t stop = (start + rows_per_cta < len) ? start + rows_per_cta : len;
    // ---- phase A ---------------------------------------------------------------------------------
    __syncthreads();
    if (sl.tiles) {
      // single-problem call: the block's tile was built once for all the CTAs that share it
      const uint4* src = reinterpret_cast<const uint4*>(sl.tiles + static_cast<size_t>(chunk) * fv.n_rows * NC);
      uint4* dst = reinterpret_cast<uint4*>(smem + kOffTile);
      for (int i = tid; i < fv.n_rows * (NC / 16); i += THREADS) dst[i] = __ldcg(src + i);
    } else {
      // thresholds of the per-pair features: into the idle chunk buffers when they fit
      const float* T = stage_thresholds(fv, 0, fv.thr_cand0, reinterpret_cast<float*>(smem + kOffBuf0),
                                        fv.pair_class ? 0 : kNBuf * RG * fv.buf_bytes / 4);
      __syncthreads();
      const int combo = s_pt.dtype_ab * 4 + s_pt.dtype_d;
      const bool reuse = THREADS > 256 && block_major && fv.pair_class && chunk == held_chunk && combo == held_combo;
      fill_tile<THREADS, NC>(desc, s_pt, c, fv, seg_off, seg_idx, C, lo_idx, start, stop, T, s_fq, s_pbin,
                             smem + kOffTile, prob, THREADS > 256 && block_major ? s_cid : nullptr, reuse);
      held_chunk = chunk;
      held_combo = combo;
    }
    __syncthreads();  // tile complete; the threshold table is no longer needed

    // ---- phase B ---------------------------------------------------------------------------------
    if (tid == 0) {
      fence_async_proxy();
      // ring g takes the chunks ch_begin + g, ch_begin + g + RG, ... through its own buffers
      for (int g = 0; g < RG; ++g)
        for (int b = 0; b < kNBuf && ch_begin + g + b * RG < ch_end; ++b) {
          const int rb = g * kNBuf + b;
          // test hook: a barrier armed for more bytes than its copy brings never completes
          mbar_expect_tx(bar0 + 8u * rb, fv.chunk_bytes + (fv.starve ? 16 : 0));
          bulk_copy_g2s(sbase + kOffBuf0 + rb * fv.buf_bytes,
                        reinterpret_cast<const char*>(fv.chunks) + static_cast<size_t>(ch_begin + g + b * RG) * fv.chunk_bytes,
                        fv.chunk_bytes, bar0 + 8u * rb);
          s_pending[rb] = 1;
        }
    }
    float score[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    const uint32_t cb = sbase + kOffTile + word * 4;
    const int tpc = fv.tpc, grp_trees = (tpc + GPR - 1) / GPR;
    const int np = NP >= 0 ? NP : fv.depth - L;
    constexpr int kTop = (1 << L) - 1;
    const int ring = grp / GPR;
    // the groups of a ring share out the trees of its chunks
    const int t_first = (grp % GPR) * grp_trees;
    const int t_count = t_first + grp_trees <= tpc ? grp_trees : (tpc > t_first ? tpc - t_first : 0);
#ifdef KS_DEBUG_BOUNDS
    const uint32_t tile0 = sbase + kOffTile, tile_bytes = static_cast<uint32_t>(fv.n_rows) * NC;
#else
    constexpr uint32_t tile0 = 0, tile_bytes = 0;
#endif
    // this ring's chunks: n_mine of them; the floor form walks its first kNBuf again and again
    const int n_mine = ch_end - ch_begin > ring ? (ch_end - ch_begin - ring + RG - 1) / RG : 0;
    const int n_walks = kFloor ? n_mine * sl.repeat : n_mine;
#pragma unroll 1
    for (int it = 0; it < n_walks; ++it) {
      const int b = it % kNBuf, rb = ring * kNBuf + b;
      const int ch = ch_begin + ring + (kFloor ? b : it) * RG;  // the chunk whose trees are walked
      const uint32_t bar = bar0 + 8u * rb;
      const uint32_t par = (phases >> b) & 1u;
      // A wait that runs out ends the walk of this CTA: the buffer was never filled, so it is not
      // read; the call fails, and the CTAs that start later leave at once.
      if (!kFloor || it < kNBuf) {
        if (*v_fail || !mbar_wait_bounded(bar, par, fv.wait_limit, v_fail)) {
          if (!*v_fail) {
            s_fail = 1;
            atomicExch(&g_fast_abort, 1);
            if (status) atomicExch(status, KS_ERR_TIMEOUT);
          }
          break;
        }
        phases ^= 1u << b;
      }
      const uint32_t buf = sbase + kOffBuf0 + rb * fv.buf_bytes;
      // With A_l the shared address of a walk's node at level l, A_{l+1} = 2 A_l + (4 tpc - buf)
      // + 4 bit for every level, and after the last level A points at the walk's leaf.
      const uint32_t k0 = 4u * tpc - buf;  // modulo 2^32, like the additions it enters
      const uint32_t lvlL = buf + 4u * tpc * kTop;  // first node of level L
#pragma unroll 4
      for (int tt = 0; tt < t_count; ++tt) {
        const int t = t_first + tt;
        uint32_t a[4];
        if (L == 0) {
#pragma unroll
          for (int r = 0; r < 4; ++r) a[r] = buf + 4u * t;
        } else {
          // Word-wise evaluation of the top L levels for the four candidates of this word.
          // A tile byte is 0x80 | bin and a node constant (j + 1) in every byte, so byte r of
          // d[n] keeps its top bit iff candidate r goes right at node n; no byte borrows.
          uint32_t d[kTop > 0 ? kTop : 1];
          if (kCompact) {
            const uint32_t* tw = reinterpret_cast<const uint32_t*>(top.w) +
                                 static_cast<size_t>(KS_IDX(ch * tpc + t, 2 * kFastTopPairs / (kTop > 0 ? kTop : 1))) * kTop;
#pragma unroll
            for (int n = 0; n < kTop; ++n) {
              const uint32_t v = tw[n];
              d[n] = lds_u32(cb + static_cast<uint32_t>(KS_IDX(v >> 8, fv.n_rows * NC))) - __byte_perm(v, 0u, 0u);
            }
          } else {
            const uint2* tw = top.w + static_cast<size_t>(KS_IDX(ch * tpc + t, kFastTopPairs / (kTop > 0 ? kTop : 1))) * kTop;
#pragma unroll
            for (int n = 0; n < kTop; ++n)
              d[n] = lds_u32(cb + static_cast<uint32_t>(KS_IDX(tw[n].x, fv.n_rows * NC))) - tw[n].y;
          }
          uint32_t x = d[0] & 0x80808080u;  // path bits: level 0 in bit 7 of each byte, ...
          if (L >= 2) {
            const uint32_t s1 = byte_select(d[0], d[2], d[1]);
            x |= (s1 >> 1) & 0x40404040u;
            if (L >= 3) {
              const uint32_t sa = byte_select(s1, d[4], d[3]);
              const uint32_t sb = byte_select(s1, d[6], d[5]);
              const uint32_t s2 = byte_select(d[0], sb, sa);
              x |= (s2 >> 2) & 0x20202020u;
            }
          }
          // byte r of x holds candidate r's node index at level L in its top L bits (the rest
          // is zero), so x >> (6 - L) holds 4 * index in every byte
          const uint32_t y = x >> (6 - L);
          const uint32_t tbase = lvlL + (static_cast<uint32_t>(t) << (L + 2));
#pragma unroll
          for (int r = 0; r < 4; ++r) a[r] = tbase + __byte_perm(y, 0u, 0x4440u + r);
        }
        if (NP >= 0) {
#pragma unroll
          for (int l = 0; l < (NP >= 0 ? NP : 0); ++l)
#pragma unroll
            for (int r = 0; r < 4; ++r) a[r] = path_step(a[r], cb + r, k0, buf, tile0, tile_bytes);
        } else {
#pragma unroll 1
          for (int l = 0; l < np; ++l)
#pragma unroll
            for (int r = 0; r < 4; ++r) a[r] = path_step(a[r], cb + r, k0, buf, tile0, tile_bytes);
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
#ifdef KS_DEBUG_BOUNDS
          a[r] = buf + 4u * static_cast<uint32_t>(KS_IDX((a[r] - buf) >> 2, fv.buf_bytes / 4));
#endif
          score[r] += lds_f32(a[r]);
        }
      }
      // Release the buffer without a block-wide barrier: every warp of the group counts itself
      // out, and the last one to leave refills the buffer (nobody waits; warps may run a chunk ahead).
      __syncwarp();
      if (!kFloor && (tid & 31) == 0) {
        if (atomicAdd(&s_done[rb], 1) == THREADS / 32 / RG - 1) {
          s_done[rb] = 0;
          s_pending[rb] = 0;
          if (ch + kNBuf * RG < ch_end && !*v_fail) {
            fence_async_proxy();
            mbar_expect_tx(bar, fv.chunk_bytes + (fv.starve ? 16 : 0));
            bulk_copy_g2s(buf, reinterpret_cast<const char*>(fv.chunks) +
                                   static_cast<size_t>(KS_IDX(ch + kNBuf * RG, fv.n_chunks)) * fv.chunk_bytes,
                          fv.chunk_bytes, bar);
            s_pending[rb] = 1;
          }
        }
      }
    }
    __syncthreads();  // all walks are done: the buffers are free
    if (kFloor && tid < kNBuf * RG && !*v_fail) s_pending[tid] = 0;  // copied once, landed, never refilled
    if (*v_fail) {
      // The call has failed. Before this CTA gives its shared memory back, give the copies that
      // may still be in flight the time to land (bounded again); the test hook's copies land in
      // full although their barriers never complete, so there a short pause stands in for it.
      if (word == 0 && grp % GPR == 0) {  // one thread per ring, for its ring's buffers (it knows their parities)
        for (int b = 0; b < kNBuf; ++b) {
          if (!s_pending[ring * kNBuf + b]) continue;
          if (fv.starve) {
            for (int i = 0; i < 64; ++i) __nanosleep(kSleepNs);
          } else {
            mbar_wait_bounded(bar0 + 8u * (ring * kNBuf + b), (phases >> b) & 1u, fv.wait_limit, &s_abort /* stays 0 */);
          }
        }
      }
      __syncthreads();
      if (tid < k && slice == 0 && partial) partial[(static_cast<size_t>(prob) * nblk + chunk) * k + tid] = 0ull;
      return;
    }

    // ---- phase C ---------------------------------------------------------------------------------
    float* s_part = reinterpret_cast<float*>(smem + kOffBuf0);  // [G - 1][4][W], buffers are idle now
    if (grp > 0) {
#pragma unroll
      for (int r = 0; r < 4; ++r) s_part[((grp - 1) * 4 + r) * W + word] = score[r];
    }
    __syncthreads();
    // this thread's sum over the groups, in a fixed order
    float total[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      total[r] = score[r];
      if (grp == 0)
        for (int g = 1; g < G; ++g) total[r] += s_part[((g - 1) * 4 + r) * W + word];
    }
    if (sl.score_out) {
      // scoring call: the scores are the result (same order of additions as the ranking path)
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int64_t row = start + 4 * word + r;
        if (grp == 0 && row < stop) sl.score_out[lo + row] = (fv.base + total[r]) + 0.0f;
      }
      continue;
    }
    if (S > 1) {
      // slice mode: publish this CTA's partial scores, let the last arrival finish the block
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int64_t row = start + 4 * word + r;
        if (grp == 0 && row < stop) __stcg(sl.scores + static_cast<size_t>(slice) * sl.pairs + lo + row, total[r]);
      }
      __threadfence();
      __syncthreads();
      if (tid == 0) {
        int* cnt = sl.counters + static_cast<size_t>(prob) * nblk + chunk;
        s_last = atomicAdd(cnt, 1) == S - 1;
        if (s_last) *cnt = 0;  // nobody else touches this counter again in this launch
      }
      __syncthreads();
      if (!s_last) return;
      __threadfence();
    }
    unsigned long long keys[5];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      keys[r] = 0ull;
      // byte r of word `word` is row 4 word + r of the block
      const int64_t row = start + 4 * word + r;
      if (grp == 0 && row < stop) {
        float s;
        if (S > 1) {
          s = fv.base;
          for (int q = 0; q < S; ++q) s += __ldcg(sl.scores + static_cast<size_t>(q) * sl.pairs + lo + row);
        } else {
          s = fv.base + total[r];
        }
        keys[r] = make_key(s + 0.0f, seg_idx ? seg_idx[lo_idx + row] : static_cast<int>(row));
      }
    }
    keys[4] = tid < k ? s_list[tid] : 0ull;
    __syncthreads();
    block_topk<5>(keys, k, s_warp, s_list);
  }
  if (sl.score_out) return;
  if (tid < k)
    partial[KS_IDX((static_cast<size_t>(prob) * nblk + chunk) * k + tid, static_cast<size_t>(P) * nblk * k)] = s_list[tid];
  if (S > 1 && sl.out_idx) {
    // single-problem form: the last block to finish merges the per-block lists
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = atomicAdd(sl.counters + nblk, 1) == nblk - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // the whole CTA ranks the nblk * k keys (each key is read once)
    const int n_keys = nblk * k;
    __syncthreads();
    if (tid < KS_MAX_K) s_list[tid] = 0ull;
    for (int base = 0; base < n_keys; base += 2 * THREADS) {
      unsigned long long keys[3];
      keys[0] = base + tid < n_keys ? __ldcg(partial + base + tid) : 0ull;
      keys[1] = base + THREADS + tid < n_keys ? __ldcg(partial + base + THREADS + tid) : 0ull;
      __syncthreads();
      keys[2] = tid < k ? s_list[tid] : 0ull;
      __syncthreads();
      block_topk<3>(keys, k, s_warp, s_list);
    }
    if (tid < k) {
      sl.out_idx[tid] = key_index(s_list[tid]);
      sl.out_score[tid] = key_score(s_list[tid]);
      __threadfence_system();
    }
    __syncthreads();
    if (tid == 0) {
      sl.counters[nblk] = 0;
      if (sl.out_seq) {  // the results are in place: tell the host, which polls this word
        __threadfence_system();
        *reinterpret_cast<volatile int*>(sl.out_seq) = sl.seq;
      }
    }
  }
  }  // items
}

}  // namespace

// ------------------------------------------------------------------------------------------
// host: repack
// ------------------------------------------------------------------------------------------

// The orderings of L levels used by rank rows (lowest rank first).
static const int* partition_perm(int L, int q) {
  static const int p2[1][4] = {{0, 1, 0, 0}};
  static const int p3[2][4] = {{0, 1, 2, 0}, {0, 2, 1, 0}};
  static const int p4[3][4] = {{0, 1, 2, 3}, {1, 3, 0, 2}, {1, 2, 0, 3}};
  return L == 2 ? p2[q] : (L == 3 ? p3[q] : p4[q]);
}
// How a membership mask is tested: levels of rank >= cut in ordering `perm` go right, or, with
// `swap`, go left (the mask is the complement of that upper set).
struct PartitionCode {
  int perm, cut;
  bool swap;
};
static std::vector<PartitionCode> partition_codes(int L) {
  const int n_perm = L == 2 ? 1 : (L == 3 ? 2 : 3);
  const uint32_t full = (1u << L) - 1;
  std::vector<PartitionCode> code(full + 1, PartitionCode{-1, 0, false});
  for (int q = 0; q < n_perm; ++q)
    for (int c = 1; c < L; ++c) {
      uint32_t up = 0;
      for (int r = c; r < L; ++r) up |= 1u << partition_perm(L, q)[r];
      if (code[up].perm < 0) code[up] = PartitionCode{q, c, false};
      if (code[full ^ up].perm < 0) code[full ^ up] = PartitionCode{q, c, true};
    }
  return code;
}

// Tile geometry by the number of rows: the [row][candidate] tile and the two chunk buffers have to
// fit the shared memory of one SM (228 KiB, 1 KiB of it reserved per CTA; a CTA's own limit is
// 227 KiB including its static part). What was measured to matter on one ensemble: (i) four trees
// or more per thread and chunk, which the compiler interleaves (13 %); (ii) up to 128 registers
// per thread - the 64-register forms (two CTAs of 512 threads) ran 54 to 63 ms on the same
// ensemble depending on how unrelated code around the loop happened to be compiled, and one CTA
// of 512 threads gained 15 % from the larger budget; (iii) two CTAs per SM, so that one CTA's
// tile fill and ranking overlap the other's walk, when the tile leaves room for them; sixteen
// walking warps per SM saturate the walk, eight do not. Hence, in order of preference: two CTAs
// of 256 threads x 1,024 candidates (eight trees per thread and chunk; up to 74 rows); one CTA of
// 512 threads x 1,024 candidates with 32 KB chunk buffers (eight trees per thread and chunk; up
// to 156 rows); two CTAs of 256 threads x 512 candidates; one CTA of 512 threads x 1,024
// candidates with 16 KB buffers (up to 188 rows) or x 512 candidates (up to 376 rows). Every CTA
// streams the whole ensemble, so a halved block doubles that traffic (two CTAs of 256 threads x
// 256 candidates measured slower than one CTA of 512 x 512; two CTAs of 128 x 512 and one CTA of
// 256 x 1,024 have too few warps). More rows than 376: the general kernel.
// KS_FAST_GEOMETRY="threads,candidates,buffer KiB" overrides the choice (a tuning aid; a geometry
// that does not fit is refused).
struct Geometry {
  int threads, cands, buf_bytes, ctas_per_sm;
};
static size_t geometry_smem(const Geometry& g, int n_rows) {
  // static shared memory of the kernel, with slack (the one-CTA forms keep a class per candidate)
  const size_t stat = 2560 + static_cast<size_t>(g.threads) / 32 * KS_MAX_K * 8 + 256 + (g.threads > 256 && g.cands == 1024 ? 4 * g.cands : 0);
  return static_cast<size_t>(kNBuf) * g.buf_bytes + static_cast<size_t>(n_rows) * g.cands + stat;
}
static bool geometry_fits(const Geometry& g, int n_rows) {
  const size_t per_cta = geometry_smem(g, n_rows);
  if (per_cta > 227 * 1024) return false;
  return g.ctas_per_sm * (per_cta + 1024) <= 228 * 1024;
}
static bool geometry_known(int t, int c) {
  return (t == 512 && c == 1024) || (t == 256 && c == 512) || (t == 512 && c == 512) || (t == 256 && c == 1024);
}
static bool pick_geometry(int n_rows, Geometry* out) {
  if (const char* env = std::getenv("KS_FAST_GEOMETRY")) {
    int t = 0, c = 0, kb = 0;
    if (std::sscanf(env, "%d,%d,%d", &t, &c, &kb) == 3 && geometry_known(t, c) && kb >= 8 && kb <= 64) {
      Geometry g{t, c, kb * 1024, 2};
      if (!geometry_fits(g, n_rows)) g.ctas_per_sm = 1;
      if (geometry_fits(g, n_rows)) {
        *out = g;
        return true;
      }
    }
  }
  const Geometry order[] = {{256, 1024, kBufBytes, 2},     {512, 1024, 2 * kBufBytes, 1}, {256, 512, kBufBytes, 2},
                            {512, 1024, kBufBytes, 1},     {512, 512, 2 * kBufBytes, 1},  {512, 512, kBufBytes, 1}};
  for (const Geometry& g : order)
    if (geometry_fits(g, n_rows)) {
      *out = g;
      return true;
    }
  return false;
}

cudaError_t build_fast_gbdt(GbdtModel& m, int n_trees, const int64_t* off, const ks_node_host* nodes) {
  m.fast = false;
  if (n_trees < 1 || m.max_depth < 1 || m.max_depth > kFastMaxDepth) return cudaSuccess;
  const int D = m.max_depth;
  // distinct thresholds per feature, sliced into rows of at most 127
  std::vector<std::vector<float>> thr(KS_F);
  // Partition splits: "level in S goes right" becomes a bin comparison on a rank row. A rank row
  // orders the field's levels by one of a few fixed permutations; S (or its complement, with the
  // node's children exchanged) is then the set of levels of rank >= c for some c, i.e. the
  // ordinary test "bin <= c - 1 goes left". The permutations below reach every proper subset of
  // 2, 3 and 4 levels up to complement.
  std::vector<std::vector<PartitionCode>> part(KS_F);  // per feature: code of every mask
  bool perm_used[KS_F][3] = {};
  for (int64_t i = 0; i < off[n_trees]; ++i) {
    const ks_node_host& nd = nodes[i];
    if (nd.feat == 0xFFFF) continue;
    if (nd.kind == KS_NODE_PARTITION) {
      const int L = categorical_levels(nd.feat);
      if (L == 0) return cudaSuccess;
      if (part[nd.feat].empty()) part[nd.feat] = partition_codes(L);
      uint32_t mask;
      std::memcpy(&mask, &nd.thr_or_leaf, 4);
      if (mask == 0 || mask >= (1u << L)) return cudaSuccess;
      if (mask != (1u << L) - 1) perm_used[nd.feat][part[nd.feat][mask].perm] = true;
    } else {
      thr[nd.feat].push_back(nd.thr_or_leaf);
    }
  }
  FeatQ fq[64];
  std::memset(fq, 0, sizeof(fq));
  int rank_row[KS_F][3];  // row offset (within the feature's rows) of each permutation in use
  int n_rows = 0, n_class[3] = {0, 0, 0}, thr_class[3] = {0, 0, 0};
  for (int f = 0; f < KS_F; ++f) {
    auto& v = thr[f];
    std::sort(v.begin(), v.end());
    v.erase(std::unique(v.begin(), v.end()), v.end());
    if (v.size() > 65000) return cudaSuccess;
    const int n_slices = static_cast<int>((v.size() + kSlice - 1) / kSlice);
    int cnt = n_slices, n_rank = 0;
    for (int q = 0; q < 3; ++q) {
      rank_row[f][q] = perm_used[f][q] ? cnt++ : -1;
      if (perm_used[f][q]) {
        const int L = categorical_levels(f);
        for (int r = 0; r < L; ++r) fq[f].rank[n_rank][partition_perm(L, q)[r]] = static_cast<uint8_t>(r);
        ++n_rank;
      }
    }
    fq[f].nthr = static_cast<uint16_t>(v.size());
    fq[f].nslice = static_cast<uint16_t>(n_slices);
    fq[f].nrank = static_cast<uint16_t>(n_rank);
    n_class[feat_class(f)] += cnt;
    thr_class[feat_class(f)] += static_cast<int>(v.size());
    n_rows += cnt;
  }
  Geometry geom{};
  if (n_rows == 0 || !pick_geometry(n_rows, &geom)) return cudaSuccess;  // generic path
  if (n_class[0] > kFastMaxProbRows || n_class[1] > kFastMaxCandRec) return cudaSuccess;
  const int NC = geom.cands, threads = geom.threads;
  // rows and thresholds ordered: per-pair, candidate-only, problem-only features
  std::vector<float> table;
  int next = 0;
  for (int cls : {2, 1, 0}) {
    for (int f = 0; f < KS_F; ++f) {
      if (feat_class(f) != cls) continue;
      fq[f].row0 = static_cast<uint16_t>(next);
      fq[f].thr0 = static_cast<uint32_t>(table.size());
      table.insert(table.end(), thr[f].begin(), thr[f].end());
      next += fq[f].nslice + fq[f].nrank;
    }
  }
  if (table.empty()) table.push_back(0.0f);
  const int G = threads / (NC / 4);
  const int per_tree_words = (2 << D) - 1;
  // A chunk is what one ring's buffer holds (the geometry's buffer size is shared out among the
  // rings); ring r takes the chunks r, r + rings, ..., and the groups of a ring split a chunk's trees.
  const int rings = ring_count(G), gpr = G / rings;
  const int group_buf = geom.buf_bytes / rings / 16 * 16;
  int tpc = group_buf / (per_tree_words * 4) / gpr * gpr;
  if (tpc < gpr) return cudaSuccess;
  if (tpc > (n_trees + G - 1) / G * gpr) tpc = (n_trees + G - 1) / G * gpr;  // a small ensemble: one short chunk per ring
  const int n_chunks = (n_trees + tpc - 1) / tpc;
  const int chunk_words = (tpc * per_tree_words + 3) / 4 * 4;  // bulk copies move multiples of 16 bytes
  if (chunk_words * 4 > group_buf) return cudaSuccess;
  int L = D < 3 ? D : 3;  // levels whose nodes travel as kernel-parameter constants
  while (L > 0 && static_cast<int64_t>(n_chunks) * tpc * ((1 << L) - 1) > kFastTopPairs) --L;
  // three levels in the compact form (one word per node) when the pair form would leave fewer
  bool compact = false;
  if (L < 3 && D >= 3 && static_cast<int64_t>(n_chunks) * tpc * 7 <= 2 * kFastTopPairs) {
    L = 3;
    compact = true;
  }
  const int n_top = (1 << L) - 1;
  std::vector<uint32_t> chunks(static_cast<size_t>(n_chunks) * chunk_words);
  FastTopParams* top = new (std::nothrow) FastTopParams();
  if (!top) return cudaErrorMemoryAllocation;
  const uint32_t always_left = 0xFFu;  // row 0, threshold 127: no byte (0x80 | bin) exceeds 0xFF
  for (int ch = 0; ch < n_chunks; ++ch) {
    uint32_t* base = chunks.data() + static_cast<size_t>(ch) * chunk_words;
    float* leaves = reinterpret_cast<float*>(base + tpc * ((1 << D) - 1));
    for (int tt = 0; tt < tpc; ++tt) {
      const int t = ch * tpc + tt;
      std::vector<int> src(1, t < n_trees ? 0 : -1);
      std::vector<float> carry(1, 0.0f);  // leaf value carried below an original leaf
      for (int l = 0; l < D; ++l) {
        uint32_t* lvl = base;
        for (int q = 0; q < l; ++q) lvl += tpc << q;
        std::vector<int> nsrc(2 << l);
        std::vector<float> ncarry(2 << l);
        for (int i = 0; i < (1 << l); ++i) {
          uint32_t word = always_left;
          uint2 tw = make_uint2(0u, 128u * 0x01010101u);
          int ls = -1, rs = -1;
          float lc = carry[i], rc = carry[i];
          if (src[i] >= 0) {
            const ks_node_host& nd = nodes[off[t] + src[i]];
            if (nd.feat == 0xFFFF) {
              lc = rc = nd.thr_or_leaf;
            } else {
              uint32_t row, jl;
              bool swap = false, always_right = false;
              if (nd.kind == KS_NODE_PARTITION) {
                uint32_t mask;
                std::memcpy(&mask, &nd.thr_or_leaf, 4);
                if (mask == (1u << categorical_levels(nd.feat)) - 1) {
                  always_right = true;  // every level is a member
                  row = 0;
                  jl = 127;
                } else {
                  const PartitionCode pc = part[nd.feat][mask];
                  row = fq[nd.feat].row0 + rank_row[nd.feat][pc.perm];
                  jl = pc.cut - 1;
                  swap = pc.swap;
                }
              } else {
                const auto& v = thr[nd.feat];
                const int j = static_cast<int>(std::lower_bound(v.begin(), v.end(), nd.thr_or_leaf) - v.begin());
                row = fq[nd.feat].row0 + j / kSlice;
                jl = j % kSlice;
              }
              ls = nd.left;
              rs = nd.left + 1;
              if (always_right) {
                ls = rs;  // the walk always goes left here: put the right subtree on both sides
              } else {
                word = (row * NC) << 8 | (0x80u | jl);
                tw = make_uint2(row * NC, (jl + 1) * 0x01010101u);
                if (swap) std::swap(ls, rs);
              }
            }
          }
          lvl[tt * (1 << l) + i] = word;
          if (l < L) {
            const size_t at = static_cast<size_t>(t) * n_top + ((1 << l) - 1) + i;
            if (compact) reinterpret_cast<uint32_t*>(top->w)[at] = (tw.x << 8) | (tw.y & 0xFFu);
            else top->w[at] = tw;
          }
          nsrc[2 * i] = ls;
          nsrc[2 * i + 1] = rs;
          ncarry[2 * i] = lc;
          ncarry[2 * i + 1] = rc;
        }
        src.swap(nsrc);
        carry.swap(ncarry);
      }
      for (int i = 0; i < (1 << D); ++i) {
        float v = carry[i];
        if (src[i] >= 0) v = nodes[off[t] + src[i]].thr_or_leaf;
        leaves[tt * (1 << D) + i] = v;
      }
    }
  }
  cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&m.d_qnodes), chunks.size() * 4);
  if (e == cudaSuccess) e = cudaMemcpy(m.d_qnodes, chunks.data(), chunks.size() * 4, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&m.d_qthr), table.size() * 4);
  if (e == cudaSuccess) e = cudaMemcpy(m.d_qthr, table.data(), table.size() * 4, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&m.d_qfeat), sizeof(fq));
  if (e == cudaSuccess) e = cudaMemcpy(m.d_qfeat, fq, sizeof(fq), cudaMemcpyHostToDevice);
  if (e != cudaSuccess) {
    delete top;
    return e;
  }
  m.h_top = top;
  m.top_levels = L;
  m.top_compact = compact;
  m.fast = true;
  m.fast_depth = D;
  m.fast_threads = threads;
  m.block_cands = NC;
  m.buf_bytes = group_buf;
  m.ctas_per_sm = geom.ctas_per_sm;
  m.n_qrows = n_rows;
  m.n_pair_rows = n_class[2];
  m.n_cand_rows = n_class[1];
  m.n_prob_rows = n_class[0];
  m.n_qthr = thr_class[0] + thr_class[1] + thr_class[2];
  m.thr_cand0 = thr_class[2];
  m.thr_prob0 = thr_class[2] + thr_class[1];
  m.tpc = tpc;
  m.n_chunks = n_chunks;
  m.chunk_bytes = chunk_words * 4;
  return cudaSuccess;
}

void free_fast_gbdt(GbdtModel& m) {
  delete m.h_top;
  m.h_top = nullptr;
}

// ------------------------------------------------------------------------------------------
// launcher
// ------------------------------------------------------------------------------------------

// Blocks per problem: full tiles of the model's block size. A block's cost does not depend on how
// many of its slots are live, so an under-filled machine is filled by splitting the trees over
// several CTAs per block (slices) rather than by shorter blocks.
void fast_tiling(const GbdtModel& g, int P, int64_t per_problem, int* nblk, int* rows_per_cta) {
  int64_t n = (per_problem + g.block_cands - 1) / g.block_cands;
  if (n < 1) n = 1;
  (void)P;
  *nblk = static_cast<int>(n);
  *rows_per_cta = g.block_cands;
}

static int cand_rec_bytes(const GbdtModel& g) { return g.n_cand_rows > 0 ? (g.n_cand_rows + 15) / 16 * 16 : 16; }
static int pair_rec_bytes(const GbdtModel& g) { return (g.n_pair_rows + 15) / 16 * 16; }

size_t fast_scratch_bytes(const GbdtModel& g, int C) {
  return 256 + static_cast<size_t>(kCombos) * C * cand_rec_bytes(g);
}

// Memo of the per-pair rows (see MemoView): worth its per-problem table only for a batch of
// problems. The table is held for at most `fast_memo_batch` problems at a time (256 MiB of
// records); a larger call is served batch by batch. 0 = not used.
size_t memo_fixed_bytes(int C) {
  return static_cast<size_t>(kMemoCombos) * kMemoCap * (sizeof(unsigned long long) + 2 * sizeof(int)) + 256 +
         (static_cast<size_t>(kMemoCombos) * C * sizeof(unsigned) + 255) / 256 * 256;
}
MemoView memo_view(void* mem, int C) {
  char* m = static_cast<char*>(mem);
  const size_t slots = static_cast<size_t>(kMemoCombos) * kMemoCap;
  MemoView v{};
  v.keys = reinterpret_cast<unsigned long long*>(m);
  v.count = reinterpret_cast<int*>(m + slots * sizeof(unsigned long long));
  v.dense = reinterpret_cast<int*>(m + slots * sizeof(unsigned long long) + 256);
  v.reps = v.dense + slots;
  v.cls = reinterpret_cast<unsigned*>(v.reps + slots);
  v.tab = m + memo_fixed_bytes(C);
  return v;
}
cudaError_t memo_clear(const MemoView& memo, cudaStream_t stream) {
  return cudaMemsetAsync(memo.keys, 0, static_cast<size_t>(kMemoCombos) * kMemoCap * sizeof(unsigned long long), stream);
}
cudaError_t memo_compact(const MemoView& memo, cudaStream_t stream) {
  memo_compact_kernel<<<kMemoCombos, 1024, 0, stream>>>(memo);
  return cudaGetLastError();
}

int fast_memo_batch(const GbdtModel& g, int P) {
  if (P < kMemoMinProblems || g.n_pair_rows < 1 || g.n_pair_rows > kFastMaxPairRec) return 0;
  const size_t per_problem = static_cast<size_t>(kMemoCap) * pair_rec_bytes(g);
  int64_t batch = static_cast<int64_t>(kMemoTableBytes / per_problem);
  if (batch < kMemoMinProblems) batch = kMemoMinProblems;
  return static_cast<int>(batch < P ? batch : P);
}

size_t fast_memo_bytes(const GbdtModel& g, int P, int C) {
  const int batch = fast_memo_batch(g, P);
  if (batch == 0 || C < 1) return 0;
  return memo_fixed_bytes(C) + static_cast<size_t>(batch) * (static_cast<size_t>(kMemoCap) * pair_rec_bytes(g) + kProbRec);
}

// Slice count of the single-problem call: the trees are split over S CTAs per candidate block.
// A CTA costs its tile fill (about 0.15 of a whole-ensemble walk of its block) plus 1 / S of that
// walk, and blocks x S CTAs run in waves of the CTAs the machine holds at once: the S with the
// shortest estimated makespan wins.
int fast_slices(const GbdtModel& g, int64_t blocks) {
  if (blocks < 1) blocks = 1;
  if (blocks > kMaxSliceBlocks) return 1;
  const int64_t slots = static_cast<int64_t>(g.ctas_per_sm) * kSmCount;
  if (blocks >= slots) return 1;  // the machine is full without slices
  int best = 1;
  double best_cost = 1e30;
  for (int s = 1; s <= g.n_chunks && s <= 32; ++s) {
    const int64_t waves = (blocks * s + slots - 1) / slots;
    const double cost = static_cast<double>(waves) * (0.15 + 1.0 / s);
    if (cost < best_cost - 1e-9) {
      best_cost = cost;
      best = s;
    }
  }
  return best;
}

size_t fast_prepared_rows_bytes(const GbdtModel& g, int C) { return static_cast<size_t>(kCombos) * C * cand_rec_bytes(g); }
size_t fast_prepared_memo_bytes(const GbdtModel& g, int C) {
  if (g.n_pair_rows < 1 || g.n_pair_rows > kFastMaxPairRec || C < 1) return 0;
  return memo_fixed_bytes(C) + static_cast<size_t>(kMemoCap) * pair_rec_bytes(g) + kProbRec;
}

namespace {

struct WalkArgs {
  ks_gpu_desc desc;
  const ks_problem* d_p;
  ks_problem pv;
  int uv;
  const ks_candidate* d_c;
  int P, C, nblk, rows_per_cta;
  const int64_t* seg_off;
  const int32_t* seg_idx;
  FastView fv;
  int k;
  unsigned long long* partial;
  int* status;
  SliceArgs sl;
  const FastTopParams* top;
  cudaStream_t stream;
  int dependent;  // launched right behind the kernel whose tables it reads
};

template <int L, int NP, bool kCompact, int THREADS, int NC, bool kFloor = false>
cudaError_t launch_ln(const WalkArgs& a) {
  const size_t smem = static_cast<size_t>(kNBuf) * ring_count(THREADS / (NC / 4)) * a.fv.buf_bytes +
                      static_cast<size_t>(a.fv.n_rows) * NC;
  auto kernel = &select_fast_kernel<L, NP, kCompact, THREADS, NC, kFloor>;
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kernel), smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg{};
  // One CTA per item, or - batch form of the geometries that hold one CTA per SM - one CTA per SM,
  // each serving many items. (Two persistent CTAs on an SM run in step, so that both fill and rank
  // at the same time and neither hides the other's: measured 6 % slower than one CTA per item.)
  const int64_t n_items = static_cast<int64_t>(a.P) * a.nblk * a.sl.n_slices;
  const bool persistent = THREADS > 256 && a.sl.n_slices == 1 && !a.sl.score_out && !a.sl.tiles;
  const int64_t slots = kSmCount;
  cfg.gridDim = dim3(static_cast<unsigned>(persistent && n_items > slots ? slots : n_items));
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = a.stream;
  // behind a table kernel the grid is launched as its programmatic dependent: its CTAs may start
  // their set-up while that kernel still runs, and wait for it (griddepcontrol.wait) before they
  // read its tables
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = a.dependent ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, a.desc, a.d_p, a.pv, a.uv, a.d_c, a.P, a.C, a.nblk, a.rows_per_cta,
                            a.seg_off, a.seg_idx, a.fv, a.k, a.partial, a.status, a.sl, static_cast<int>(n_items),
                            *a.top);
}

// the instantiation for a model's top levels and depth, within one tile geometry
template <int THREADS, int NC>
cudaError_t launch_walk_geom(const GbdtModel& g, const WalkArgs& a) {
  const int L = g.top_levels, np = g.fast_depth - L;
  if (g.top_compact) {
    if (np == 5) return launch_ln<3, 5, true, THREADS, NC>(a);
    if (np == 4) return launch_ln<3, 4, true, THREADS, NC>(a);
    return launch_ln<3, -1, true, THREADS, NC>(a);
  }
  if (L == 3 && np == 5) return launch_ln<3, 5, false, THREADS, NC>(a);
  if (THREADS == 512 && NC == 1024) {  // the shapes met so far only in small ensembles
    if (L == 3 && np == 3) return launch_ln<3, 3, false, 512, 1024>(a);
    if (L == 2 && np == 6) return launch_ln<2, 6, false, 512, 1024>(a);
    if (L == 2 && np == 5) return launch_ln<2, 5, false, 512, 1024>(a);  // the paper-sized ensemble: 916 trees of depth 7
  }
  if (L == 3 && np == 4) return launch_ln<3, 4, false, THREADS, NC>(a);
  if (L == 3) return launch_ln<3, -1, false, THREADS, NC>(a);
  if (L == 2) return launch_ln<2, -1, false, THREADS, NC>(a);
  if (L == 1) return launch_ln<1, -1, false, THREADS, NC>(a);
  return launch_ln<0, -1, false, THREADS, NC>(a);
}

// The floor measurement exists for the two geometries and the ensemble shape of the benchmark's
// first configuration (three word-wise levels, five path levels, top constants as pairs).
cudaError_t launch_walk_floor(const GbdtModel& g, const WalkArgs& a) {
  if (g.top_compact || g.top_levels != 3 || g.fast_depth != 8 || g.block_cands != 1024 ||
      g.n_chunks < kNBuf * ring_count(g.fast_threads / 256))  // every ring needs its kNBuf resident chunks
    return cudaErrorNotSupported;
  if (g.fast_threads == 512) return launch_ln<3, 5, false, 512, 1024, true>(a);
  return launch_ln<3, 5, false, 256, 1024, true>(a);
}

cudaError_t launch_walk(const GbdtModel& g, const WalkArgs& a) {
  if (g.fast_threads == 512 && g.block_cands == 1024) return launch_walk_geom<512, 1024>(g, a);
  if (g.fast_threads == 512) return launch_walk_geom<512, 512>(g, a);
  if (g.block_cands == 512) return launch_walk_geom<256, 512>(g, a);
  return launch_walk_geom<256, 1024>(g, a);
}

FastView make_view(const GbdtModel& g, const FastWait* wait) {
  FastView fv{};
  fv.n_rows = g.n_qrows;
  fv.n_pair_rows = g.n_pair_rows;
  fv.n_cand_rows = g.n_cand_rows;
  fv.n_prob_rows = g.n_prob_rows;
  fv.depth = g.fast_depth;
  fv.n_chunks = g.n_chunks;
  fv.chunk_bytes = g.chunk_bytes;
  fv.tpc = g.tpc;
  fv.n_thr = g.n_qthr;
  fv.thr_cand0 = g.thr_cand0;
  fv.thr_prob0 = g.thr_prob0;
  fv.cand_rec = cand_rec_bytes(g);
  fv.pair_rec = pair_rec_bytes(g);
  fv.wait_limit = wait && wait->limit > 0 ? wait->limit : kFastWaitLimit;
  fv.starve = wait ? wait->starve : 0;
  fv.buf_bytes = g.buf_bytes;
  fv.base = g.base;
  fv.chunks = g.d_qnodes;
  fv.thr = g.d_qthr;
  fv.feat = g.d_qfeat;
  return fv;
}

// Dynamic shared memory for `count` staged thresholds: all of them when they fit, else none (the
// kernel then searches the global array). Returns the capacity in floats to pass to the kernel.
int staged_floats(int count, size_t* bytes) {
  constexpr int kCap = 48 * 1024;  // floats: 192 KB
  const int cap = count <= kCap ? (count > 0 ? count : 1) : 0;
  *bytes = static_cast<size_t>(cap > 0 ? cap : 1) * sizeof(float);
  return cap;
}

}  // namespace

// Prepared catalogue: the candidate-only rows of every candidate under every element-type
// combination, and the candidates' classes, computed once for a (catalogue, model) pair.
cudaError_t fast_prepare(const ks_gpu_desc& desc, const GbdtModel& g, const ks_candidate* d_c, int C, void* d_rows,
                         void* memo_mem, cudaStream_t stream, int64_t* launches) {
  FastView fv = make_view(g, nullptr);
  MemoView memo{};
  if (memo_mem) memo = memo_view(memo_mem, C);
  size_t cthr = 0;
  const int cap = staged_floats(g.thr_prob0 - g.thr_cand0, &cthr);
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(&cand_rows_kernel), cthr);
  if (e != cudaSuccess) return e;
  if (memo.keys) {
    e = memo_clear(memo, stream);
    if (e != cudaSuccess) return e;
  }
  cand_rows_kernel<<<dim3((C + 255) / 256, kCombos), 256, cthr, stream>>>(desc, d_c, C, nullptr, 0xFFFFu, fv,
                                                                          static_cast<uint8_t*>(d_rows), memo, cap);
  ++*launches;
  if (memo.keys) {
    e = memo_compact(memo, stream);
    if (e != cudaSuccess) return e;
    ++*launches;
  }
  return cudaGetLastError();
}

// Problems per launch when a call is served in batches of at most `cap`. In the launch form
// with one CTA per SM every launch runs its items in rounds of kSmCount, and a last round that
// is nearly empty still takes a whole item's time; a batch a little below the cap can save a
// round per launch (4,096 problems x 32 blocks in batches of 226 instead of 227: 889 rounds
// instead of 903: 133.3 -> 130.7 ms). Picks the size within an eighth below the cap that needs
// the fewest rounds. (With two CTAs per SM, one per item, the hardware hands out the items and
// the same rule measured 0.6 % slower: not applied there.)
static int balanced_step(const GbdtModel& g, int P, int cap, int nblk) {
  if (P <= cap || g.ctas_per_sm != 1 || cap < 16) return cap;
  int best = cap;
  int64_t best_rounds = INT64_MAX;
  for (int n = cap; n >= cap - cap / 8; --n) {
    int64_t rounds = 0;
    for (int first = 0; first < P; first += n) {
      const int64_t items = static_cast<int64_t>(P - first < n ? P - first : n) * nblk;
      rounds += (items + kSmCount - 1) / kSmCount;
    }
    if (rounds < best_rounds) {
      best_rounds = rounds;
      best = n;
    }
  }
  return best;
}

cudaError_t launch_select_fast(const ks_gpu_desc& desc, const GbdtModel& g, const ks_problem* d_p,
                               const ks_problem* p_by_value, int P, const ks_candidate* d_c, int C,
                               int nblk, int rows_per_cta, const int64_t* seg_off, const int32_t* seg_idx,
                               int k, unsigned long long* partial, void* scratch, int* status,
                               cudaStream_t stream, int64_t* launches, cudaEvent_t ev_begin,
                               const FastSlice* slice, void* memo_mem, const FastWait* wait,
                               const FastPrepared* prep, const int32_t* perm) {
  WalkArgs a{};
  a.desc = desc;
  if (p_by_value) a.pv = *p_by_value;
  a.uv = p_by_value != nullptr;
  a.d_c = d_c;
  a.C = C;
  a.nblk = nblk;
  a.rows_per_cta = rows_per_cta;
  a.seg_idx = seg_idx;
  a.k = k;
  a.status = status;
  a.top = g.h_top;
  a.stream = stream;
  FastView& fv = a.fv;
  fv = make_view(g, wait);
  unsigned* d_mask = static_cast<unsigned*>(scratch);
  uint8_t* d_rows = static_cast<uint8_t*>(scratch) + 256;
  fv.cand_rows = d_rows;
  if (!seg_off && perm) a.seg_idx = perm;  // dense form ranked in the given order of the catalogue
  MemoView memo{};
  int memo_batch = (memo_mem && !p_by_value && C > 0) ? fast_memo_batch(g, P) : 0;
  if (memo_batch > 0) memo = memo_view(memo_mem, C);
  if (prep) {  // prepared catalogue: candidate-only rows and classes were made once, for every type combination
    fv.cand_rows = prep->cand_rows;
    if (prep->memo_mem) {
      memo = memo_view(prep->memo_mem, C);
      memo_batch = 1;
    }
  }

  // candidate-only rows for the type combinations in use
  cudaError_t e = cudaSuccess;
  unsigned mask_value = 0;
  if (prep) {
    // nothing to do per call
  } else if (a.uv) {
    mask_value = 1u << ((a.pv.dtype_ab & 3) * 4 + (a.pv.dtype_d & 3));
  } else {
    e = cudaMemsetAsync(d_mask, 0, sizeof(unsigned), stream);
    if (e != cudaSuccess) return e;
    combo_mask_kernel<<<P >= 4096 ? 16 : 1, 256, 0, stream>>>(d_p, P, d_mask);
    ++*launches;
  }
  const bool tiles_mode = a.uv && slice && slice->n_slices > 1 && slice->tiles && P == 1 && !seg_off;
  // shared memory of the table kernel: the per-pair thresholds when they fit beside its 256 records
  size_t pthr_bytes = 0;
  int pthr_cap = staged_floats(g.thr_cand0, &pthr_bytes);
  {
    const size_t rec_bytes = static_cast<size_t>(256) * pair_rec_bytes(g);
    size_t thr_part = pthr_cap > 0 ? static_cast<size_t>((pthr_cap + 3) / 4 * 4) * sizeof(float) : 0;
    if (thr_part + rec_bytes > 200 * 1024) {
      pthr_cap = 0;
      thr_part = 0;
    }
    pthr_bytes = thr_part + rec_bytes + 16;
  }
  if (prep) {
    if (memo.keys) {
      e = ensure_dynamic_smem(reinterpret_cast<const void*>(&pair_table_kernel), pthr_bytes);
      if (e != cudaSuccess) return e;
      fv.pair_class = memo.cls;
      fv.pair_tab = static_cast<const uint8_t*>(memo.tab);
      fv.prob_tab = fv.pair_tab + static_cast<size_t>(kMemoCap) * pair_rec_bytes(g);
    }
  } else if (tiles_mode) {
    // one launch, two roles (blockIdx.y): the per-pair rows, and the candidate- / problem-only rows
    size_t tthr = 0;
    const int cap = staged_floats(std::max(g.thr_cand0, g.n_qthr - g.thr_cand0), &tthr);
    e = ensure_dynamic_smem(reinterpret_cast<const void*>(&tile_one_kernel), tthr);
    if (e != cudaSuccess) return e;
    tile_one_kernel<<<dim3(nblk * (g.block_cands / 256), 2), 256, tthr, stream>>>(desc, a.pv, d_c, C, fv,
                                                                                   g.block_cands, slice->tiles, cap);
    ++*launches;
  } else if (C > 0) {
    size_t cthr = 0;
    const int cap = staged_floats(g.thr_prob0 - g.thr_cand0, &cthr);
    e = ensure_dynamic_smem(reinterpret_cast<const void*>(&cand_rows_kernel), cthr);
    if (e != cudaSuccess) return e;
    if (memo.keys) {
      e = memo_clear(memo, stream);
      if (e != cudaSuccess) return e;
    }
    cand_rows_kernel<<<dim3((C + 255) / 256, kCombos), 256, cthr, stream>>>(desc, d_c, C, a.uv ? nullptr : d_mask,
                                                                            mask_value, fv, d_rows, memo, cap);
    ++*launches;
    if (memo.keys) {
      e = ensure_dynamic_smem(reinterpret_cast<const void*>(&pair_table_kernel), pthr_bytes);
      if (e != cudaSuccess) return e;
      e = memo_compact(memo, stream);
      if (e != cudaSuccess) return e;
      ++*launches;
      fv.pair_class = memo.cls;
      fv.pair_tab = static_cast<const uint8_t*>(memo.tab);
      fv.prob_tab = fv.pair_tab + static_cast<size_t>(memo_batch) * kMemoCap * pair_rec_bytes(g);
    }
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (ev_begin) cudaEventRecord(ev_begin, stream);

  a.sl.n_slices = 1;
  if (slice && slice->n_slices > 1) {
    a.sl.n_slices = slice->n_slices;
    a.sl.pairs = slice->pairs;
    a.sl.scores = slice->scores;
    a.sl.counters = slice->counters;
    a.sl.out_idx = slice->out_idx;
    a.sl.out_score = slice->out_score;
    a.sl.tiles = tiles_mode ? slice->tiles : nullptr;
    a.sl.out_seq = slice->out_seq;
    a.sl.seq = slice->seq;
  }
  // problems in batches when the memo's table does not hold them all at once
  const int step = memo.keys ? balanced_step(g, P, memo_batch, nblk) : P;
  for (int first = 0; first < P; first += step) {
    const int n = P - first < step ? P - first : step;
    if (memo.keys) {
      // as many blocks as the machine holds at once (two per SM by registers, fewer when the staged
      // thresholds take more than half an SM's shared memory); never more blocks than items
      const int64_t table_items = static_cast<int64_t>(kMemoCap / 256) * n;
      const int64_t table_slots = static_cast<int64_t>(kSmCount) * (2 * (pthr_bytes + 4096) <= 227 * 1024 ? 2 : 1);
      pair_table_kernel<<<static_cast<unsigned>(table_items < table_slots ? table_items : table_slots), 256, pthr_bytes,
                          stream>>>(
          desc, d_p ? d_p + first : nullptr, a.pv, a.uv, n, d_c, fv, memo, pthr_cap);
      ++*launches;
    }
    a.dependent = memo.keys != nullptr;
    a.d_p = d_p ? d_p + first : nullptr;
    a.P = n;
    a.seg_off = seg_off ? seg_off + first : nullptr;
    a.partial = partial + static_cast<size_t>(first) * nblk * k;
    e = launch_walk(g, a);
    ++*launches;
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// ks_score on the quantised path. Rows are taken in batches so that the tiles (n_rows bytes per
// row) stay a bounded workspace; every batch is one tile launch and one walk launch.
constexpr int64_t kScoreBatchRows = 4096 * 1024;

size_t score_fast_scratch_bytes(const GbdtModel& g, int64_t rows) {
  int64_t blocks = (std::min(rows, kScoreBatchRows) + g.block_cands - 1) / g.block_cands;
  return static_cast<size_t>(blocks) * g.n_qrows * g.block_cands;
}

cudaError_t launch_score_fast(const ks_gpu_desc& desc, const GbdtModel& g, const float* d_feat, int64_t rows,
                              float* d_scores, void* scratch, int* status, cudaStream_t stream,
                              int64_t* launches, const FastWait* wait, int floor_repeat) {
  WalkArgs a{};
  a.desc = desc;
  a.uv = 1;
  a.P = 1;
  a.rows_per_cta = g.block_cands;
  a.status = status;
  a.top = g.h_top;
  a.stream = stream;
  a.fv = make_view(g, wait);
  uint8_t* tiles = static_cast<uint8_t*>(scratch);
  size_t tthr = 0;
  const int cap = staged_floats(g.n_qthr, &tthr);
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(&tile_rows_kernel), tthr);
  if (e != cudaSuccess) return e;
  for (int64_t first = 0; first < rows; first += kScoreBatchRows) {
    const int64_t n = rows - first < kScoreBatchRows ? rows - first : kScoreBatchRows;
    const int nblk = static_cast<int>((n + g.block_cands - 1) / g.block_cands);
    tile_rows_kernel<<<nblk, g.block_cands / 4, tthr, stream>>>(d_feat + first * KS_F_PAD, n, a.fv, tiles, cap);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    a.C = static_cast<int>(n);
    a.nblk = nblk;
    a.sl = SliceArgs{};
    a.sl.n_slices = 1;
    a.sl.tiles = tiles;
    a.sl.score_out = d_scores + first;
    a.sl.repeat = floor_repeat;
    *launches += 2;
    e = floor_repeat > 0 ? launch_walk_floor(g, a) : launch_walk(g, a);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

#ifdef KS_DEBUG_BOUNDS
int fast_bounds_line() {
  int v = 0;
  cudaMemcpyFromSymbol(&v, g_bounds_line, sizeof(int));
  return v;
}
void fast_bounds_clear() {
  const int z = 0;
  cudaMemcpyToSymbol(g_bounds_line, &z, sizeof(int));
}
#else
int fast_bounds_line() { return -1; }
void fast_bounds_clear() {}
#endif

}  // namespace ks
