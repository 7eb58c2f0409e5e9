// Quantised fast path of the fused select kernel for tree ensembles (Model A).
//
// Repack (host, at model-create time)
//   A split "x[f] < thr" only needs to know how many of feature f's distinct thresholds are
//   <= x. With the thresholds of f sorted, bin(x) = #{j : thr_j <= x}, and
//   x < thr_j  <=>  bin(x) <= j  exactly, so a pair's feature row shrinks from 64 floats to
//   one byte per "row" (a feature, or a 127-threshold slice of one) and a node to one 32-bit
//   word. Trees are padded to complete trees of the ensemble's depth D and stored in chunks,
//   each chunk laid out level by level ([level][tree][node]) followed by its leaves, so that a
//   chunk is one contiguous block a CTA copies into shared memory with one bulk async copy.
//   The nodes of the top levels are also kept as (row offset, replicated threshold) pairs that
//   travel as a kernel parameter, i.e. through the constant bank.
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
// Kernel (one CTA = one problem x up to kFastRows candidates, kFastThreads threads, two CTAs per SM)
//   phase A  fill the [row][candidate] byte tile. A 32-bit word of a row holds the four
//            candidates that share a lane slot, so a warp's byte loads of any mix of rows
//            touch 32 distinct banks and one word load serves four candidates;
//   phase B  stream the ensemble through two shared-memory buffers (cp.async.bulk + mbarrier,
//            bounded waits). Thread (w, h) owns the four candidates of word w and walks the
//            trees of half h of every chunk. The top levels are evaluated for all four
//            candidates at once, node by node, with byte-parallel arithmetic on whole words;
//            below that each candidate follows its own path: a' = 2 a + k0 (+ 4 to go right), a
//            multiply-add plus a predicated add;
//   phase C  add the two halves' partial scores, rank the block's keys, write a partial
//            top-k list.
#include <algorithm>
#include <cmath>
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

constexpr int kBufBytes = 16 * 1024;   // one tree-chunk buffer
constexpr int kMaxRows = 80;           // quantised rows the kernel supports (tile <= 160 KB)
constexpr int kThrPerRow = 128;        // 127 thresholds + padding
constexpr int kRowStride = kFastRows;  // bytes between rows of the tile (one byte per candidate)
constexpr int kWords = kFastRows / 4;  // words per row = lane slots
constexpr unsigned kSleepNs = 1200;  // asked-for sleep between two probes of a chunk barrier (400 to 2500 measured alike)
constexpr int kSpinLimit = 1 << 23;  // probes (a sleep ends early, ~0.2 us measured): a wait gives up after a few seconds
constexpr int kCandRec = 64;           // bytes per (combination, candidate) record of quantised rows
constexpr int kCombos = 16;            // dtype_ab x dtype_d

static_assert(kFastThreads == 2 * kWords && kFastR == 2, "tile geometry");

// shared memory map (byte offsets from the dynamic shared base)
constexpr int kNBuf = 2;                // tree-chunk buffers (a ring; four of 8 KB and three of 12 KB measured slower)
constexpr int kOffBuf0 = 0;
constexpr int kOffTile = kNBuf * kBufBytes;

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
// or without a time hint); gives up after kSpinLimit probes and reports false.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  if (mbar_test_wait(bar, parity)) return true;
  for (int i = 0; i < kSpinLimit; ++i) {
    __nanosleep(kSleepNs);
    if (mbar_test_wait(bar, parity)) return true;
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

// #{j : T[j] <= v} over 127 sorted thresholds padded with +inf: 7 branch-free steps.
__device__ __forceinline__ int bin_search(const float* T, float v) {
  int pos = 0;
#pragma unroll
  for (int s = 64; s >= 1; s >>= 1) pos += (T[pos + s - 1] <= v) ? s : 0;
  return pos;
}

// Bin of value v in one row of the threshold table. A row whose last slot is negative infinity is
// a rank row of a categorical field: slot c holds the rank of level c in the row's ordering of
// the levels (see build_fast_gbdt), and the bin is that rank.
__device__ __forceinline__ int row_bin(const float* T, float v) {
  if (T[kThrPerRow - 1] < 0.0f) {
    const int code = __float2int_rz(v);
    return (code >= 0 && code < 4) ? __float2int_rz(T[code]) : 0;
  }
  return bin_search(T, v);
}

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
  const uint8_t* tiles;    // prepared tiles [blocks][rows][kRowStride] (tile_one_kernel), or null
  int* out_seq;            // single-problem form: receives `seq` once the k results are written
  int seq;
  float* score_out;        // scoring call (ks_score): the scores of the block's rows go here, no ranking
};

struct FastView {
  int n_rows, n_pair_rows, n_cand_rows, n_prob_rows;  // rows are ordered pair, candidate, problem
  int depth, n_chunks, chunk_bytes, tpc;
  float base;
  const uint32_t* chunks;      // [n_chunks][chunk_bytes / 4]
  const float* thr;            // [n_rows][kThrPerRow]
  const uint8_t* feat_row0;    // [64] first row of each feature column
  const uint8_t* feat_rowcnt;  // [64] number of rows of each feature column
  const uint8_t* cand_rows;    // [kCombos][C][kCandRec] quantised candidate-only rows
  const unsigned* pair_class;  // [kCombos][C] class of every candidate, or null (no memo)
  const uint8_t* pair_tab;     // [P][kMemoCap][kMemoRec] per-pair tile bytes of every (problem, class)
};

// Memo of the per-pair rows (classes: ks_memo.cuh). Per problem the tile bytes of the per-pair
// rows are evaluated once per class from the class's member; phase A then copies a 64-byte
// record instead of evaluating 21 columns and searching their rows.
constexpr int kMemoRec = 64;  // bytes per record = most per-pair rows a memoised model may have

// ------------------------------------------------------------------------------------------
// candidate-only rows, once per call
// ------------------------------------------------------------------------------------------

__global__ void combo_mask_kernel(const ks_problem* __restrict__ p, int P, unsigned* __restrict__ mask) {
  unsigned m = 0;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < P; i += gridDim.x * blockDim.x)
    m |= 1u << ((p[i].dtype_ab & 3) * 4 + (p[i].dtype_d & 3));
  m = __reduce_or_sync(0xFFFFFFFFu, m);
  if ((threadIdx.x & 31) == 0 && m) atomicOr(mask, m);
}

__global__ void __launch_bounds__(256)
cand_rows_kernel(ks_gpu_desc desc, const ks_candidate* __restrict__ c, int C, const unsigned* mask_ptr,
                 unsigned mask_value, FastView fv, uint8_t* __restrict__ out, MemoView memo) {
  extern __shared__ float s_cthr[];  // thresholds of the candidate-only rows
  __shared__ uint8_t s_r0[64], s_rc[64];
  const int combo = blockIdx.y;
  if (blockIdx.x == 0 && combo == 0 && threadIdx.x == 0) g_fast_abort = 0;
  const unsigned mask = mask_ptr ? *mask_ptr : mask_value;
  if (!((mask >> combo) & 1u)) return;
  const int first = fv.n_pair_rows;
  for (int i = threadIdx.x; i < fv.n_cand_rows * kThrPerRow; i += blockDim.x)
    s_cthr[i] = __ldg(fv.thr + first * kThrPerRow + i);
  if (threadIdx.x < 64) {
    s_r0[threadIdx.x] = fv.feat_row0[threadIdx.x];
    s_rc[threadIdx.x] = fv.feat_rowcnt[threadIdx.x];
  }
  __syncthreads();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= C) return;
  ks_problem fake{};
  fake.m = fake.n = fake.k = 1;
  fake.dtype_ab = static_cast<uint8_t>(combo >> 2);
  fake.dtype_d = static_cast<uint8_t>(combo & 3);
  ProblemTerms t;
  problem_terms(fake, desc, t);
  const ks_candidate cand = c[i];
  uint32_t rec[kCandRec / 4];
#pragma unroll
  for (int q = 0; q < kCandRec / 4; ++q) rec[q] = 0x80808080u;
  featurize_pair(t, cand, desc, [&](int col, float v) {
    if (feat_class(col) != 1) return;
    const int r0 = s_r0[col] - first, rc = s_rc[col];
    for (int q = 0; q < rc; ++q) {
      const uint32_t b = 0x80u | row_bin(s_cthr + (r0 + q) * kThrPerRow, v);
      const int at = r0 + q;
#pragma unroll
      for (int w = 0; w < kCandRec / 4; ++w)
        if (w == (at >> 2)) rec[w] = (rec[w] & ~(0xFFu << (8 * (at & 3)))) | (b << (8 * (at & 3)));
    }
  });
  uint4* dst = reinterpret_cast<uint4*>(out + (static_cast<size_t>(combo) * C + i) * kCandRec);
#pragma unroll
  for (int q = 0; q < kCandRec / 16; ++q)
    if (q * 16 < fv.n_cand_rows) dst[q] = make_uint4(rec[4 * q], rec[4 * q + 1], rec[4 * q + 2], rec[4 * q + 3]);
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

// Per problem: the tile bytes of the per-pair rows of every class, from the class's member.
// grid (kMemoCap / 256, P); blocks past the number of classes leave at once.
__global__ void __launch_bounds__(256)
pair_table_kernel(ks_gpu_desc desc, const ks_problem* __restrict__ p, const ks_candidate* __restrict__ c,
                  FastView fv, MemoView memo) {
  extern __shared__ float s_pthr[];  // thresholds of the per-pair rows
  __shared__ ProblemTerms s_pt;
  __shared__ uint8_t s_r0[64], s_rc[64];
  const int prob = blockIdx.y, j = blockIdx.x * 256 + threadIdx.x;
  const ks_problem pr = p[prob];
  const int combo = (pr.dtype_ab & 3) * 4 + (pr.dtype_d & 3);
  const int n_classes = memo.count[combo];
  if (blockIdx.x * 256 >= n_classes) return;
  const int slot = j < n_classes ? memo.dense[static_cast<size_t>(combo) * kMemoCap + j] : 0;
  const unsigned long long key = j < n_classes ? 1ull : 0ull;
  for (int i = threadIdx.x; i < fv.n_pair_rows * kThrPerRow; i += 256) s_pthr[i] = __ldg(fv.thr + i);
  if (threadIdx.x < 64) {
    s_r0[threadIdx.x] = fv.feat_row0[threadIdx.x];
    s_rc[threadIdx.x] = fv.feat_rowcnt[threadIdx.x];
  }
  if (threadIdx.x == 0) problem_terms(pr, desc, s_pt);
  __syncthreads();
  if (key == 0ull) return;
  const ks_candidate cand = c[memo.reps[static_cast<size_t>(combo) * kMemoCap + slot]];
  const long long b_eff = resources(s_pt, cand, desc).b_eff;
  uint8_t* rec = static_cast<uint8_t*>(memo.tab) + (static_cast<size_t>(prob) * kMemoCap + slot) * kMemoRec;
  pair_columns<true>(s_pt, cand, desc, b_eff, [&](int col, float v) {
    const int r0 = s_r0[col], rc = s_rc[col];
    for (int q = 0; q < rc; ++q)
      rec[r0 + q] = static_cast<uint8_t>(0x80 | bin_search(s_pthr + (r0 + q) * kThrPerRow, v));
  });
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
                                              uint8_t* __restrict__ tiles, float* s_thr) {
  __shared__ ProblemTerms s_pt;
  __shared__ uint8_t s_r0[64], s_rc[64];
  const int tid = threadIdx.x;
  if (blockIdx.x == 0 && tid == 0) g_fast_abort = 0;
  // rows are ordered per-pair, candidate-only, problem-only
  const int first = kPairRows ? 0 : fv.n_pair_rows;
  const int count = kPairRows ? fv.n_pair_rows : fv.n_rows - fv.n_pair_rows;
  for (int i = tid; i < count * kThrPerRow; i += blockDim.x) s_thr[i] = __ldg(fv.thr + first * kThrPerRow + i);
  if (tid < 64) {
    s_r0[tid] = fv.feat_row0[tid];
    s_rc[tid] = fv.feat_rowcnt[tid];
  }
  if (tid == 0) problem_terms(p_value, desc, s_pt);
  __syncthreads();
  const int slot = blockIdx.x * blockDim.x + tid;
  const int blk = slot / kFastRows, in = slot % kFastRows;
  const int t = in % kFastThreads, r = in / kFastThreads;  // phase-A thread and its candidate
  uint8_t* my = tiles + static_cast<size_t>(blk) * fv.n_rows * kRowStride + (t % kWords) * 4 + (t / kWords) * kFastR + r;
  if (slot >= C) {
    for (int q = first; q < first + count; ++q) my[q * kRowStride] = 0x80;
    return;
  }
  const ks_candidate cand = c[slot];
  featurize_pair(s_pt, cand, desc, [&](int col, float v) {
    if ((feat_class(col) == 2) != kPairRows) return;
    const int r0 = s_r0[col], rc = s_rc[col];
    for (int q = 0; q < rc; ++q)
      my[(r0 + q) * kRowStride] = static_cast<uint8_t>(0x80 | row_bin(s_thr + (r0 + q - first) * kThrPerRow, v));
  });
}

// blockIdx.y picks the role, so that both halves of the work are in flight together
__global__ void __launch_bounds__(256)
tile_one_kernel(ks_gpu_desc desc, ks_problem p_value, const ks_candidate* __restrict__ c, int C, FastView fv,
                uint8_t* __restrict__ tiles) {
  extern __shared__ float s_thr[];  // thresholds of this role's rows
  if (blockIdx.y == 0) tile_one_rows<true>(desc, p_value, c, C, fv, tiles, s_thr);
  else tile_one_rows<false>(desc, p_value, c, C, fv, tiles, s_thr);
}

// ------------------------------------------------------------------------------------------
// scoring call: tiles from feature rows
// ------------------------------------------------------------------------------------------

// ks_score with a qualifying ensemble: one thread per tile word quantises all columns of the
// word's four feature rows into the tile layout of phase A and stores whole words, so that a
// warp's stores are full lines; the walk kernel then copies the tiles as in the single-problem
// call and writes scores instead of ranking. A NaN goes right at every numeric split (x < t is
// false), like +inf: the last bin. Slots past the last row get the neutral byte. Also clears
// the abort flag.
__global__ void __launch_bounds__(kWords)
tile_rows_kernel(const float* __restrict__ feat, int64_t rows, FastView fv, uint8_t* __restrict__ tiles) {
  extern __shared__ float s_thr[];  // thresholds of every row
  __shared__ uint8_t s_r0[64], s_rc[64];
  const int word = threadIdx.x;
  if (blockIdx.x == 0 && word == 0) g_fast_abort = 0;
  {
    const float4* src = reinterpret_cast<const float4*>(fv.thr);
    float4* dst = reinterpret_cast<float4*>(s_thr);
    for (int i = word; i < fv.n_rows * (kThrPerRow / 4); i += kWords) dst[i] = __ldg(src + i);
  }
  if (word < 64) {
    s_r0[word] = fv.feat_row0[word];
    s_rc[word] = fv.feat_rowcnt[word];
  }
  __syncthreads();
  // byte b of the word belongs to phase-A thread word + kWords * (b / 2), candidate b % 2
  const int64_t base = static_cast<int64_t>(blockIdx.x) * kFastRows;
  const float4* src[4];
  bool live[4];
#pragma unroll
  for (int b = 0; b < 4; ++b) {
    const int64_t slot = base + (b & 1) * kFastThreads + word + kWords * (b >> 1);
    live[b] = slot < rows;
    src[b] = reinterpret_cast<const float4*>(feat + (live[b] ? slot : 0) * KS_F_PAD);
  }
  uint32_t* out = reinterpret_cast<uint32_t*>(tiles + static_cast<size_t>(blockIdx.x) * fv.n_rows * kRowStride) + word;
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
      const int r0 = s_r0[col], rc = s_rc[col];
      for (int q = 0; q < rc; ++q) {
        const float* T = s_thr + (r0 + q) * kThrPerRow;
        const bool rank_row = T[kThrPerRow - 1] < 0.0f;
        uint32_t w = 0;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          const float x = v[b][j];
          int bin = (x != x && !rank_row) ? kThrPerRow - 1 : row_bin(T, x);
          if (!live[b]) bin = 0;
          w |= static_cast<uint32_t>(0x80 | bin) << (8 * b);
        }
        out[static_cast<size_t>(r0 + q) * (kRowStride / 4)] = w;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// phase A
// ------------------------------------------------------------------------------------------

// Fills the tile bytes of the two candidates this thread owns in phase A: candidate-only rows
// from the per-call table, problem-only rows from s_pbin, per-pair rows computed here. Slots
// past the end of the segment get a neutral byte so that word-wise arithmetic on the tile
// never borrows across bytes.
__device__ __noinline__ void fill_tile(const ks_gpu_desc& desc, const ProblemTerms& pt,
                                       const ks_candidate* __restrict__ c, const FastView& fv,
                                       const int64_t* __restrict__ seg_off, const int32_t* __restrict__ seg_idx,
                                       int C, int64_t lo, int64_t start, int64_t stop, const float* s_thr,
                                       const uint8_t* s_row0, const uint8_t* s_rowcnt, const uint8_t* s_pbin,
                                       unsigned char* tile, int prob) {
  const int tid = threadIdx.x;
  const int combo = pt.dtype_ab * 4 + pt.dtype_d;
#pragma unroll 1
  for (int r = 0; r < kFastR; ++r) {
    const int64_t row = start + static_cast<int64_t>(r) * kFastThreads + tid;
    unsigned char* my = tile + (tid % kWords) * 4 + (tid / kWords) * kFastR + r;
    if (row >= stop) {
      for (int q = 0; q < fv.n_rows; ++q) my[q * kRowStride] = 0x80;
      continue;
    }
    const int ci = seg_off ? seg_idx[lo + row] : static_cast<int>(row);
    const ks_candidate cand = c[ci];
    // candidate-only rows
    const uint4* rec = reinterpret_cast<const uint4*>(fv.cand_rows + (static_cast<size_t>(combo) * C + ci) * kCandRec);
    unsigned char* dst = my + fv.n_pair_rows * kRowStride;
#pragma unroll
    for (int v = 0; v < kCandRec / 16; ++v) {
      if (v * 16 < fv.n_cand_rows) {
        const uint4 q = __ldg(rec + v);
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int b = 0; b < 16; ++b)
          if (v * 16 + b < fv.n_cand_rows)
            dst[(v * 16 + b) * kRowStride] = static_cast<unsigned char>(w[b >> 2] >> (8 * (b & 3)));
      }
    }
    // problem-only rows
    dst = my + (fv.n_pair_rows + fv.n_cand_rows) * kRowStride;
    for (int q = 0; q < fv.n_prob_rows; ++q) dst[q * kRowStride] = s_pbin[q];
    // per-pair rows: the record of the candidate's class, when there is one
    if (fv.pair_class) {
      const unsigned cid = __ldg(fv.pair_class + static_cast<size_t>(combo) * C + ci);
      if (cid != kNoClass) {
        const uint4* prec =
            reinterpret_cast<const uint4*>(fv.pair_tab + (static_cast<size_t>(prob) * kMemoCap + cid) * kMemoRec);
#pragma unroll
        for (int v = 0; v < kMemoRec / 16; ++v) {
          if (v * 16 < fv.n_pair_rows) {
            const uint4 q = __ldg(prec + v);
            const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int b = 0; b < 16; ++b)
              if (v * 16 + b < fv.n_pair_rows)
                my[(v * 16 + b) * kRowStride] = static_cast<unsigned char>(w[b >> 2] >> (8 * (b & 3)));
          }
        }
        continue;
      }
    }
    featurize_pair(pt, cand, desc, [&](int col, float v) {
      if (feat_class(col) != 2) return;
      const int r0 = s_row0[col], rc = s_rowcnt[col];
      for (int q = 0; q < rc; ++q)
        my[(r0 + q) * kRowStride] = static_cast<unsigned char>(0x80 | bin_search(s_thr + (r0 + q) * kThrPerRow, v));
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
__device__ __forceinline__ uint32_t path_step(uint32_t a, uint32_t cb_r, uint32_t k0) {
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

// L levels evaluated word-wise; NP path levels unrolled (-1: runtime count); kCompact: the top
// levels' constants travel as one 32-bit word per node (row offset << 8 | j + 1) instead of a
// (row offset, replicated j + 1) pair, so that twice as many trees keep their word-wise levels.
template <int L, int NP, bool kCompact = false>
__global__ void __launch_bounds__(kFastThreads, 2)
select_fast_kernel(ks_gpu_desc desc, const ks_problem* __restrict__ p, ks_problem p_value, int use_value,
                   const ks_candidate* __restrict__ c, int P, int C, int nblk, int rows_per_cta,
                   const int64_t* __restrict__ seg_off, const int32_t* __restrict__ seg_idx, FastView fv,
                   int k, unsigned long long* __restrict__ partial, int* __restrict__ status,
                   SliceArgs sl, const __grid_constant__ FastTopParams top) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ ProblemTerms s_pt;
  __shared__ unsigned long long s_warp[kFastThreads / 32 * KS_MAX_K];
  __shared__ unsigned long long s_list[KS_MAX_K];
  __shared__ __align__(8) unsigned long long s_bar[kNBuf];
  __shared__ uint8_t s_row0[64], s_rowcnt[64], s_pbin[64];
  __shared__ float s_pfeat[64];
  __shared__ int s_fail, s_last, s_done[kNBuf], s_abort;

  const int tid = threadIdx.x;
  const int S = sl.n_slices;
  const int prob = blockIdx.x / (nblk * S), chunk = (blockIdx.x / S) % nblk, slice = blockIdx.x % S;
  if (tid == 0) s_abort = *reinterpret_cast<volatile int*>(&g_fast_abort);
  __syncthreads();
  if (s_abort) {  // a wait ran out in an earlier CTA of this launch: the call fails, leave at once
    if (tid < k && slice == 0) partial[(static_cast<size_t>(prob) * nblk + chunk) * k + tid] = 0ull;
    return;
  }
  int64_t lo, len;
  if (seg_off) {
    lo = seg_off[prob];
    len = seg_off[prob + 1] - lo;
  } else {
    lo = static_cast<int64_t>(prob) * C;
    len = C;
  }
  // chunks of the ensemble this CTA walks
  const int ch_begin = static_cast<int>(static_cast<int64_t>(fv.n_chunks) * slice / S);
  const int ch_end = static_cast<int>(static_cast<int64_t>(fv.n_chunks) * (slice + 1) / S);
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bar0 = smem_u32(&s_bar[0]);  // barrier of buffer b: bar0 + 8 b
  const bool tiles_given = sl.tiles != nullptr;  // the tiles were built in front: no feature work here
  if (tid == 0) {
    if (!tiles_given) {
      problem_terms(use_value ? p_value : p[prob], desc, s_pt);
      // problem-only columns do not look at the candidate: evaluate them on a dummy one
      ks_candidate dummy{};
      dummy.tile_m = dummy.tile_n = dummy.tile_k = 64;
      dummy.stages = dummy.cluster_m = dummy.cluster_n = 1;
      featurize_pair(s_pt, dummy, desc, [&](int col, float v) {
        if (feat_class(col) == 0) s_pfeat[col] = v;
      });
    }
    for (int b = 0; b < kNBuf; ++b) mbar_init(bar0 + 8u * b, 1);
    s_fail = 0;
    for (int b = 0; b < kNBuf; ++b) s_done[b] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < 64) {
    s_row0[tid] = fv.feat_row0[tid];
    s_rowcnt[tid] = fv.feat_rowcnt[tid];
  }
  if (tid < KS_MAX_K) s_list[tid] = 0ull;
  __syncthreads();
  if (!tiles_given && tid < KS_F && feat_class(tid) == 0) {
    const int first = fv.n_pair_rows + fv.n_cand_rows;
    for (int q = 0; q < s_rowcnt[tid]; ++q)
      s_pbin[s_row0[tid] + q - first] =
          static_cast<uint8_t>(0x80 | row_bin(fv.thr + (s_row0[tid] + q) * kThrPerRow, s_pfeat[tid]));
  }
  uint32_t phases = 0;  // bit b: parity of buffer b's barrier
  const int word = tid % kWords, half = tid / kWords;

  for (int64_t start = static_cast<int64_t>(chunk) * rows_per_cta; start < len;
       start += static_cast<int64_t>(nblk) * rows_per_cta) {
    const int64_t stop = (start + rows_per_cta < len) ? start + rows_per_cta : len;
    // ---- phase A ---------------------------------------------------------------------------------
    __syncthreads();
    if (sl.tiles) {
      // single-problem call: the block's tile was built once for all the CTAs that share it
      const uint4* src = reinterpret_cast<const uint4*>(sl.tiles + static_cast<size_t>(chunk) * fv.n_rows * kRowStride);
      uint4* dst = reinterpret_cast<uint4*>(smem + kOffTile);
      for (int i = tid; i < fv.n_rows * (kRowStride / 16); i += kFastThreads) dst[i] = __ldcg(src + i);
    } else {
      {
        float4* dst = reinterpret_cast<float4*>(smem + kOffBuf0);
        const float4* src = reinterpret_cast<const float4*>(fv.thr);
        for (int i = tid; i < fv.n_pair_rows * kThrPerRow / 4; i += kFastThreads) dst[i] = __ldg(src + i);
      }
      __syncthreads();
      fill_tile(desc, s_pt, c, fv, seg_off, seg_idx, C, lo, start, stop,
                reinterpret_cast<const float*>(smem + kOffBuf0), s_row0, s_rowcnt, s_pbin, smem + kOffTile, prob);
    }
    __syncthreads();  // tile complete; the threshold table is no longer needed

    // ---- phase B ---------------------------------------------------------------------------------
    if (tid == 0) {
      fence_async_proxy();
      const char* src = reinterpret_cast<const char*>(fv.chunks) + static_cast<size_t>(ch_begin) * fv.chunk_bytes;
      for (int b = 0; b < kNBuf && ch_begin + b < ch_end; ++b) {
        mbar_expect_tx(bar0 + 8u * b, fv.chunk_bytes);
        bulk_copy_g2s(sbase + kOffBuf0 + b * kBufBytes, src + static_cast<size_t>(b) * fv.chunk_bytes, fv.chunk_bytes,
                      bar0 + 8u * b);
      }
    }
    float score[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    const uint32_t cb = sbase + kOffTile + word * 4;
    const int tpc = fv.tpc, half_trees = tpc / 2;
    const int np = NP >= 0 ? NP : fv.depth - L;
    constexpr int kTop = (1 << L) - 1;
#pragma unroll 1
    for (int ch = ch_begin; ch < ch_end; ++ch) {
      const int b = (ch - ch_begin) % kNBuf;
      const uint32_t bar = bar0 + 8u * b;
      const uint32_t par = (phases >> b) & 1u;
      // after one wait has run out the CTA stops waiting (and refilling): the call fails, and
      // the CTAs that start later leave at once
      if (*reinterpret_cast<volatile int*>(&s_fail) || !mbar_wait_bounded(bar, par)) {
        if (!*reinterpret_cast<volatile int*>(&s_fail)) {
          s_fail = 1;
          atomicExch(&g_fast_abort, 1);
          if (status) atomicExch(status, KS_ERR_TIMEOUT);
        }
      }
      phases ^= 1u << b;
      const uint32_t buf = sbase + kOffBuf0 + b * kBufBytes;
      // With A_l the shared address of a walk's node at level l, A_{l+1} = 2 A_l + (4 tpc - buf)
      // + 4 bit for every level, and after the last level A points at the walk's leaf.
      const uint32_t k0 = 4u * tpc - buf;  // modulo 2^32, like the additions it enters
      const uint32_t lvlL = buf + 4u * tpc * kTop;  // first node of level L
      const int t_first = half * half_trees;
#pragma unroll 4
      for (int tt = 0; tt < half_trees; ++tt) {
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
            const uint32_t* tw = reinterpret_cast<const uint32_t*>(top.w) + static_cast<size_t>(ch * tpc + t) * kTop;
#pragma unroll
            for (int n = 0; n < kTop; ++n) {
              const uint32_t v = tw[n];
              d[n] = lds_u32(cb + (v >> 8)) - __byte_perm(v, 0u, 0u);
            }
          } else {
            const uint2* tw = top.w + static_cast<size_t>(ch * tpc + t) * kTop;
#pragma unroll
            for (int n = 0; n < kTop; ++n) d[n] = lds_u32(cb + tw[n].x) - tw[n].y;
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
            for (int r = 0; r < 4; ++r) a[r] = path_step(a[r], cb + r, k0);
        } else {
#pragma unroll 1
          for (int l = 0; l < np; ++l)
#pragma unroll
            for (int r = 0; r < 4; ++r) a[r] = path_step(a[r], cb + r, k0);
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) score[r] += lds_f32(a[r]);
      }
      // Release the buffer without a block-wide barrier: every warp counts itself out, and the
      // last one to leave refills the buffer (nobody waits; warps may run a chunk ahead).
      __syncwarp();
      if ((tid & 31) == 0) {
        if (atomicAdd(&s_done[b], 1) == kFastThreads / 32 - 1) {
          s_done[b] = 0;
          if (ch + kNBuf < ch_end && !s_fail) {
            fence_async_proxy();
            mbar_expect_tx(bar, fv.chunk_bytes);
            bulk_copy_g2s(buf, reinterpret_cast<const char*>(fv.chunks) + static_cast<size_t>(ch + kNBuf) * fv.chunk_bytes,
                          fv.chunk_bytes, bar);
          }
        }
      }
    }
    __syncthreads();  // all walks are done: the buffers are free

    // ---- phase C ---------------------------------------------------------------------------------
    float* s_part = reinterpret_cast<float*>(smem + kOffBuf0);  // [4][kWords], buffers are idle now
    if (half == 1) {
#pragma unroll
      for (int r = 0; r < 4; ++r) s_part[r * kWords + word] = score[r];
    }
    __syncthreads();
    if (sl.score_out) {
      // scoring call: the scores are the result (same order of additions as the ranking path)
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int64_t row = start + static_cast<int64_t>(r & 1) * kFastThreads + word + kWords * (r >> 1);
        if (half == 0 && row < stop)
          sl.score_out[lo + row] = ((fv.base + score[r]) + s_part[r * kWords + word]) + 0.0f;
      }
      continue;
    }
    if (S > 1) {
      // slice mode: publish this CTA's partial scores, let the last arrival finish the block
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int64_t row = start + static_cast<int64_t>(r & 1) * kFastThreads + word + kWords * (r >> 1);
        if (half == 0 && row < stop)
          __stcg(sl.scores + static_cast<size_t>(slice) * sl.pairs + lo + row, score[r] + s_part[r * kWords + word]);
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
      // byte r of word `word` belongs to phase-A thread word + kWords * (r / 2), candidate r % 2
      const int64_t row = start + static_cast<int64_t>(r & 1) * kFastThreads + word + kWords * (r >> 1);
      if (half == 0 && row < stop) {
        float s;
        if (S > 1) {
          s = fv.base;
          for (int q = 0; q < S; ++q) s += __ldcg(sl.scores + static_cast<size_t>(q) * sl.pairs + lo + row);
        } else {
          s = (fv.base + score[r]) + s_part[r * kWords + word];
        }
        keys[r] = make_key(s + 0.0f, seg_off ? seg_idx[lo + row] : static_cast<int>(row));
      }
    }
    keys[4] = tid < k ? s_list[tid] : 0ull;
    __syncthreads();
    block_topk<5>(keys, k, s_warp, s_list);
  }
  if (tid < k) partial[(static_cast<size_t>(prob) * nblk + chunk) * k + tid] = s_list[tid];
  if (S > 1 && sl.out_idx) {
    // single-problem form: the last block to finish merges the per-block lists (one warp)
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = atomicAdd(sl.counters + nblk, 1) == nblk - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (tid < 32) {
      const int n_keys = nblk * k;
      unsigned long long prev = ~0ull;
      for (int j = 0; j < k; ++j) {
        unsigned long long best = 0ull;
        for (int i = tid; i < n_keys; i += 32) {
          const unsigned long long v = __ldcg(partial + i);
          if (v < prev && v > best) best = v;
        }
        best = warp_max_u64(best);
        if (tid == 0) {
          sl.out_idx[j] = key_index(best);
          sl.out_score[j] = key_score(best);
        }
        prev = best;
      }
    }
    if (tid == 0) {
      sl.counters[nblk] = 0;
      if (sl.out_seq) {  // the results are in place: tell the host, which polls this word
        __threadfence_system();
        *reinterpret_cast<volatile int*>(sl.out_seq) = sl.seq;
      }
    }
  }
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
  std::vector<uint8_t> row0(64, 0), rowcnt(64, 0);
  int rank_row[KS_F][3];  // row offset (within the feature's rows) of each permutation in use
  int n_rows = 0, n_class[3] = {0, 0, 0};
  for (int f = 0; f < KS_F; ++f) {
    auto& v = thr[f];
    std::sort(v.begin(), v.end());
    v.erase(std::unique(v.begin(), v.end()), v.end());
    int cnt = static_cast<int>((v.size() + 126) / 127);
    for (int q = 0; q < 3; ++q) rank_row[f][q] = perm_used[f][q] ? cnt++ : -1;
    rowcnt[f] = static_cast<uint8_t>(cnt);
    n_class[feat_class(f)] += cnt;
    n_rows += cnt;
  }
  if (n_rows == 0 || n_rows > kMaxRows || n_class[1] > kCandRec) return cudaSuccess;  // generic path
  // rows ordered: per-pair, candidate-only, problem-only
  std::vector<float> table(static_cast<size_t>(n_rows) * kThrPerRow, std::numeric_limits<float>::infinity());
  int next = 0;
  for (int cls : {2, 1, 0}) {
    for (int f = 0; f < KS_F; ++f) {
      if (feat_class(f) != cls) continue;
      row0[f] = static_cast<uint8_t>(next);
      const int n_thr_rows = static_cast<int>((thr[f].size() + 126) / 127);
      for (int q = 0; q < n_thr_rows; ++q, ++next)
        for (int j = 0; j < 127; ++j) {
          const size_t s = static_cast<size_t>(q) * 127 + j;
          if (s < thr[f].size()) table[static_cast<size_t>(next) * kThrPerRow + j] = thr[f][s];
        }
      for (int q = 0; q < 3; ++q) {  // rank rows: slot c = rank of level c, last slot = marker
        if (rank_row[f][q] < 0) continue;
        const int L = categorical_levels(f);
        float* row = table.data() + static_cast<size_t>(next) * kThrPerRow;
        for (int c = 0; c < 4; ++c) row[c] = 0.0f;
        for (int r = 0; r < L; ++r) row[partition_perm(L, q)[r]] = static_cast<float>(r);
        row[kThrPerRow - 1] = -std::numeric_limits<float>::infinity();
        ++next;
      }
    }
  }
  const int per_tree_words = (2 << D) - 1;
  int tpc = kBufBytes / (per_tree_words * 4) / 2 * 2;  // even: the two halves of a CTA share a chunk's trees
  if (tpc < 2) return cudaSuccess;
  if (tpc > (n_trees + 1) / 2 * 2) tpc = (n_trees + 1) / 2 * 2;  // a small ensemble is one short chunk
  const int n_chunks = (n_trees + tpc - 1) / tpc;
  const int chunk_words = (tpc * per_tree_words + 3) / 4 * 4;  // bulk copies move multiples of 16 bytes
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
                  row = row0[nd.feat] + rank_row[nd.feat][pc.perm];
                  jl = pc.cut - 1;
                  swap = pc.swap;
                }
              } else {
                const auto& v = thr[nd.feat];
                const int j = static_cast<int>(std::lower_bound(v.begin(), v.end(), nd.thr_or_leaf) - v.begin());
                row = row0[nd.feat] + j / 127;
                jl = j % 127;
              }
              ls = nd.left;
              rs = nd.left + 1;
              if (always_right) {
                ls = rs;  // the walk always goes left here: put the right subtree on both sides
              } else {
                word = (row * kRowStride) << 8 | (0x80u | jl);
                tw = make_uint2(row * kRowStride, (jl + 1) * 0x01010101u);
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
  if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&m.d_qrow0), 64);
  if (e == cudaSuccess) e = cudaMemcpy(m.d_qrow0, row0.data(), 64, cudaMemcpyHostToDevice);
  if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&m.d_qrowcnt), 64);
  if (e == cudaSuccess) e = cudaMemcpy(m.d_qrowcnt, rowcnt.data(), 64, cudaMemcpyHostToDevice);
  if (e != cudaSuccess) {
    delete top;
    return e;
  }
  m.h_top = top;
  m.top_levels = L;
  m.top_compact = compact;
  m.fast = true;
  m.fast_depth = D;
  m.n_qrows = n_rows;
  m.n_pair_rows = n_class[2];
  m.n_cand_rows = n_class[1];
  m.n_prob_rows = n_class[0];
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

// Blocks per problem: full tiles of kFastRows rows. A block's cost does not depend on how many
// of its slots are live, so an under-filled machine is filled by splitting the trees over
// several CTAs per block (slices) rather than by shorter blocks.
void fast_tiling(int P, int64_t per_problem, int* nblk, int* rows_per_cta) {
  int64_t n = (per_problem + kFastRows - 1) / kFastRows;
  if (n < 1) n = 1;
  (void)P;
  *nblk = static_cast<int>(n);
  *rows_per_cta = kFastRows;
}

size_t fast_scratch_bytes(int C) { return 256 + static_cast<size_t>(kCombos) * C * kCandRec; }

// Memo of the per-pair rows (see MemoView): worth its per-problem table only for a batch of
// problems, and only when the per-pair rows fit a record. 0 = not used.
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

size_t fast_memo_bytes(const GbdtModel& g, int P, int C) {
  if (P < kMemoMinProblems || P > kMemoMaxProblems || C < 1 || g.n_pair_rows < 1 || g.n_pair_rows > kMemoRec) return 0;
  return memo_fixed_bytes(C) + static_cast<size_t>(P) * kMemoCap * kMemoRec;
}

// Slice count of the single-problem call: as many tree slices as keep every CTA in the first
// wave (one CTA per SM).
int fast_slices(const GbdtModel& g, int64_t blocks) {
  if (blocks < 1) blocks = 1;
  if (blocks > kMaxSliceBlocks) return 1;
  int64_t s = 296 / blocks;
  if (s > g.n_chunks) s = g.n_chunks;
  return static_cast<int>(s < 1 ? 1 : s);
}

template <int L, int NP, bool kCompact = false>
static cudaError_t launch_ln(const ks_gpu_desc& desc, const ks_problem* d_p, const ks_problem& pv, int uv, int P,
                             const ks_candidate* d_c, int C, int nblk, int rows_per_cta, const int64_t* seg_off,
                             const int32_t* seg_idx, const FastView& fv, int k, unsigned long long* partial,
                             int* status, const SliceArgs& sl, const FastTopParams& top, cudaStream_t stream) {
  const size_t smem = kOffTile + static_cast<size_t>(fv.n_rows) * kRowStride;
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(&select_fast_kernel<L, NP, kCompact>), smem);
  if (e != cudaSuccess) return e;
  select_fast_kernel<L, NP, kCompact><<<static_cast<unsigned>(static_cast<int64_t>(P) * nblk * sl.n_slices), kFastThreads, smem,
                              stream>>>(desc, d_p, pv, uv, d_c, P, C, nblk, rows_per_cta, seg_off, seg_idx, fv, k,
                                        partial, status, sl, top);
  return cudaGetLastError();
}

cudaError_t launch_select_fast(const ks_gpu_desc& desc, const GbdtModel& g, const ks_problem* d_p,
                               const ks_problem* p_by_value, int P, const ks_candidate* d_c, int C,
                               int nblk, int rows_per_cta, const int64_t* seg_off, const int32_t* seg_idx,
                               int k, unsigned long long* partial, void* scratch, int* status,
                               cudaStream_t stream, int64_t* launches, cudaEvent_t ev_begin,
                               const FastSlice* slice, void* memo_mem) {
  ks_problem pv{};
  if (p_by_value) pv = *p_by_value;
  const int uv = p_by_value != nullptr;
  FastView fv;
  fv.n_rows = g.n_qrows;
  fv.n_pair_rows = g.n_pair_rows;
  fv.n_cand_rows = g.n_cand_rows;
  fv.n_prob_rows = g.n_prob_rows;
  fv.depth = g.fast_depth;
  fv.n_chunks = g.n_chunks;
  fv.chunk_bytes = g.chunk_bytes;
  fv.tpc = g.tpc;
  fv.base = g.base;
  fv.chunks = g.d_qnodes;
  fv.thr = g.d_qthr;
  fv.feat_row0 = g.d_qrow0;
  fv.feat_rowcnt = g.d_qrowcnt;
  unsigned* d_mask = static_cast<unsigned*>(scratch);
  uint8_t* d_rows = static_cast<uint8_t*>(scratch) + 256;
  fv.cand_rows = d_rows;
  fv.pair_class = nullptr;
  fv.pair_tab = nullptr;
  MemoView memo{};
  if (memo_mem && !p_by_value && fast_memo_bytes(g, P, C) != 0) memo = memo_view(memo_mem, C);

  // candidate-only rows for the type combinations in use
  cudaError_t e = cudaSuccess;
  unsigned mask_value = 0;
  if (uv) {
    mask_value = 1u << ((pv.dtype_ab & 3) * 4 + (pv.dtype_d & 3));
  } else {
    e = cudaMemsetAsync(d_mask, 0, sizeof(unsigned), stream);
    if (e != cudaSuccess) return e;
    combo_mask_kernel<<<P >= 4096 ? 16 : 1, 256, 0, stream>>>(d_p, P, d_mask);
    ++*launches;
  }
  const bool tiles_mode = uv && slice && slice->n_slices > 1 && slice->tiles && P == 1 && !seg_off;
  if (tiles_mode) {
    // one launch, two roles (blockIdx.y): the per-pair rows, and the candidate- / problem-only rows
    const size_t tthr = sizeof(float) * kThrPerRow * g.n_qrows;
    e = ensure_dynamic_smem(reinterpret_cast<const void*>(&tile_one_kernel), tthr);
    if (e != cudaSuccess) return e;
    tile_one_kernel<<<dim3(nblk * (kFastRows / 256), 2), 256, tthr, stream>>>(desc, pv, d_c, C, fv, slice->tiles);
    ++*launches;
  } else if (C > 0) {
    const size_t cthr = sizeof(float) * kThrPerRow * (g.n_cand_rows > 0 ? g.n_cand_rows : 1);
    if (memo.keys) {
      e = memo_clear(memo, stream);
      if (e != cudaSuccess) return e;
    }
    cand_rows_kernel<<<dim3((C + 255) / 256, kCombos), 256, cthr, stream>>>(desc, d_c, C, uv ? nullptr : d_mask,
                                                                            mask_value, fv, d_rows, memo);
    ++*launches;
    if (memo.keys) {
      const size_t pthr = sizeof(float) * kThrPerRow * g.n_pair_rows;
      e = ensure_dynamic_smem(reinterpret_cast<const void*>(&pair_table_kernel), pthr);
      if (e != cudaSuccess) return e;
      e = memo_compact(memo, stream);
      if (e != cudaSuccess) return e;
      pair_table_kernel<<<dim3(kMemoCap / 256, P), 256, pthr, stream>>>(desc, d_p, d_c, fv, memo);
      *launches += 2;
      fv.pair_class = memo.cls;
      fv.pair_tab = static_cast<const uint8_t*>(memo.tab);
    }
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (ev_begin) cudaEventRecord(ev_begin, stream);

  SliceArgs sl{};
  sl.n_slices = 1;
  if (slice && slice->n_slices > 1) {
    sl.n_slices = slice->n_slices;
    sl.pairs = slice->pairs;
    sl.scores = slice->scores;
    sl.counters = slice->counters;
    sl.out_idx = slice->out_idx;
    sl.out_score = slice->out_score;
    sl.tiles = tiles_mode ? slice->tiles : nullptr;
    sl.out_seq = slice->out_seq;
    sl.seq = slice->seq;
  }
  const FastTopParams& top = *g.h_top;
  const int L = g.top_levels, np = g.fast_depth - L;
  ++*launches;
#define KS_GO(LL, NN) \
  return launch_ln<LL, NN>(desc, d_p, pv, uv, P, d_c, C, nblk, rows_per_cta, seg_off, seg_idx, fv, k, partial, status, sl, top, stream)
  if (g.top_compact) {
#define KS_GOC(NN) \
  return launch_ln<3, NN, true>(desc, d_p, pv, uv, P, d_c, C, nblk, rows_per_cta, seg_off, seg_idx, fv, k, partial, status, sl, top, stream)
    if (np == 5) KS_GOC(5);
    if (np == 4) KS_GOC(4);
    KS_GOC(-1);
#undef KS_GOC
  }
  if (L == 3 && np == 5) KS_GO(3, 5);
  if (L == 3 && np == 3) KS_GO(3, 3);
  if (L == 2 && np == 6) KS_GO(2, 6);
  if (L == 2 && np == 5) KS_GO(2, 5);  // the paper-sized ensemble: 916 trees of depth 7
  if (L == 3 && np == 4) KS_GO(3, 4);
  if (L == 3) KS_GO(3, -1);
  if (L == 2) KS_GO(2, -1);
  if (L == 1) KS_GO(1, -1);
  KS_GO(0, -1);
#undef KS_GO
}

// ks_score on the quantised path. Rows are taken in batches so that the tiles (n_rows bytes per
// row) stay a bounded workspace; every batch is one tile launch and one walk launch.
constexpr int64_t kScoreBatchBlocks = 4096;

size_t score_fast_scratch_bytes(const GbdtModel& g, int64_t rows) {
  int64_t blocks = (rows + kFastRows - 1) / kFastRows;
  if (blocks > kScoreBatchBlocks) blocks = kScoreBatchBlocks;
  return static_cast<size_t>(blocks) * g.n_qrows * kRowStride;
}

cudaError_t launch_score_fast(const ks_gpu_desc& desc, const GbdtModel& g, const float* d_feat, int64_t rows,
                              float* d_scores, void* scratch, int* status, cudaStream_t stream,
                              int64_t* launches) {
  FastView fv{};
  fv.n_rows = g.n_qrows;
  fv.n_pair_rows = g.n_pair_rows;
  fv.n_cand_rows = g.n_cand_rows;
  fv.n_prob_rows = g.n_prob_rows;
  fv.depth = g.fast_depth;
  fv.n_chunks = g.n_chunks;
  fv.chunk_bytes = g.chunk_bytes;
  fv.tpc = g.tpc;
  fv.base = g.base;
  fv.chunks = g.d_qnodes;
  fv.thr = g.d_qthr;
  fv.feat_row0 = g.d_qrow0;
  fv.feat_rowcnt = g.d_qrowcnt;
  uint8_t* tiles = static_cast<uint8_t*>(scratch);
  const size_t tthr = sizeof(float) * kThrPerRow * g.n_qrows;
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(&tile_rows_kernel), tthr);
  if (e != cudaSuccess) return e;
  const FastTopParams& top = *g.h_top;
  const int L = g.top_levels, np = g.fast_depth - L;
  const ks_problem pv{};
  for (int64_t first = 0; first < rows; first += kScoreBatchBlocks * kFastRows) {
    const int64_t n = rows - first < kScoreBatchBlocks * kFastRows ? rows - first : kScoreBatchBlocks * kFastRows;
    const int nblk = static_cast<int>((n + kFastRows - 1) / kFastRows);
    tile_rows_kernel<<<nblk, kWords, tthr, stream>>>(d_feat + first * KS_F_PAD, n, fv, tiles);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    SliceArgs sl{};
    sl.n_slices = 1;
    sl.tiles = tiles;
    sl.score_out = d_scores + first;
    *launches += 2;
#define KS_GO(LL, NN)                                                                                          \
  e = launch_ln<LL, NN>(desc, nullptr, pv, 1, 1, nullptr, static_cast<int>(n), nblk, kFastRows, nullptr, nullptr, \
                        fv, 0, nullptr, status, sl, top, stream)
    if (g.top_compact && np == 5) e = launch_ln<3, 5, true>(desc, nullptr, pv, 1, 1, nullptr, static_cast<int>(n), nblk, kFastRows, nullptr, nullptr, fv, 0, nullptr, status, sl, top, stream);
    else if (g.top_compact && np == 4) e = launch_ln<3, 4, true>(desc, nullptr, pv, 1, 1, nullptr, static_cast<int>(n), nblk, kFastRows, nullptr, nullptr, fv, 0, nullptr, status, sl, top, stream);
    else if (g.top_compact) e = launch_ln<3, -1, true>(desc, nullptr, pv, 1, 1, nullptr, static_cast<int>(n), nblk, kFastRows, nullptr, nullptr, fv, 0, nullptr, status, sl, top, stream);
    else if (L == 3 && np == 5) KS_GO(3, 5);
    else if (L == 3 && np == 3) KS_GO(3, 3);
    else if (L == 2 && np == 6) KS_GO(2, 6);
    else if (L == 2 && np == 5) KS_GO(2, 5);
    else if (L == 3 && np == 4) KS_GO(3, 4);
    else if (L == 3) KS_GO(3, -1);
    else if (L == 2) KS_GO(2, -1);
    else if (L == 1) KS_GO(1, -1);
    else KS_GO(0, -1);
#undef KS_GO
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace ks
