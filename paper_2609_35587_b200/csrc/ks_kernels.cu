// Generic kernels of libks: the standalone feature map, the standalone scorers, the generic
// fused featurize + score + top-k kernel (any tree shape, any MLP the ABI accepts) and the
// per-problem merge of partial top-k lists. The quantised fast path for complete trees lives
// in ks_gbdt_fast.cu.
#include <cuda_bf16.h>

#include <cstdlib>
#include <cstring>
#include <new>

#include "ks_features.cuh"
#include "ks_internal.h"
#include "ks_memo.cuh"
#include "ks_topk.cuh"

namespace ks {

// ------------------------------------------------------------------------------------------
// block -> (problem, chunk) mapping shared by the pair kernels
// ------------------------------------------------------------------------------------------

struct PairMap {
  int P, C, nblk;           // nblk blocks per problem
  int rows_per_block;       // rows one block covers per pass
  const int64_t* seg_off;   // null = dense
  const int32_t* seg_idx;
};

__device__ __forceinline__ void segment_of(const PairMap& m, int prob, int64_t& lo, int64_t& len) {
  if (m.seg_off) {
    lo = m.seg_off[prob];
    len = m.seg_off[prob + 1] - lo;
  } else {
    lo = static_cast<int64_t>(prob) * m.C;
    len = m.C;
  }
}

__device__ __forceinline__ int pool_index(const PairMap& m, int64_t lo, int64_t r) {
  return m.seg_off ? m.seg_idx[lo + r] : static_cast<int>(r);
}

// ------------------------------------------------------------------------------------------
// ks_featurize: one thread per pair, rows staged through shared memory for coalesced stores
// ------------------------------------------------------------------------------------------

__global__ void __launch_bounds__(kBlock)
featurize_kernel(ks_gpu_desc desc, const ks_problem* __restrict__ p, const ks_candidate* __restrict__ c,
                 PairMap map, float* __restrict__ out) {
  extern __shared__ float s_tile[];  // [kBlock][65]
  __shared__ ProblemTerms s_pt;
  const int prob = blockIdx.x / map.nblk, chunk = blockIdx.x % map.nblk;
  int64_t lo, len;
  segment_of(map, prob, lo, len);
  if (threadIdx.x == 0) problem_terms(p[prob], desc, s_pt);
  __syncthreads();
  // every warp stages and stores its own 32 rows, so that one warp's stores overlap another's
  // arithmetic without block-wide barriers
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float* w_tile = s_tile + warp * 32 * 65;
  for (int64_t start = static_cast<int64_t>(chunk) * kBlock; start < len;
       start += static_cast<int64_t>(map.nblk) * kBlock) {
    const int64_t w0 = start + warp * 32;  // first row of this warp
    if (w0 >= len) break;
    if (w0 + lane < len) {
      const ks_candidate cand = c[pool_index(map, lo, w0 + lane)];
      float* row = w_tile + lane * 65;
      featurize_pair(s_pt, cand, desc, [&](int col, float v) { row[col] = v; });
    }
    __syncwarp();
    const int n_rows = (len - w0 < 32) ? static_cast<int>(len - w0) : 32;
    float* dst = out + (lo + w0) * kRow;
    for (int i = lane; i < n_rows * kRow; i += 32) __stcs(dst + i, w_tile[(i >> 6) * 65 + (i & 63)]);
    __syncwarp();
  }
}

// Dense form (every problem against the whole pool). The work is cut into items of 32
// candidates x 1 problem, ordered candidate slab first, and every warp of the grid takes a
// contiguous run of items of equal length (to within one), so that no SM idles in a last
// partial wave. A lane keeps its candidate, the candidate-only columns and the candidate's
// resident-block count in registers while the problems of the run change (re-evaluated only
// when the element-type combination does); the problem-only terms and columns come from a
// table written once per call. Only the per-pair columns are arithmetic per pair. Same
// functions, same operands: the rows are bit-identical to featurize_pair's.
struct ProblemEntry {
  ProblemTerms t;
  float pc[16];  // the problem-only columns, in column order
};

__host__ __device__ constexpr int class_slot(int col) {
  int n = 0;
  for (int q = 0; q < col; ++q)
    if (feat_class(q) == feat_class(col)) ++n;
  return n;
}

__global__ void __launch_bounds__(128)
problem_table_kernel(ks_gpu_desc desc, const ks_problem* __restrict__ p, int P, ProblemEntry* __restrict__ tab) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= P) return;
  ProblemEntry e;
  problem_terms(p[i], desc, e.t);
  ks_candidate dummy{};
  dummy.tile_m = dummy.tile_n = dummy.tile_k = 64;
  dummy.stages = dummy.cluster_m = dummy.cluster_n = 1;
#pragma unroll
  for (int q = 0; q < 16; ++q) e.pc[q] = 0.0f;
  featurize_pair(e.t, dummy, desc, [&](int col, float v) {
    if (feat_class(col) == 0) e.pc[class_slot(col)] = v;
  });
  tab[i] = e;
}

__global__ void __launch_bounds__(kBlock, 3)
featurize_dense_kernel(ks_gpu_desc desc, const ProblemEntry* __restrict__ tab, const ks_candidate* __restrict__ c,
                       int P, int C, float* __restrict__ out) {
  extern __shared__ float s_tile[];  // [kBlock][65], one 32-row slab per warp
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float* row = s_tile + (warp * 32 + lane) * 65;
  const float* w_tile = s_tile + warp * 32 * 65;
  const int64_t n_warps = static_cast<int64_t>(gridDim.x) * (kBlock / 32);
  const int64_t me = static_cast<int64_t>(blockIdx.x) * (kBlock / 32) + warp;
  const int64_t total = static_cast<int64_t>((C + 31) / 32) * P;
  const int64_t i_end = total * (me + 1) / n_warps;
  ks_candidate cand{};
  float cc[29];
  long long b_eff = 1;
  int slab_prev = -1, combo_prev = -1, w0 = 0, n_rows = 0;
  bool live = false;
#pragma unroll 1
  for (int64_t i = total * me / n_warps; i < i_end; ++i) {
    const int slab = static_cast<int>(i / P), prob = static_cast<int>(i - static_cast<int64_t>(slab) * P);
    if (slab != slab_prev) {
      slab_prev = slab;
      combo_prev = -1;
      w0 = slab * 32;
      n_rows = C - w0 < 32 ? C - w0 : 32;
      live = lane < n_rows;
      cand = c[live ? w0 + lane : C - 1];
    }
    const ProblemEntry& e = tab[prob];
    const ProblemTerms t = e.t;
    const int combo = t.dtype_ab * 4 + t.dtype_d;
    if (combo != combo_prev) {  // the same for every lane
      combo_prev = combo;
      b_eff = resources(t, cand, desc).b_eff;
      featurize_pair(t, cand, desc, [&](int col, float v) {
        if (feat_class(col) == 1) cc[class_slot(col)] = v;
      });
    }
#pragma unroll
    for (int col = 0; col < KS_F; ++col) {
      if (feat_class(col) == 1) row[col] = cc[class_slot(col)];
      if (feat_class(col) == 0) row[col] = __ldg(&e.pc[class_slot(col)]);
    }
    row[KS_F] = 0.0f;
    pair_columns<true>(t, cand, desc, b_eff, [&](int col, float v) { row[col] = v; });
    __syncwarp();
    float* dst = out + (static_cast<int64_t>(prob) * C + w0) * kRow;
    for (int q = lane; q < n_rows * kRow; q += 32) __stcs(dst + q, w_tile[(q >> 6) * 65 + (q & 63)]);
    __syncwarp();
  }
}

// ------------------------------------------------------------------------------------------
// generic tree walk: nodes from global memory (read-only path), features from a shared tile
// laid out [column][thread] so that a warp's reads of one column are conflict-free
// ------------------------------------------------------------------------------------------

__device__ __forceinline__ DevNode load_node(const DevNode* p) {
  const uint2 u = __ldg(reinterpret_cast<const uint2*>(p));
  DevNode n;
  n.v = __uint_as_float(u.x);
  n.feat = static_cast<uint16_t>(u.y & 0xFFFFu);
  n.left = static_cast<uint16_t>(u.y >> 16);
  return n;
}

// returns base + sum of leaves; optionally records the leaf node index of every tree
__device__ __forceinline__ float walk_ensemble(const DevNode* __restrict__ nodes,
                                               const int* __restrict__ roots, int n_trees, float base,
                                               const float* s_cols /* [64][kBlock], this thread's lane */,
                                               uint16_t* leaf_out) {
  float s = base;
  for (int t = 0; t < n_trees; ++t) {
    const DevNode* tree = nodes + roots[t];
    int i = 0;
    DevNode nd = load_node(tree);
#pragma unroll 1
    for (int d = 0; d <= KS_MAX_DEPTH && nd.feat != 0xFFFFu; ++d) {
      const float x = s_cols[(nd.feat & 0x7FFFu) * kBlock];
      int right;
      if (nd.feat & 0x8000u) {  // partition split: v's bits are the set of levels that go right
        const unsigned code = static_cast<unsigned>(__float2int_rz(x));
        right = code < 32u ? (__float_as_uint(nd.v) >> code) & 1u : 0;
      } else {
        right = x < nd.v ? 0 : 1;
      }
      i = nd.left + right;
      nd = load_node(tree + i);
    }
    if (leaf_out) leaf_out[t] = static_cast<uint16_t>(i);
    s += nd.v;
  }
  return s;
}

__global__ void __launch_bounds__(kBlock)
score_gbdt_kernel(const DevNode* __restrict__ nodes, const int* __restrict__ roots, int n_trees,
                  float base, const float* __restrict__ feat, int64_t rows, float* __restrict__ scores,
                  uint16_t* __restrict__ leaf_idx) {
  extern __shared__ float s_cols[];  // [64][kBlock]
  const int64_t r = static_cast<int64_t>(blockIdx.x) * kBlock + threadIdx.x;
  if (r < rows) {
    const float4* src = reinterpret_cast<const float4*>(feat + r * kRow);
#pragma unroll 4
    for (int q = 0; q < kRow / 4; ++q) {
      const float4 v = __ldg(src + q);
      s_cols[(4 * q + 0) * kBlock + threadIdx.x] = v.x;
      s_cols[(4 * q + 1) * kBlock + threadIdx.x] = v.y;
      s_cols[(4 * q + 2) * kBlock + threadIdx.x] = v.z;
      s_cols[(4 * q + 3) * kBlock + threadIdx.x] = v.w;
    }
    const float s = walk_ensemble(nodes, roots, n_trees, base, s_cols + threadIdx.x,
                                  leaf_idx ? leaf_idx + r * n_trees : nullptr);
    scores[r] = s + 0.0f;
  }
}

// ------------------------------------------------------------------------------------------
// generic MLP on a tile of kBlock rows held as [column][thread] fp32 in shared memory.
// Rows are processed 32 at a time; thread (r = tid % 32, g = tid / 32) computes the outputs
// o = g, g + 8, ... of row r. Activations are bf16 in shared memory, [unit][32].
// ------------------------------------------------------------------------------------------

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }

__device__ void mlp_tile(const MlpView& m, int max_width, const float* s_cols /* [64][kBlock] */,
                         __nv_bfloat16* s_act /* [2][max_width][32] */, float* s_scores /* [kBlock] */) {
  const int r = threadIdx.x & 31, g = threadIdx.x >> 5;
  constexpr int kGroups = kBlock / 32;
  for (int grp = 0; grp < kGroups; ++grp) {
    __nv_bfloat16* cur = s_act;
    __nv_bfloat16* nxt = s_act + max_width * 32;
    const bool onehot = m.widths[0] == KS_F_ONEHOT;
    for (int pos = g; pos < m.widths[0]; pos += kGroups) {
      float v = 0.0f;
      bool live;
      if (!onehot) {
        live = pos < KS_F;
        if (live) v = s_cols[pos * kBlock + grp * 32 + r];
      } else {
        // one-hot form: the columns other than 5, 9, 17, 18 in order, then the level indicators
        live = pos < 73;
        if (pos < 59) {
          const int col = pos + (pos >= 5) + (pos >= 8) + 2 * (pos >= 15);
          v = s_cols[col * kBlock + grp * 32 + r];
        } else if (live) {
          const int q = pos - 59;  // operand type 0..3, activation 4..6, kernel sched 7..10, epilogue sched 11..13
          const int col = q < 4 ? 5 : (q < 7 ? 9 : (q < 11 ? 17 : 18));
          const int level = q < 4 ? q : (q < 7 ? q - 4 : (q < 11 ? q - 7 : q - 11));
          v = __float2int_rz(s_cols[col * kBlock + grp * 32 + r]) == level ? 1.0f : 0.0f;
        }
      }
      if (live) {
        if (!isfinite(v)) v = 0.0f;
        v = __fdiv_rn(__fsub_rn(v, m.mu[pos]), m.sigma[pos]);
      }
      cur[pos * 32 + r] = __float2bfloat16_rn(v);
    }
    __syncthreads();
    for (int l = 0; l < m.n_layers; ++l) {
      const int wi = m.widths[l], wo = m.widths[l + 1];
      const bool last = (l == m.n_layers - 1);
      for (int o = g; o < wo; o += kGroups) {
        const uint4* wrow = reinterpret_cast<const uint4*>(m.w[l] + static_cast<size_t>(o) * wi);
        float acc = 0.0f;
        for (int i8 = 0; i8 < wi / 8; ++i8) {
          const uint4 wv = __ldg(wrow + i8);
          const uint32_t ww[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const int i = i8 * 8 + 2 * q;
            acc = fmaf(bf16_bits_to_float(ww[q] & 0xFFFFu), __bfloat162float(cur[i * 32 + r]), acc);
            acc = fmaf(bf16_bits_to_float(ww[q] >> 16), __bfloat162float(cur[(i + 1) * 32 + r]), acc);
          }
        }
        float v = acc + m.b[l][o];
        if (last) {
          if (o == 0) s_scores[grp * 32 + r] = v;
        } else {
          nxt[o * 32 + r] = __float2bfloat16_rn(fmaxf(v, 0.0f));
        }
      }
      __syncthreads();
      __nv_bfloat16* tmp = cur;
      cur = nxt;
      nxt = tmp;
    }
  }
}

__global__ void __launch_bounds__(kBlock)
score_mlp_kernel(MlpView m, int max_width, const float* __restrict__ feat, int64_t rows,
                 float* __restrict__ scores) {
  extern __shared__ __align__(16) unsigned char s_raw[];
  float* s_cols = reinterpret_cast<float*>(s_raw);                       // [64][kBlock]
  float* s_scores = s_cols + kRow * kBlock;                              // [kBlock]
  __nv_bfloat16* s_act = reinterpret_cast<__nv_bfloat16*>(s_scores + kBlock);
  const int64_t r = static_cast<int64_t>(blockIdx.x) * kBlock + threadIdx.x;
  const float4* src = reinterpret_cast<const float4*>(feat + min(r, rows - 1) * kRow);
#pragma unroll 4
  for (int q = 0; q < kRow / 4; ++q) {
    const float4 v = __ldg(src + q);
    s_cols[(4 * q + 0) * kBlock + threadIdx.x] = v.x;
    s_cols[(4 * q + 1) * kBlock + threadIdx.x] = v.y;
    s_cols[(4 * q + 2) * kBlock + threadIdx.x] = v.z;
    s_cols[(4 * q + 3) * kBlock + threadIdx.x] = v.w;
  }
  __syncthreads();
  mlp_tile(m, max_width, s_cols, s_act, s_scores);
  if (r < rows) scores[r] = s_scores[threadIdx.x] + 0.0f;
}

// ------------------------------------------------------------------------------------------
// generic fused select: featurize a sub-tile of kBlock pairs into shared memory, score it,
// keep one key per thread per sub-tile, rank the block's keys, write a partial top-k list.
// ------------------------------------------------------------------------------------------

template <int kModel>  // 0 = tree ensemble, 1 = MLP, 2 = static sampling score (no feature tile)
__global__ void __launch_bounds__(kBlock)
select_generic_kernel(ks_gpu_desc desc, const ks_problem* __restrict__ p, ks_problem p_value,
                      int use_value, const ks_candidate* __restrict__ c, PairMap map, int sub_tiles,
                      const DevNode* __restrict__ nodes, const int* __restrict__ roots, int n_trees,
                      float base, MlpView mlp, int max_width, int k,
                      unsigned long long* __restrict__ partial /* [P][nblk][k] */) {
  extern __shared__ __align__(16) unsigned char s_raw[];
  float* s_cols = reinterpret_cast<float*>(s_raw);  // [64][kBlock]
  float* s_scores = s_cols + kRow * kBlock;         // [kBlock] (MLP only)
  __nv_bfloat16* s_act = reinterpret_cast<__nv_bfloat16*>(s_scores + kBlock);
  __shared__ ProblemTerms s_pt;
  __shared__ unsigned long long s_warp[kBlock / 32 * KS_MAX_K];
  __shared__ unsigned long long s_list[KS_MAX_K];

  const int prob = blockIdx.x / map.nblk, chunk = blockIdx.x % map.nblk;
  int64_t lo, len;
  segment_of(map, prob, lo, len);
  if (threadIdx.x == 0) problem_terms(use_value ? p_value : p[prob], desc, s_pt);
  if (threadIdx.x < KS_MAX_K) s_list[threadIdx.x] = 0ull;
  __syncthreads();

  const int64_t pass_rows = static_cast<int64_t>(sub_tiles) * kBlock;
  for (int64_t start = static_cast<int64_t>(chunk) * pass_rows; start < len;
       start += static_cast<int64_t>(map.nblk) * pass_rows) {
    unsigned long long keys[kSubTilesMax + 1];
#pragma unroll
    for (int s = 0; s <= kSubTilesMax; ++s) keys[s] = 0ull;
    // carry the list of the previous pass in as extra keys
    if (threadIdx.x < k) keys[kSubTilesMax] = s_list[threadIdx.x];
#pragma unroll 1
    for (int s = 0; s < sub_tiles; ++s) {
      const int64_t r = start + static_cast<int64_t>(s) * kBlock + threadIdx.x;
      const bool live = r < len;
      int idx = 0;
      __syncthreads();  // previous sub-tile's readers are done with s_cols
      float direct = 0.0f;
      if (live) {
        idx = pool_index(map, lo, r);
        const ks_candidate cand = c[idx];
        if (kModel == 2) {
          direct = static_score(s_pt, cand, desc);
        } else {
          float* col0 = s_cols + threadIdx.x;
          featurize_pair(s_pt, cand, desc, [&](int col, float v) { col0[col * kBlock] = v; });
        }
      } else if (kModel == 1) {
        for (int col = 0; col < kRow; ++col) s_cols[col * kBlock + threadIdx.x] = 0.0f;
      }
      float score;
      if (kModel == 2) {
        score = direct;
      } else if (kModel == 0) {
        score = live ? walk_ensemble(nodes, roots, n_trees, base, s_cols + threadIdx.x, nullptr) : 0.0f;
      } else {
        __syncthreads();
        mlp_tile(mlp, max_width, s_cols, s_act, s_scores);
        score = s_scores[threadIdx.x];
      }
      const unsigned long long key = live ? make_key(score + 0.0f, idx) : 0ull;
#pragma unroll
      for (int q = 0; q < kSubTilesMax; ++q)
        if (q == s) keys[q] = key;
    }
    block_topk<kSubTilesMax + 1>(keys, k, s_warp, s_list);
  }
  if (threadIdx.x < k)
    partial[(static_cast<size_t>(prob) * map.nblk + chunk) * k + threadIdx.x] = s_list[threadIdx.x];
}

// ------------------------------------------------------------------------------------------
// linear scorer (one weight layer): s = b + sum_j w_j * bf16((x_j - mu_j) / sigma_j). The sum
// splits by what a column depends on: the candidate-only part is formed once per call and
// candidate (per element-type combination), the problem-only part once per block, and only the
// 21 per-pair columns are evaluated per pair, without a feature tile.
// ------------------------------------------------------------------------------------------

__device__ __forceinline__ float ridge_term(const RidgeParams& prm, int col, float v) {
  if (!isfinite(v)) v = 0.0f;
  const float x = __bfloat162float(__float2bfloat16_rn(__fdiv_rn(__fsub_rn(v, prm.mu[col]), prm.sigma[col])));
  return prm.w[col] * x;
}
__device__ __forceinline__ float ridge_level(const float (&lut)[4], float v) {
  const int code = __float2int_rz(v);
  return (code >= 0 && code < 4) ? lut[code] : 0.0f;
}

// per (type combination, candidate): (candidate-only part of the sum, resident-block count)
__global__ void __launch_bounds__(256)
ridge_cand_kernel(ks_gpu_desc desc, const ks_candidate* __restrict__ c, int C, const unsigned* mask_ptr,
                  unsigned mask_value, const __grid_constant__ RidgeParams prm, float2* __restrict__ out,
                  MemoView memo) {
  const int combo = blockIdx.y;
  const unsigned mask = mask_ptr ? *mask_ptr : mask_value;
  if (!((mask >> combo) & 1u)) return;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= C) return;
  ks_problem fake{};
  fake.m = fake.n = fake.k = 1;
  fake.dtype_ab = static_cast<uint8_t>(combo >> 2);
  fake.dtype_d = static_cast<uint8_t>(combo & 3);
  ProblemTerms t;
  problem_terms(fake, desc, t);
  const ks_candidate cand = c[i];
  float s = 0.0f;
  featurize_pair(t, cand, desc, [&](int col, float v) {
    if (feat_class(col) != 1) return;
    s += ridge_term(prm, col, v);
    if (col == 17) s += ridge_level(prm.lut17, v);
    if (col == 18) s += ridge_level(prm.lut18, v);
  });
  const long long b_eff = resources(t, cand, desc).b_eff;
  out[static_cast<size_t>(combo) * C + i] = make_float2(s, static_cast<float>(b_eff));
  if (memo.keys) memo.cls[static_cast<size_t>(combo) * C + i] = memo_assign(memo, combo, i, cand, b_eff);
}

// Per (problem, class): the per-pair part of the sum, from the class's member (classes:
// ks_memo.cuh). grid (kMemoCap / 256, P); blocks past the number of classes leave at once.
__global__ void __launch_bounds__(256)
ridge_pair_kernel(ks_gpu_desc desc, const ks_problem* __restrict__ p, const ks_candidate* __restrict__ c,
                  const float2* __restrict__ cand_tab, int C, const __grid_constant__ RidgeParams prm, MemoView memo) {
  __shared__ ProblemTerms s_pt;
  const int prob = blockIdx.y, j = blockIdx.x * 256 + threadIdx.x;
  const ks_problem pr = p[prob];
  const int combo = (pr.dtype_ab & 3) * 4 + (pr.dtype_d & 3);
  const int n_classes = memo.count[combo];
  if (blockIdx.x * 256 >= n_classes) return;
  if (threadIdx.x == 0) problem_terms(pr, desc, s_pt);
  __syncthreads();
  if (j >= n_classes) return;
  const int slot = memo.dense[static_cast<size_t>(combo) * kMemoCap + j];
  const int rep = memo.reps[static_cast<size_t>(combo) * kMemoCap + slot];
  const ks_candidate cand = c[rep];
  const float2 t = __ldg(cand_tab + static_cast<size_t>(combo) * C + rep);
  float pair = 0.0f;
  pair_columns<true>(s_pt, cand, desc, static_cast<long long>(t.y),
                     [&](int col, float v) { pair += ridge_term(prm, col, v); });
  static_cast<float*>(memo.tab)[static_cast<size_t>(prob) * kMemoCap + slot] = pair;
}

__global__ void ridge_combo_mask_kernel(const ks_problem* __restrict__ p, int P, unsigned* __restrict__ mask) {
  unsigned m = 0;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < P; i += gridDim.x * blockDim.x)
    m |= 1u << ((p[i].dtype_ab & 3) * 4 + (p[i].dtype_d & 3));
  m = __reduce_or_sync(0xFFFFFFFFu, m);
  if ((threadIdx.x & 31) == 0 && m) atomicOr(mask, m);
}

__global__ void __launch_bounds__(kBlock)
select_ridge_kernel(ks_gpu_desc desc, const ks_problem* __restrict__ p, ks_problem p_value, int use_value,
                    const ks_candidate* __restrict__ c, PairMap map, int sub_tiles,
                    const float2* __restrict__ cand_tab, const __grid_constant__ RidgeParams prm, int k,
                    unsigned long long* __restrict__ partial /* [P][nblk][k] */, MemoView memo) {
  __shared__ ProblemTerms s_pt;
  __shared__ float s_prob;  // bias + problem-only part of the sum
  __shared__ unsigned long long s_warp[kBlock / 32 * KS_MAX_K];
  __shared__ unsigned long long s_list[KS_MAX_K];
  const int prob = blockIdx.x / map.nblk, chunk = blockIdx.x % map.nblk;
  int64_t lo, len;
  segment_of(map, prob, lo, len);
  if (threadIdx.x == 0) {
    problem_terms(use_value ? p_value : p[prob], desc, s_pt);
    ks_candidate dummy{};
    dummy.tile_m = dummy.tile_n = dummy.tile_k = 64;
    dummy.stages = dummy.cluster_m = dummy.cluster_n = 1;
    float s = prm.bias;
    featurize_pair(s_pt, dummy, desc, [&](int col, float v) {
      if (feat_class(col) != 0) return;
      s += ridge_term(prm, col, v);
      if (col == 5) s += ridge_level(prm.lut5, v);
      if (col == 9) s += ridge_level(prm.lut9, v);
    });
    s_prob = s;
  }
  if (threadIdx.x < KS_MAX_K) s_list[threadIdx.x] = 0ull;
  __syncthreads();
  const float2* tab = cand_tab + static_cast<size_t>(s_pt.dtype_ab * 4 + s_pt.dtype_d) * map.C;
  // with classes: the per-pair part is one float per (problem, class)
  const unsigned* cls = memo.keys ? memo.cls + static_cast<size_t>(s_pt.dtype_ab * 4 + s_pt.dtype_d) * map.C : nullptr;
  const float* pair_tab = memo.keys ? static_cast<const float*>(memo.tab) + static_cast<size_t>(prob) * kMemoCap : nullptr;

  const int64_t pass_rows = static_cast<int64_t>(sub_tiles) * kBlock;
  for (int64_t start = static_cast<int64_t>(chunk) * pass_rows; start < len;
       start += static_cast<int64_t>(map.nblk) * pass_rows) {
    unsigned long long keys[kSubTilesMax + 1];
#pragma unroll
    for (int s = 0; s <= kSubTilesMax; ++s) keys[s] = 0ull;
    if (threadIdx.x < k) keys[kSubTilesMax] = s_list[threadIdx.x];
#pragma unroll 1
    for (int s = 0; s < sub_tiles; ++s) {
      const int64_t r = start + static_cast<int64_t>(s) * kBlock + threadIdx.x;
      unsigned long long key = 0ull;
      if (r < len) {
        const int idx = pool_index(map, lo, r);
        const float2 t = __ldg(tab + idx);
        const unsigned cid = cls ? __ldg(cls + idx) : kNoClass;
        float pair = 0.0f;
        if (cid != kNoClass) {
          pair = __ldg(pair_tab + cid);
        } else {
          const ks_candidate cand = c[idx];
          pair_columns<true>(s_pt, cand, desc, static_cast<long long>(t.y),
                             [&](int col, float v) { pair += ridge_term(prm, col, v); });
        }
        key = make_key(((s_prob + t.x) + pair) + 0.0f, idx);
      }
#pragma unroll
      for (int q = 0; q < kSubTilesMax; ++q)
        if (q == s) keys[q] = key;
    }
    block_topk<kSubTilesMax + 1>(keys, k, s_warp, s_list);
  }
  if (threadIdx.x < k)
    partial[(static_cast<size_t>(prob) * map.nblk + chunk) * k + threadIdx.x] = s_list[threadIdx.x];
}

// ------------------------------------------------------------------------------------------
// merge: one warp per problem ranks the nblk * k partial keys
// ------------------------------------------------------------------------------------------

__global__ void __launch_bounds__(kBlock)
topk_merge_kernel(const unsigned long long* __restrict__ partial, int P, int n_keys, int k,
                  int32_t* __restrict__ out_idx, float* __restrict__ out_score) {
  const int warp = (blockIdx.x * kBlock + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= P) return;
  const unsigned long long* keys = partial + static_cast<size_t>(warp) * n_keys;
  unsigned long long prev = ~0ull;
  for (int j = 0; j < k; ++j) {
    unsigned long long best = 0ull;
    for (int i = lane; i < n_keys; i += 32) {
      const unsigned long long v = keys[i];
      if (v < prev && v > best) best = v;
    }
    best = warp_max_u64(best);
    if (lane == 0) {
      out_idx[static_cast<size_t>(warp) * k + j] = key_index(best);
      out_score[static_cast<size_t>(warp) * k + j] = key_score(best);
    }
    prev = best == 0ull ? 0ull : best;
  }
}

// Merge of ranked lists (the exchange step of a candidate-split selection): per problem, n
// (index, score) entries gathered from several partial top-k lists, index -1 = empty; the k best
// by (score descending, index ascending) go to the output. One warp per problem.
__global__ void __launch_bounds__(kBlock)
merge_lists_kernel(const int32_t* __restrict__ in_idx, const float* __restrict__ in_score, int P, int n, int k,
                   int32_t* __restrict__ out_idx, float* __restrict__ out_score) {
  const int warp = (blockIdx.x * kBlock + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= P) return;
  const int32_t* idx = in_idx + static_cast<size_t>(warp) * n;
  const float* sc = in_score + static_cast<size_t>(warp) * n;
  unsigned long long prev = ~0ull;
  for (int j = 0; j < k; ++j) {
    unsigned long long best = 0ull;
    for (int i = lane; i < n; i += 32) {
      const unsigned long long v = idx[i] >= 0 ? make_key(sc[i] + 0.0f, idx[i]) : 0ull;
      if (v < prev && v > best) best = v;
    }
    best = warp_max_u64(best);
    if (lane == 0) {
      out_idx[static_cast<size_t>(warp) * k + j] = key_index(best);
      out_score[static_cast<size_t>(warp) * k + j] = key_score(best);
    }
    prev = best;
  }
}

cudaError_t launch_merge_lists(const int32_t* d_idx, const float* d_score, int P, int n, int k, int32_t* d_out_idx,
                               float* d_out_score, cudaStream_t stream, int64_t* launches) {
  merge_lists_kernel<<<(P * 32 + kBlock - 1) / kBlock, kBlock, 0, stream>>>(d_idx, d_score, P, n, k, d_out_idx,
                                                                           d_out_score);
  ++*launches;
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// launchers
// ------------------------------------------------------------------------------------------

static PairMap make_map(int P, int C, int64_t pairs, const int64_t* seg_off, const int32_t* seg_idx,
                        int rows_per_block) {
  PairMap m;
  m.P = P;
  m.C = C;
  m.seg_off = seg_off;
  m.seg_idx = seg_idx;
  m.rows_per_block = rows_per_block;
  const int64_t per_problem = seg_off ? (P > 0 ? (pairs + P - 1) / P : 0) : C;
  m.nblk = static_cast<int>(per_problem > 0 ? (per_problem + rows_per_block - 1) / rows_per_block : 1);
  if (m.nblk < 1) m.nblk = 1;
  return m;
}

cudaError_t launch_featurize(const ks_gpu_desc& desc, const ks_problem* d_p, int P,
                             const ks_candidate* d_c, int C, const int64_t* d_seg_off,
                             const int32_t* d_seg_idx, int64_t pairs, float* d_out, void* scratch,
                             cudaStream_t stream, int64_t* launches) {
  if (P == 0 || pairs == 0) return cudaSuccess;
  const PairMap map = make_map(P, C, pairs, d_seg_off, d_seg_idx, kBlock);
  const size_t smem = sizeof(float) * kBlock * 65;
  if (!d_seg_off && C > 0 && scratch) {
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(&featurize_dense_kernel), smem);
    if (e != cudaSuccess) return e;
    ProblemEntry* tab = static_cast<ProblemEntry*>(scratch);
    problem_table_kernel<<<(P + 127) / 128, 128, 0, stream>>>(desc, d_p, P, tab);
    const int64_t total = static_cast<int64_t>((C + 31) / 32) * P;
    int64_t grid = (total + kBlock / 32 - 1) / (kBlock / 32);
    if (grid > 3 * 148) grid = 3 * 148;  // three resident blocks per SM
    featurize_dense_kernel<<<static_cast<unsigned>(grid), kBlock, smem, stream>>>(desc, tab, d_c, P, C, d_out);
    *launches += 2;
    return cudaGetLastError();
  }
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(&featurize_kernel), smem);
  if (e != cudaSuccess) return e;
  featurize_kernel<<<static_cast<unsigned>(static_cast<int64_t>(P) * map.nblk), kBlock, smem, stream>>>(
      desc, d_p, d_c, map, d_out);
  ++*launches;
  return cudaGetLastError();
}

cudaError_t launch_score_gbdt(const GbdtModel& m, const float* d_feat, int64_t rows, float* d_scores,
                              uint16_t* d_leaf_idx, cudaStream_t stream, int64_t* launches) {
  if (rows == 0) return cudaSuccess;
  const size_t smem = sizeof(float) * kRow * kBlock;
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(&score_gbdt_kernel), smem);
  if (e != cudaSuccess) return e;
  score_gbdt_kernel<<<static_cast<unsigned>((rows + kBlock - 1) / kBlock), kBlock, smem, stream>>>(
      m.d_nodes, m.d_roots, m.n_trees, m.base, d_feat, rows, d_scores, d_leaf_idx);
  ++*launches;
  return cudaGetLastError();
}

static MlpView make_view(const MlpModel& m) {
  MlpView v{};
  v.n_layers = m.n_layers;
  for (int l = 0; l <= m.n_layers; ++l) v.widths[l] = m.widths[l];
  for (int l = 0; l < m.n_layers; ++l) {
    v.w[l] = m.d_w[l];
    v.b[l] = m.d_b[l];
  }
  v.mu = m.d_mu;
  v.sigma = m.d_sigma;
  return v;
}

static size_t mlp_smem_bytes(int max_width) {
  return sizeof(float) * (kRow * kBlock + kBlock) + sizeof(__nv_bfloat16) * 2 * max_width * 32;
}

cudaError_t launch_score_mlp(const MlpModel& m, const float* d_feat, int64_t rows, float* d_scores,
                             cudaStream_t stream, int64_t* launches) {
  if (rows == 0) return cudaSuccess;
  const size_t smem = mlp_smem_bytes(m.max_width);
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(&score_mlp_kernel), smem);
  if (e != cudaSuccess) return e;
  score_mlp_kernel<<<static_cast<unsigned>((rows + kBlock - 1) / kBlock), kBlock, smem, stream>>>(
      make_view(m), m.max_width, d_feat, rows, d_scores);
  ++*launches;
  return cudaGetLastError();
}

static float bf16_bits_host(uint16_t b) {
  const uint32_t u = static_cast<uint32_t>(b) << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return f;
}
static float round_bf16_host(float v) {
  uint32_t u;
  std::memcpy(&u, &v, 4);
  if ((u & 0x7F800000u) == 0x7F800000u) return v;
  u += 0x7FFFu + ((u >> 16) & 1u);
  u &= 0xFFFF0000u;
  std::memcpy(&v, &u, 4);
  return v;
}

cudaError_t build_ridge(MlpModel& m, const uint16_t* h_w, const float* h_b, const float* h_mu,
                        const float* h_sigma) {
  if (m.n_layers != 1) return cudaSuccess;
  RidgeParams* r = new (std::nothrow) RidgeParams();
  if (!r) return cudaErrorMemoryAllocation;
  std::memset(r, 0, sizeof(*r));
  for (int j = 0; j < 64; ++j) r->sigma[j] = 1.0f;
  r->bias = h_b[0];
  if (m.widths[0] == KS_F_PAD) {
    for (int j = 0; j < KS_F; ++j) {
      r->w[j] = bf16_bits_host(h_w[j]);
      r->mu[j] = h_mu[j];
      r->sigma[j] = h_sigma[j];
    }
  } else {  // one-hot form: kept columns in ascending order, then the level indicators
    int pos = 0;
    for (int j = 0; j < KS_F; ++j) {
      if (j == 5 || j == 9 || j == 17 || j == 18) continue;
      r->w[j] = bf16_bits_host(h_w[pos]);
      r->mu[j] = h_mu[pos];
      r->sigma[j] = h_sigma[pos];
      ++pos;
    }
    float* luts[4] = {r->lut5, r->lut9, r->lut17, r->lut18};
    const int levels[4] = {4, 3, 4, 3};
    for (int f = 0; f < 4; ++f) {
      for (int lv = 0; lv < levels[f]; ++lv) {  // the field is at level lv: one indicator is 1
        float s = 0.0f;
        for (int q = 0; q < levels[f]; ++q) {
          const float x = round_bf16_host(((q == lv ? 1.0f : 0.0f) - h_mu[pos + q]) / h_sigma[pos + q]);
          s += bf16_bits_host(h_w[pos + q]) * x;
        }
        luts[f][lv] = s;
      }
      pos += levels[f];
    }
  }
  m.h_ridge = r;
  return cudaSuccess;
}

void free_ridge(MlpModel& m) {
  delete m.h_ridge;
  m.h_ridge = nullptr;
}

size_t ridge_scratch_bytes(int C) { return (256 + sizeof(float2) * 16 * static_cast<size_t>(C) + 255) / 256 * 256; }
// classes and the per-(problem, class) sums of the linear scorer (0: not used)
size_t ridge_memo_bytes(int P, int C) {
  if (P < kMemoMinProblems || P > kMemoMaxProblems || C < 1) return 0;
  return memo_fixed_bytes(C) + sizeof(float) * static_cast<size_t>(P) * kMemoCap;
}

static int pick_sub_tiles(int P, int64_t per_problem) {
  for (int s = kSubTilesMax; s > 1; s >>= 1) {
    const int64_t nblk = (per_problem + static_cast<int64_t>(s) * kBlock - 1) / (static_cast<int64_t>(s) * kBlock);
    if (static_cast<int64_t>(P) * nblk >= 4 * 148) return s;
  }
  return 1;
}

static int64_t per_problem_rows(int P, int C, int64_t pairs, bool segmented) {
  return segmented ? (P > 0 ? (pairs + P - 1) / P : 0) : C;
}

size_t select_partial_bytes(const ks_model& model, int P, int C, int64_t pairs, bool segmented, int k) {
  const int64_t per = per_problem_rows(P, C, pairs, segmented);
  if (model.kind == 0 && model.gbdt.fast) {
    int nblk, rows;
    fast_tiling(model.gbdt, P, per, &nblk, &rows);
    const size_t part = (static_cast<size_t>(P) * nblk * k * sizeof(unsigned long long) + 255) / 256 * 256;
    const int S = segmented ? 1 : fast_slices(model.gbdt, static_cast<int64_t>(P) * nblk);
    const size_t planes = S > 1 ? (sizeof(float) * S * static_cast<size_t>(pairs) + 255) / 256 * 256 : 0;
    const size_t memo = S > 1 ? 0 : (fast_memo_bytes(model.gbdt, P, C) + 255) / 256 * 256;
    // a dense batch is ranked in similarity order of the catalogue (ks_order.cu)
    const size_t order = (memo > 0 && !segmented && P >= kOrderMinProblems) ? order_scratch_bytes(C) : 0;
    return part + (fast_scratch_bytes(model.gbdt, C) + 255) / 256 * 256 + planes + memo + order;
  }
  if (model.kind == 1 && model.mlp.tc) {
    const int nblk = mlp_tc_blocks_per_problem(P, per);
    const size_t part = (static_cast<size_t>(P) * nblk * k * sizeof(unsigned long long) + 255) / 256 * 256;
    return part + mlp_tc_scratch_bytes(C);
  }
  const int st = pick_sub_tiles(P, per);
  int64_t nblk = (per + static_cast<int64_t>(st) * kBlock - 1) / (static_cast<int64_t>(st) * kBlock);
  if (nblk < 1) nblk = 1;
  const size_t part = static_cast<size_t>(P) * nblk * k * sizeof(unsigned long long);
  if (model.kind == 1 && model.mlp.h_ridge)
    return (part + 255) / 256 * 256 + ridge_scratch_bytes(C) + ridge_memo_bytes(P, C);
  return part;
}

cudaError_t launch_select(const ks_gpu_desc& desc, const ks_model& model, const ks_problem* d_p,
                          const ks_problem* p_by_value, int P, const ks_candidate* d_c, int C,
                          const int64_t* d_seg_off, const int32_t* d_seg_idx, int64_t pairs, int k,
                          void* d_partial, int32_t* d_topk_idx, float* d_topk_score,
                          cudaStream_t stream, int64_t* launches, int* d_status, cudaEvent_t ev_begin,
                          cudaEvent_t ev_end, int* d_counters, const FastWait* wait) {
  if (P == 0) return cudaSuccess;
  const int64_t per = per_problem_rows(P, C, pairs, d_seg_off != nullptr);
  if (model.kind == 0 && model.gbdt.fast) {
    int nblk, rows;
    fast_tiling(model.gbdt, P, per, &nblk, &rows);
    unsigned long long* part = static_cast<unsigned long long*>(d_partial);
    const size_t part_bytes = (static_cast<size_t>(P) * nblk * k * sizeof(unsigned long long) + 255) / 256 * 256;
    // an under-filled machine: split the trees over several CTAs per block (dense form only,
    // where a block covers its rows in one pass)
    FastSlice sl{};
    sl.n_slices = (d_seg_off || !d_counters) ? 1 : fast_slices(model.gbdt, static_cast<int64_t>(P) * nblk);
    if (sl.n_slices > 1) {
      sl.pairs = pairs;
      sl.scores = reinterpret_cast<float*>(static_cast<char*>(d_partial) + part_bytes +
                                           (fast_scratch_bytes(model.gbdt, C) + 255) / 256 * 256);
      sl.counters = d_counters;
    }
    // the memo of the per-pair rows sits behind the per-call table (batches of whole-ensemble CTAs only)
    const int sized_slices = d_seg_off ? 1 : fast_slices(model.gbdt, static_cast<int64_t>(P) * nblk);  // as sized
    void* memo_mem = (sized_slices > 1 || p_by_value || fast_memo_bytes(model.gbdt, P, C) == 0)
                         ? nullptr
                         : static_cast<char*>(d_partial) + part_bytes + (fast_scratch_bytes(model.gbdt, C) + 255) / 256 * 256;
    // a dense batch of problems: rank the catalogue in similarity order (neighbouring candidates
    // then take similar paths through the trees); the order sits behind the memo
    const int32_t* perm = nullptr;
    if (memo_mem && !d_seg_off && P >= kOrderMinProblems && C > 0) {
      void* order_mem = static_cast<char*>(memo_mem) + (fast_memo_bytes(model.gbdt, P, C) + 255) / 256 * 256;
      cudaError_t eo = launch_catalogue_order(d_c, C, order_mem, stream, launches);
      if (eo != cudaSuccess) return eo;
      perm = static_cast<const int32_t*>(order_mem);
    }
    cudaError_t e = launch_select_fast(desc, model.gbdt, d_p, p_by_value, P, d_c, C, nblk, rows, d_seg_off,
                                       d_seg_idx, k, part, static_cast<char*>(d_partial) + part_bytes, d_status,
                                       stream, launches, ev_begin, sl.n_slices > 1 ? &sl : nullptr, memo_mem, wait,
                                       nullptr, perm);
    if (e != cudaSuccess) return e;
    if (ev_end) cudaEventRecord(ev_end, stream);
    topk_merge_kernel<<<(P * 32 + kBlock - 1) / kBlock, kBlock, 0, stream>>>(part, P, nblk * k, k, d_topk_idx,
                                                                            d_topk_score);
    ++*launches;
    return cudaGetLastError();
  }
  if (model.kind == 1 && model.mlp.tc) {
    const int nblk = mlp_tc_blocks_per_problem(P, per);
    unsigned long long* part = static_cast<unsigned long long*>(d_partial);
    const size_t part_bytes = (static_cast<size_t>(P) * nblk * k * sizeof(unsigned long long) + 255) / 256 * 256;
    cudaError_t e = launch_select_mlp_tc(desc, model.mlp, d_p, p_by_value, P, d_c, C, nblk, d_seg_off, d_seg_idx, k,
                                         part, static_cast<char*>(d_partial) + part_bytes, d_status, stream,
                                         launches, ev_begin, wait);
    if (e != cudaSuccess) return e;
    if (ev_end) cudaEventRecord(ev_end, stream);
    topk_merge_kernel<<<(P * 32 + kBlock - 1) / kBlock, kBlock, 0, stream>>>(part, P, nblk * k, k, d_topk_idx,
                                                                            d_topk_score);
    ++*launches;
    return cudaGetLastError();
  }
  const int st = pick_sub_tiles(P, per);
  const PairMap map = make_map(P, C, pairs, d_seg_off, d_seg_idx, st * kBlock);
  unsigned long long* partial = static_cast<unsigned long long*>(d_partial);
  const unsigned grid = static_cast<unsigned>(static_cast<int64_t>(P) * map.nblk);
  ks_problem pv{};
  if (p_by_value) pv = *p_by_value;
  cudaError_t e;
  if (model.kind == 1 && model.mlp.h_ridge) {
    // linear scorer: per-call table of candidate-only sums, then the fused kernel
    const size_t part_bytes = (static_cast<size_t>(P) * map.nblk * k * sizeof(unsigned long long) + 255) / 256 * 256;
    unsigned* d_mask = reinterpret_cast<unsigned*>(static_cast<char*>(d_partial) + part_bytes);
    float2* d_tab = reinterpret_cast<float2*>(static_cast<char*>(d_partial) + part_bytes + 256);
    unsigned mask_value = 0;
    if (p_by_value) {
      mask_value = 1u << ((pv.dtype_ab & 3) * 4 + (pv.dtype_d & 3));
    } else {
      e = cudaMemsetAsync(d_mask, 0, sizeof(unsigned), stream);
      if (e != cudaSuccess) return e;
      ridge_combo_mask_kernel<<<P >= 4096 ? 16 : 1, 256, 0, stream>>>(d_p, P, d_mask);
      ++*launches;
    }
    MemoView memo{};
    if (!p_by_value && ridge_memo_bytes(P, C) != 0)
      memo = memo_view(static_cast<char*>(d_partial) + part_bytes + ridge_scratch_bytes(C), C);
    if (C > 0) {
      if (memo.keys) {
        e = memo_clear(memo, stream);
        if (e != cudaSuccess) return e;
      }
      ridge_cand_kernel<<<dim3((C + 255) / 256, 16), 256, 0, stream>>>(desc, d_c, C, p_by_value ? nullptr : d_mask,
                                                                      mask_value, *model.mlp.h_ridge, d_tab, memo);
      ++*launches;
      if (memo.keys) {
        e = memo_compact(memo, stream);
        if (e != cudaSuccess) return e;
        ridge_pair_kernel<<<dim3(kMemoCap / 256, P), 256, 0, stream>>>(desc, d_p, d_c, d_tab, C, *model.mlp.h_ridge, memo);
        *launches += 2;
      }
    } else {
      memo = MemoView{};
    }
    if (ev_begin) cudaEventRecord(ev_begin, stream);
    select_ridge_kernel<<<grid, kBlock, 0, stream>>>(desc, d_p, pv, p_by_value != nullptr, d_c, map, st, d_tab,
                                                     *model.mlp.h_ridge, k, partial, memo);
    ++*launches;
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (ev_end) cudaEventRecord(ev_end, stream);
    topk_merge_kernel<<<(P * 32 + kBlock - 1) / kBlock, kBlock, 0, stream>>>(partial, P, map.nblk * k, k,
                                                                            d_topk_idx, d_topk_score);
    ++*launches;
    return cudaGetLastError();
  }
  if (ev_begin) cudaEventRecord(ev_begin, stream);
  if (model.kind == 2) {
    select_generic_kernel<2><<<grid, kBlock, 0, stream>>>(desc, d_p, pv, p_by_value != nullptr, d_c, map, st, nullptr,
                                                          nullptr, 0, 0.0f, MlpView{}, 0, k, partial);
  } else if (model.kind == 0) {
    const GbdtModel& g = model.gbdt;
    const size_t smem = sizeof(float) * kRow * kBlock;
    e = ensure_dynamic_smem(reinterpret_cast<const void*>(&select_generic_kernel<0>), smem);
    if (e != cudaSuccess) return e;
    select_generic_kernel<0><<<grid, kBlock, smem, stream>>>(
        desc, d_p, pv, p_by_value != nullptr, d_c, map, st, g.d_nodes, g.d_roots, g.n_trees, g.base,
        MlpView{}, 0, k, partial);
  } else {
    const size_t smem = mlp_smem_bytes(model.mlp.max_width);
    e = ensure_dynamic_smem(reinterpret_cast<const void*>(&select_generic_kernel<1>), smem);
    if (e != cudaSuccess) return e;
    select_generic_kernel<1><<<grid, kBlock, smem, stream>>>(
        desc, d_p, pv, p_by_value != nullptr, d_c, map, st, nullptr, nullptr, 0, 0.0f,
        make_view(model.mlp), model.mlp.max_width, k, partial);
  }
  ++*launches;
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (ev_end) cudaEventRecord(ev_end, stream);
  topk_merge_kernel<<<(P * 32 + kBlock - 1) / kBlock, kBlock, 0, stream>>>(partial, P, map.nblk * k, k,
                                                                          d_topk_idx, d_topk_score);
  ++*launches;
  return cudaGetLastError();
}


// Generic tree select with caller-provided node arrays and partial-list storage (dense form).
int64_t select_generic_partial_keys(int P, int C, int k) {
  const int st = pick_sub_tiles(P, C);
  const PairMap map = make_map(P, C, static_cast<int64_t>(P) * C, nullptr, nullptr, st * kBlock);
  return static_cast<int64_t>(P) * map.nblk * k;
}

cudaError_t launch_select_generic_trees(const ks_gpu_desc& desc, const DevNode* d_nodes, const int* d_roots,
                                        int n_trees, float base, const ks_problem* d_p, int P,
                                        const ks_candidate* d_c, int C, int k, unsigned long long* partial,
                                        int32_t* d_topk_idx, float* d_topk_score, cudaStream_t stream) {
  const int st = pick_sub_tiles(P, C);
  const PairMap map = make_map(P, C, static_cast<int64_t>(P) * C, nullptr, nullptr, st * kBlock);
  const size_t smem = sizeof(float) * kRow * kBlock;
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(&select_generic_kernel<0>), smem);
  if (e != cudaSuccess) return e;
  select_generic_kernel<0><<<static_cast<unsigned>(static_cast<int64_t>(P) * map.nblk), kBlock, smem, stream>>>(
      desc, d_p, ks_problem{}, 0, d_c, map, st, d_nodes, d_roots, n_trees, base, MlpView{}, 0, k, partial);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  topk_merge_kernel<<<(P * 32 + kBlock - 1) / kBlock, kBlock, 0, stream>>>(partial, P, map.nblk * k, k,
                                                                          d_topk_idx, d_topk_score);
  return cudaGetLastError();
}

size_t featurize_scratch_bytes(int P) { return sizeof(ProblemEntry) * static_cast<size_t>(P > 0 ? P : 1); }

}  // namespace ks
