// Quantised fast path of the fused select kernel for tree ensembles (Model A).
//
// Repack (host, at model-create time)
//   Every split "x[f] < thr" only needs to know how many of feature f's distinct thresholds
//   are <= x. With the thresholds of f sorted, bin(x) = #{j : thr_j <= x}, and
//   x < thr_j  <=>  bin(x) <= j  exactly, so a pair's feature row shrinks from 64 floats to
//   one byte per "row" (a feature, or a 255-threshold slice of one) and a node to one 32-bit
//   word (row << 19 | j). Trees are padded to complete trees of the ensemble's depth D and
//   stored in chunks of kTreesPerChunk trees, each chunk laid out level by level
//   ([level][tree][node]) followed by its leaves, so that a chunk is one contiguous block a
//   CTA copies into shared memory with a single bulk async copy.
//
// Kernel (one CTA = one problem x up to kFastRows candidates)
//   phase A  featurize every pair in registers, quantise each column by an 8-step branch-free
//            search in the threshold table (held in shared memory), store the bytes in a
//            [row][thread] tile whose 32-bit word holds the four candidates of one thread:
//            a warp's byte loads of any mix of rows hit 32 distinct banks;
//   phase B  stream the ensemble chunk by chunk through two shared-memory buffers
//            (cp.async.bulk + mbarrier, bounded waits); each thread walks every tree for its
//            four candidates, the four walks interleaved for latency hiding;
//   phase C  rank the block's keys and write a partial top-k list.
#include <algorithm>
#include <cmath>
#include <limits>
#include <vector>

#include "ks_features.cuh"
#include "ks_internal.h"
#include "ks_topk.cuh"

namespace ks {

namespace {

constexpr int kBufBytes = 32 * 1024;  // one tree-chunk buffer
constexpr int kMaxRows = 64;          // quantised rows the kernel supports
constexpr int kThrPerRow = 256;       // 255 thresholds + padding
constexpr int kRowStride = kFastRows;  // bytes between rows of the tile (one byte per candidate)
constexpr int kSpinLimit = 1 << 22;
constexpr int kTreesInFlight = 2;     // trees walked concurrently per candidate (tpc is a multiple of 4)

// ---- shared memory map (byte offsets from the dynamic shared base) ----------------------
constexpr int kOffBuf0 = 0;
constexpr int kOffBuf1 = kBufBytes;
constexpr int kOffTile = 2 * kBufBytes;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after kSpinLimit probes and reports false.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  for (int i = 0; i < kSpinLimit; ++i)
    if (mbar_try_wait(bar, parity)) return true;
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
__device__ __forceinline__ uint32_t lds_u8(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ float lds_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
  return v;
}

// Byte offset, inside one row of the tile, of a thread's first candidate. A 32-bit word
// holds four candidates and consecutive lanes of a warp own consecutive words, so a warp's
// byte loads of any mix of rows touch 32 distinct banks.
__device__ __forceinline__ int slot_offset(int tid) {
  constexpr int kWords = kFastRows / 4;            // words per row
  constexpr int kPerWord = 4 / kFastR;             // threads sharing a word
  static_assert(kFastThreads == kWords * kPerWord, "tile geometry");
  return (tid % kWords) * 4 + (tid / kWords) * kFastR;
}

struct FastView {
  int n_rows, depth, n_chunks, chunk_bytes, tpc;
  float base;
  const uint32_t* chunks;       // [n_chunks][chunk_bytes / 4]
  const float* thr;             // [n_rows][kThrPerRow]
  const uint8_t* feat_row0;     // [64] first row of each feature column
  const uint8_t* feat_rowcnt;   // [64] number of rows of each feature column
};

template <int D>
__global__ void __launch_bounds__(kFastThreads, 1)
select_fast_kernel(ks_gpu_desc desc, const ks_problem* __restrict__ p, ks_problem p_value, int use_value,
                   const ks_candidate* __restrict__ c, int P, int C, int nblk, int rows_per_cta,
                   const int64_t* __restrict__ seg_off, const int32_t* __restrict__ seg_idx, FastView fv,
                   int k, unsigned long long* __restrict__ partial, int* __restrict__ status) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ ProblemTerms s_pt;
  __shared__ unsigned long long s_warp[kFastThreads / 32];
  __shared__ unsigned long long s_list[KS_MAX_K];
  __shared__ __align__(8) unsigned long long s_bar[2];
  __shared__ uint8_t s_row0[64], s_rowcnt[64];
  __shared__ int s_fail;

  const int tid = threadIdx.x;
  const int prob = blockIdx.x / nblk, chunk = blockIdx.x % nblk;
  int64_t lo, len;
  if (seg_off) {
    lo = seg_off[prob];
    len = seg_off[prob + 1] - lo;
  } else {
    lo = static_cast<int64_t>(prob) * C;
    len = C;
  }
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bar0 = smem_u32(&s_bar[0]), bar1 = smem_u32(&s_bar[1]);
  if (tid == 0) {
    problem_terms(use_value ? p_value : p[prob], desc, s_pt);
    mbar_init(bar0, 1);
    mbar_init(bar1, 1);
    s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < 64) {
    s_row0[tid] = fv.feat_row0[tid];
    s_rowcnt[tid] = fv.feat_rowcnt[tid];
  }
  if (tid < KS_MAX_K) s_list[tid] = 0ull;
  uint32_t phase0 = 0, phase1 = 0;

  for (int64_t start = static_cast<int64_t>(chunk) * rows_per_cta; start < len;
       start += static_cast<int64_t>(nblk) * rows_per_cta) {
    const int64_t stop = (start + rows_per_cta < len) ? start + rows_per_cta : len;
    // ---- phase A: threshold table into the (idle) tree buffers, then featurize + quantise ----
    __syncthreads();
    {
      float4* dst = reinterpret_cast<float4*>(smem + kOffBuf0);
      const float4* src = reinterpret_cast<const float4*>(fv.thr);
      for (int i = tid; i < fv.n_rows * kThrPerRow / 4; i += kFastThreads) dst[i] = __ldg(src + i);
    }
    __syncthreads();
    const float* s_thr = reinterpret_cast<const float*>(smem + kOffBuf0);
    unsigned char* tile = smem + kOffTile;
#pragma unroll 1
    for (int r = 0; r < kFastR; ++r) {
      const int64_t row = start + static_cast<int64_t>(r) * kFastThreads + tid;
      if (row < stop) {
        const int ci = seg_off ? seg_idx[lo + row] : static_cast<int>(row);
        const ks_candidate cand = c[ci];
        unsigned char* my = tile + slot_offset(tid) + r;
        featurize_pair(s_pt, cand, desc, [&](int col, float v) {
          const int r0 = s_row0[col], rc = s_rowcnt[col];
          for (int q = 0; q < rc; ++q) {
            const float* T = s_thr + (r0 + q) * kThrPerRow;
            int pos = 0;
#pragma unroll
            for (int s = 128; s >= 1; s >>= 1) pos += (T[pos + s - 1] <= v) ? s : 0;
            my[(r0 + q) * kRowStride] = static_cast<unsigned char>(pos);
          }
        });
      }
    }
    __syncthreads();  // tile complete; the threshold table is no longer needed

    // ---- phase B: stream the ensemble through the two buffers ---------------------------------
    if (tid == 0) {
      fence_async_proxy();
      mbar_expect_tx(bar0, fv.chunk_bytes);
      bulk_copy_g2s(sbase + kOffBuf0, fv.chunks, fv.chunk_bytes, bar0);
      if (fv.n_chunks > 1) {
        mbar_expect_tx(bar1, fv.chunk_bytes);
        bulk_copy_g2s(sbase + kOffBuf1, reinterpret_cast<const char*>(fv.chunks) + fv.chunk_bytes,
                      fv.chunk_bytes, bar1);
      }
    }
    float score[kFastR];
#pragma unroll
    for (int r = 0; r < kFastR; ++r) score[r] = fv.base;
    const uint32_t cb = sbase + kOffTile + slot_offset(tid);
    const int tpc = fv.tpc;
#pragma unroll 1
    for (int ch = 0; ch < fv.n_chunks; ++ch) {
      const int b = ch & 1;
      const uint32_t bar = b ? bar1 : bar0;
      const uint32_t par = b ? phase1 : phase0;
      if (!mbar_wait_bounded(bar, par)) {
        s_fail = 1;
        if (status) atomicExch(status, KS_ERR_TIMEOUT);
      }
      if (b) phase1 ^= 1; else phase0 ^= 1;
      const uint32_t buf = sbase + (b ? kOffBuf1 : kOffBuf0);
      // With A_l the shared address of a walk's node at level l (levels stored back to back,
      // [level][tree][node]), A_{l+1} = 2 A_l + (4 tpc - buf) + 4 bit for every level, and
      // after D steps the address points at the walk's leaf.
      // The address lives in a float register as a denormal (bit pattern == integer value):
      // denormal arithmetic is exact fixed-point, so the update is one FFMA plus a predicated
      // FADD on the FMA pipe instead of integer ALU work.
      const int k0 = static_cast<int>(4u * tpc) - static_cast<int>(buf);
      const float K0f = k0 >= 0 ? __uint_as_float(static_cast<uint32_t>(k0))
                                : -__uint_as_float(static_cast<uint32_t>(-k0));
      const float four = __uint_as_float(4u);
#pragma unroll 1
      for (int t = 0; t < tpc; t += kTreesInFlight) {
        float a[kTreesInFlight][kFastR];
#pragma unroll
        for (int u = 0; u < kTreesInFlight; ++u)
#pragma unroll
          for (int r = 0; r < kFastR; ++r) a[u][r] = __uint_as_float(buf + 4u * (t + u));
#pragma unroll
        for (int l = 0; l < D; ++l) {
#pragma unroll
          for (int u = 0; u < kTreesInFlight; ++u)
#pragma unroll
            for (int r = 0; r < kFastR; ++r) {
              const uint32_t n = lds_u32(__float_as_uint(a[u][r]));
              const uint32_t x = lds_u8(cb + (n >> 8) + r);
              float nx = __fmaf_rn(a[u][r], 2.0f, K0f);
              if (x > (n & 0xFFu)) nx = __fadd_rn(nx, four);
              a[u][r] = nx;
            }
        }
#pragma unroll
        for (int u = 0; u < kTreesInFlight; ++u)
#pragma unroll
          for (int r = 0; r < kFastR; ++r) score[r] += lds_f32(__float_as_uint(a[u][r]));
      }
      __syncthreads();  // every thread is done with this buffer
      if (tid == 0 && ch + 2 < fv.n_chunks && !s_fail) {
        mbar_expect_tx(bar, fv.chunk_bytes);
        bulk_copy_g2s(buf, reinterpret_cast<const char*>(fv.chunks) + static_cast<size_t>(ch + 2) * fv.chunk_bytes,
                      fv.chunk_bytes, bar);
      }
    }

    // ---- phase C: rank -------------------------------------------------------------------------
    unsigned long long keys[kFastR + 1];
#pragma unroll
    for (int r = 0; r < kFastR; ++r) {
      const int64_t row = start + static_cast<int64_t>(r) * kFastThreads + tid;
      keys[r] = 0ull;
      if (row < stop) keys[r] = make_key(score[r] + 0.0f, seg_off ? seg_idx[lo + row] : static_cast<int>(row));
    }
    keys[kFastR] = tid < k ? s_list[tid] : 0ull;
    __syncthreads();
    block_topk<kFastR + 1>(keys, k, s_warp, s_list);
  }
  if (tid < k) partial[(static_cast<size_t>(prob) * nblk + chunk) * k + tid] = s_list[tid];
}

}  // namespace

// ------------------------------------------------------------------------------------------
// host: repack
// ------------------------------------------------------------------------------------------

cudaError_t build_fast_gbdt(GbdtModel& m, int n_trees, const int64_t* off, const ks_node_host* nodes) {
  m.fast = false;
  if (n_trees < 1 || m.max_depth < 1 || m.max_depth > kFastMaxDepth) return cudaSuccess;
  const int D = m.max_depth;
  // distinct thresholds per feature
  std::vector<std::vector<float>> thr(KS_F);
  for (int64_t i = 0; i < off[n_trees]; ++i)
    if (nodes[i].feat != 0xFFFF) thr[nodes[i].feat].push_back(nodes[i].thr_or_leaf);
  std::vector<uint8_t> row0(64, 0), rowcnt(64, 0);
  std::vector<float> table;
  int n_rows = 0;
  for (int f = 0; f < KS_F; ++f) {
    auto& v = thr[f];
    std::sort(v.begin(), v.end());
    v.erase(std::unique(v.begin(), v.end()), v.end());
    const int cnt = static_cast<int>((v.size() + 254) / 255);
    if (n_rows + cnt > kMaxRows) return cudaSuccess;  // not eligible: stays on the generic path
    row0[f] = static_cast<uint8_t>(n_rows);
    rowcnt[f] = static_cast<uint8_t>(cnt);
    for (int q = 0; q < cnt; ++q) {
      for (int j = 0; j < kThrPerRow; ++j) {
        const size_t s = static_cast<size_t>(q) * 255 + j;
        table.push_back(j < 255 && s < v.size() ? v[s] : std::numeric_limits<float>::infinity());
      }
    }
    n_rows += cnt;
  }
  if (n_rows == 0) return cudaSuccess;
  const int per_tree_words = (2 << D) - 1;
  int tpc = kBufBytes / (per_tree_words * 4) / 4 * 4;  // a multiple of 4 keeps chunks 16-byte sized
  if (tpc < 4) return cudaSuccess;
  if (tpc > (n_trees + 3) / 4 * 4) tpc = (n_trees + 3) / 4 * 4;  // a small ensemble is one short chunk
  const int n_chunks = (n_trees + tpc - 1) / tpc;
  const int chunk_words = tpc * per_tree_words;  // tpc is a multiple of 4 for D <= 10, so 16-byte sized
  if ((chunk_words * 4) % 16 != 0) return cudaSuccess;
  std::vector<uint32_t> chunks(static_cast<size_t>(n_chunks) * chunk_words);
  const uint32_t always_left = 255u;  // row 0, bin 255: every byte is <= 255
  for (int ch = 0; ch < n_chunks; ++ch) {
    uint32_t* base = chunks.data() + static_cast<size_t>(ch) * chunk_words;
    float* leaves = reinterpret_cast<float*>(base + tpc * ((1 << D) - 1));
    for (int tt = 0; tt < tpc; ++tt) {
      const int t = ch * tpc + tt;
      // walk the (padded) complete tree: slot (level l, index i) holds original node `src` or,
      // below an original leaf, a pass-through node that always goes left
      std::vector<int> src(1, t < n_trees ? 0 : -1);
      std::vector<float> carry(1, 0.0f);  // leaf value carried below an original leaf
      for (int l = 0; l < D; ++l) {
        uint32_t* lvl = base;
        for (int q = 0; q < l; ++q) lvl += tpc << q;
        std::vector<int> nsrc(2 << l);
        std::vector<float> ncarry(2 << l);
        for (int i = 0; i < (1 << l); ++i) {
          uint32_t word = always_left;
          int ls = -1, rs = -1;
          float lc = carry[i], rc = carry[i];
          if (src[i] >= 0) {
            const ks_node_host& nd = nodes[off[t] + src[i]];
            if (nd.feat == 0xFFFF) {
              lc = rc = nd.thr_or_leaf;
            } else {
              const auto& v = thr[nd.feat];
              const int j = static_cast<int>(std::lower_bound(v.begin(), v.end(), nd.thr_or_leaf) - v.begin());
              const int row = row0[nd.feat] + j / 255;
              word = (static_cast<uint32_t>(row) * kRowStride) << 8 | static_cast<uint32_t>(j % 255);
              ls = nd.left;
              rs = nd.left + 1;
            }
          }
          lvl[tt * (1 << l) + i] = word;
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
        if (src[i] >= 0) v = nodes[off[t] + src[i]].thr_or_leaf;  // depth-D original leaf
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
  if (e != cudaSuccess) return e;
  m.fast = true;
  m.fast_depth = D;
  m.n_qrows = n_rows;
  m.tpc = tpc;
  m.n_chunks = n_chunks;
  m.chunk_bytes = chunk_words * 4;
  return cudaSuccess;
}

// ------------------------------------------------------------------------------------------
// launcher
// ------------------------------------------------------------------------------------------

// Blocks per problem: full tiles of kFastRows rows, unless that would leave most SMs idle,
// in which case the rows of a problem are spread over more, shorter blocks.
void fast_tiling(int P, int64_t per_problem, int* nblk, int* rows_per_cta) {
  int64_t n = (per_problem + kFastRows - 1) / kFastRows;
  if (n < 1) n = 1;
  const int64_t want = 2 * 148;
  if (P * n < want && per_problem > 0) {
    int64_t m = (want + P - 1) / P;
    const int64_t cap = (per_problem + 127) / 128;  // at least 128 rows per block
    if (m > cap) m = cap;
    if (m > n) n = m;
  }
  int64_t rows = per_problem > 0 ? (per_problem + n - 1) / n : kFastRows;
  if (rows > kFastRows) rows = kFastRows;
  *nblk = static_cast<int>(n);
  *rows_per_cta = static_cast<int>(rows);
}

template <int D>
static cudaError_t launch_d(const ks_gpu_desc& desc, const GbdtModel& g, const ks_problem* d_p,
                            const ks_problem& pv, int use_value, int P, const ks_candidate* d_c, int C,
                            int nblk, int rows_per_cta, const int64_t* seg_off, const int32_t* seg_idx,
                            int k, unsigned long long* partial, int* status, cudaStream_t stream) {
  FastView fv;
  fv.n_rows = g.n_qrows;
  fv.depth = D;
  fv.n_chunks = g.n_chunks;
  fv.chunk_bytes = g.chunk_bytes;
  fv.tpc = g.tpc;
  fv.base = g.base;
  fv.chunks = g.d_qnodes;
  fv.thr = g.d_qthr;
  fv.feat_row0 = g.d_qrow0;
  fv.feat_rowcnt = g.d_qrowcnt;
  const size_t smem = kOffTile + static_cast<size_t>(g.n_qrows) * kRowStride;
  cudaError_t e = cudaFuncSetAttribute(select_fast_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  select_fast_kernel<D><<<static_cast<unsigned>(static_cast<int64_t>(P) * nblk), kFastThreads, smem, stream>>>(
      desc, d_p, pv, use_value, d_c, P, C, nblk, rows_per_cta, seg_off, seg_idx, fv, k, partial, status);
  return cudaGetLastError();
}

cudaError_t launch_select_fast(const ks_gpu_desc& desc, const GbdtModel& g, const ks_problem* d_p,
                               const ks_problem* p_by_value, int P, const ks_candidate* d_c, int C,
                               int nblk, int rows_per_cta, const int64_t* seg_off, const int32_t* seg_idx,
                               int k, unsigned long long* partial, int* status, cudaStream_t stream) {
  ks_problem pv{};
  if (p_by_value) pv = *p_by_value;
  const int uv = p_by_value != nullptr;
#define KS_CASE(D) \
  case D: return launch_d<D>(desc, g, d_p, pv, uv, P, d_c, C, nblk, rows_per_cta, seg_off, seg_idx, k, partial, status, stream);
  switch (g.fast_depth) {
    KS_CASE(1) KS_CASE(2) KS_CASE(3) KS_CASE(4) KS_CASE(5) KS_CASE(6) KS_CASE(7) KS_CASE(8) KS_CASE(9) KS_CASE(10)
    default: return cudaErrorInvalidValue;
  }
#undef KS_CASE
}

}  // namespace ks
