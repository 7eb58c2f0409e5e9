// Search-space enumeration (Table "Configuration knobs") and static validity filtering (Table
// "Static validity constraints") on the device: candidates are generated from their linear id
// instead of being loaded, tested against the rules, and the survivors are packed in id order.
//
// Three small launches: per-block counts of valid candidates, an exclusive scan of those counts
// by one block, and a scatter that recomputes the predicate (a few dozen integer operations,
// cheaper than storing and re-reading a flag array). A block owns kCatTile consecutive
// candidates and a thread four consecutive ones, so positions inside a block follow from a
// prefix sum over threads and the output keeps the input order.
#include <cuda_runtime.h>

#include "ks_features.cuh"
#include "ks_internal.h"

namespace ks {
namespace {

constexpr int kCatThreads = 256;
constexpr int kCatPerThread = 4;
constexpr int kCatTile = kCatThreads * kCatPerThread;

// Linear id -> candidate: a mixed-radix number whose digits follow the rows of the knob table,
// first row slowest: tile_m (4), tile_n (9), tile_k (5), stages (11), cluster shape (15),
// kernel schedule (3), epilogue schedule (3), tile scheduler (2).
__device__ __forceinline__ ks_candidate decode_candidate(long long id) {
  unsigned r = static_cast<unsigned>(id);  // ids are below 534,600
  const unsigned tile_sched = r % 2u; r /= 2u;
  const unsigned epi_sched = r % 3u; r /= 3u;
  const unsigned kernel_sched = r % 3u; r /= 3u;
  const unsigned cl = r % 15u; r /= 15u;
  const unsigned st = r % 11u; r /= 11u;
  const unsigned tk = r % 5u; r /= 5u;
  const unsigned tn = r % 9u; r /= 9u;
  const unsigned tm = r;
  // tile_n values {16,32,48,64,80,96,128,192,256} in units of 16: one hex digit each, 16 -> 0
  const unsigned tn16 = (0x0C8654321ull >> (4 * tn)) & 15u;
  // the 15 pairs (c_M, c_N) of powers of two with c_M c_N <= 16, c_M slowest: log2 per digit
  const unsigned lm = (0x433222111100000ull >> (4 * cl)) & 15u;
  const unsigned ln = (0x010210321043210ull >> (4 * cl)) & 15u;
  ks_candidate c;
  c.tile_m = static_cast<uint16_t>(64u * (tm + 1u));
  c.tile_n = static_cast<uint16_t>(tn == 8u ? 256u : 16u * tn16);
  c.tile_k = static_cast<uint16_t>(32u << tk);
  c.instr_n = c.tile_n;
  c.stages = static_cast<uint8_t>(2u + st);
  c.cluster_m = static_cast<uint8_t>(1u << lm);
  c.cluster_n = static_cast<uint8_t>(1u << ln);
  c.kernel_sched = static_cast<uint8_t>(kernel_sched);
  c.epi_sched = static_cast<uint8_t>(epi_sched);
  c.tile_sched = static_cast<uint8_t>(tile_sched);
  c.instr_m = 64;
  c.instr_k = 16;
  return c;
}

// What the predicate needs of the problem.
struct ValidArgs {
  int bA, bD;
  int a_col_major, b_row_major;
  unsigned two_m, two_n;  // 2M, 2N saturated to 32 bits (the wasteful-tile rule)
  unsigned flags;
};

// The five rules of the table, then the optional ones.
__device__ __forceinline__ bool is_valid(const ValidArgs& a, const ks_candidate& c, const ks_gpu_desc& h) {
  const bool coop = c.kernel_sched == 2;
  bool ok = !(c.tile_sched == 1 && !coop);                       // Stream-K => cooperative mainloop
  ok = ok && !(coop && (c.tile_m % 128u) != 0);                  // cooperative => T_M = 0 mod 128
  const SmemTerms sm = smem_terms(a.bA, a.bD, c, h);
  ok = ok && ((a.flags & KS_VALID_PRINTED_CAPACITY) ? sm.both : sm.B_smem) <= static_cast<long long>(h.smem_per_cta_max);  // capacity per CTA
  ok = ok && !(a.a_col_major && c.tile_k > 256u * c.cluster_n);  // A column-major: T_K <= 256 C_N
  ok = ok && !(a.b_row_major && c.tile_k > 256u * c.cluster_m);  // B row-major: T_K <= 256 C_M
  if (a.flags & KS_VALID_COUPLED) {
    ok = ok && !(c.epi_sched == 2 && !coop);
    ok = ok && !(c.epi_sched == 1 && coop);
  }
  if (a.flags & KS_VALID_WASTEFUL) ok = ok && c.tile_n <= a.two_m && c.tile_n <= a.two_n;
  return ok;
}

// 16-byte moves of a record without assuming more than its natural alignment for locals.
union CandidateBits {
  ks_candidate c;
  uint4 v;
};

__device__ __forceinline__ ks_candidate load_candidate(const ks_candidate* d_c, long long j) {
  if (!d_c) return decode_candidate(j);
  CandidateBits b;
  b.v = __ldg(reinterpret_cast<const uint4*>(d_c) + j);
  return b.c;
}

__device__ __forceinline__ void store_candidate(ks_candidate* d, long long j, const ks_candidate& c) {
  CandidateBits b;
  b.c = c;
  reinterpret_cast<uint4*>(d)[j] = b.v;
}

__global__ void __launch_bounds__(kCatThreads) enumerate_kernel(long long first, long long count,
                                                                ks_candidate* __restrict__ out) {
  for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < count;
       i += static_cast<long long>(gridDim.x) * blockDim.x)
    store_candidate(out, i, decode_candidate(first + i));
}

// kScatter false: block b writes how many of its candidates are valid to block_sums[b].
// kScatter true: block_sums holds the exclusive prefix; survivors go to out_c / out_index.
template <bool kScatter>
__global__ void __launch_bounds__(kCatThreads)
valid_kernel(const __grid_constant__ ks_gpu_desc desc, ValidArgs args, const ks_candidate* __restrict__ d_c,
             int C, int* __restrict__ block_sums, ks_candidate* __restrict__ out_c,
             int32_t* __restrict__ out_index) {
  __shared__ int s_warp[kCatThreads / 32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const long long base = static_cast<long long>(blockIdx.x) * kCatTile + threadIdx.x * kCatPerThread;
  ks_candidate c[kCatPerThread];
  unsigned mask = 0;
#pragma unroll
  for (int i = 0; i < kCatPerThread; ++i) {
    const long long j = base + i;
    if (j < C) {
      c[i] = load_candidate(d_c, j);
      if (is_valid(args, c[i], desc)) mask |= 1u << i;
    }
  }
  const int mine = __popc(mask);
  int incl = mine;  // inclusive prefix over the warp's lanes
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += v;
  }
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  int before = 0, total = 0;
#pragma unroll
  for (int w = 0; w < kCatThreads / 32; ++w) {
    const int v = s_warp[w];
    if (w < warp) before += v;
    total += v;
  }
  if (!kScatter) {
    if (threadIdx.x == 0) block_sums[blockIdx.x] = total;
    return;
  }
  int pos = block_sums[blockIdx.x] + before + incl - mine;
#pragma unroll
  for (int i = 0; i < kCatPerThread; ++i) {
    if (mask & (1u << i)) {
      if (out_c) store_candidate(out_c, pos, c[i]);
      if (out_index) out_index[pos] = static_cast<int32_t>(base + i);
      ++pos;
    }
  }
}

// One block: block_sums[0..n) -> exclusive prefix in place; the grand total goes to d_count.
__global__ void __launch_bounds__(1024) scan_block_sums_kernel(int* __restrict__ block_sums, int n,
                                                               int32_t* __restrict__ d_count) {
  __shared__ int s_warp[32];
  __shared__ int s_carry;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) s_carry = 0;
  __syncthreads();
  for (int lo = 0; lo < n; lo += 1024) {
    const int i = lo + threadIdx.x;
    const int v = i < n ? block_sums[i] : 0;
    int incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += u;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      int w = s_warp[lane];
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int u = __shfl_up_sync(0xffffffffu, w, d);
        if (lane >= d) w += u;
      }
      s_warp[lane] = w;  // inclusive prefix over warps
    }
    __syncthreads();
    const int carry = s_carry;
    const int before = warp ? s_warp[warp - 1] : 0;
    if (i < n) block_sums[i] = carry + before + incl - v;
    __syncthreads();
    if (threadIdx.x == 1023) s_carry = carry + s_warp[31];
    __syncthreads();
  }
  if (threadIdx.x == 0) *d_count = s_carry;
}

__global__ void remap_indices_kernel(int32_t* __restrict__ idx, long long n, const int32_t* __restrict__ map,
                                     int map_len) {
  for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < n;
       i += static_cast<long long>(gridDim.x) * blockDim.x) {
    const int32_t v = idx[i];
    idx[i] = (v >= 0 && v < map_len) ? __ldg(map + v) : -1;
  }
}

}  // namespace

cudaError_t launch_enumerate(long long first, long long count, ks_candidate* d_out, cudaStream_t stream,
                             int64_t* launches) {
  if (count == 0) return cudaSuccess;
  const long long want = (count + kCatThreads - 1) / kCatThreads;
  const unsigned grid = static_cast<unsigned>(want < 148 * 8 ? want : 148 * 8);
  enumerate_kernel<<<grid, kCatThreads, 0, stream>>>(first, count, d_out);
  ++*launches;
  return cudaGetLastError();
}

size_t valid_catalogue_scratch_bytes(int C) {
  return sizeof(int) * static_cast<size_t>((C + kCatTile - 1) / kCatTile + 1);
}

cudaError_t launch_valid_catalogue(const ks_gpu_desc& desc, const ks_problem& p, unsigned flags,
                                   const ks_candidate* d_c, int C, void* d_scratch, ks_candidate* d_out,
                                   int32_t* d_out_index, int32_t* d_count, cudaStream_t stream,
                                   int64_t* launches) {
  if (C == 0) return cudaMemsetAsync(d_count, 0, sizeof(int32_t), stream);
  ValidArgs a;
  const int dab = p.dtype_ab & 3, dd = p.dtype_d & 3;
  a.bA = dab == 2 ? 1 : (dab == 3 ? 4 : 2);
  a.bD = dd == 2 ? 1 : (dd == 3 ? 4 : 2);
  a.a_col_major = p.layout == 2 || p.layout == 3;
  a.b_row_major = p.layout == 1 || p.layout == 3;
  a.two_m = p.m > 0x7fffffffu ? 0xffffffffu : 2u * p.m;
  a.two_n = p.n > 0x7fffffffu ? 0xffffffffu : 2u * p.n;
  a.flags = flags;
  const int nblk = (C + kCatTile - 1) / kCatTile;
  int* sums = static_cast<int*>(d_scratch);
  valid_kernel<false><<<nblk, kCatThreads, 0, stream>>>(desc, a, d_c, C, sums, nullptr, nullptr);
  scan_block_sums_kernel<<<1, 1024, 0, stream>>>(sums, nblk, d_count);
  *launches += 2;
  if (d_out || d_out_index) {
    valid_kernel<true><<<nblk, kCatThreads, 0, stream>>>(desc, a, d_c, C, sums, d_out, d_out_index);
    ++*launches;
  }
  return cudaGetLastError();
}

cudaError_t launch_remap_indices(int32_t* d_idx, long long n, const int32_t* d_map, int map_len,
                                 cudaStream_t stream, int64_t* launches) {
  if (n == 0) return cudaSuccess;
  const long long want = (n + 255) / 256;
  const unsigned grid = static_cast<unsigned>(want < 148 * 8 ? want : 148 * 8);
  remap_indices_kernel<<<grid, 256, 0, stream>>>(d_idx, n, d_map, map_len);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace ks
