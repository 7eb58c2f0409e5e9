// Ranking keys and the block / warp selection primitives of the segmented top-k.
//
// A (score, pool index) pair becomes one 64-bit key whose unsigned order is the ranking
// order of the selection rule: higher score first, lower index first among equal scores.
// Key 0 means "no candidate". Because keys are distinct, the j-th best key is the largest key
// below the (j-1)-th, so selection needs no removal step.
#pragma once

#include <cstdint>

namespace ks {

__device__ __forceinline__ unsigned long long make_key(float score, int idx) {
  unsigned u = __float_as_uint(score);
  u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  return (static_cast<unsigned long long>(u) << 32) | static_cast<unsigned>(~idx);
}

__device__ __forceinline__ int key_index(unsigned long long key) {
  return key == 0ull ? -1 : static_cast<int>(~static_cast<unsigned>(key));
}

__device__ __forceinline__ float key_score(unsigned long long key) {
  if (key == 0ull) return __uint_as_float(0xFF800000u);  // -inf
  unsigned u = static_cast<unsigned>(key >> 32);
  u = (u & 0x80000000u) ? (u & 0x7FFFFFFFu) : ~u;
  return __uint_as_float(u);
}

__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
  const unsigned hi = __reduce_max_sync(0xFFFFFFFFu, static_cast<unsigned>(v >> 32));
  const unsigned lo =
      __reduce_max_sync(0xFFFFFFFFu, static_cast<unsigned>(v >> 32) == hi ? static_cast<unsigned>(v) : 0u);
  return (static_cast<unsigned long long>(hi) << 32) | lo;
}

// A warp's running top-k list: lane j < k holds the j-th best key seen so far, the other lanes 0.
// Merges one new key per lane (0 = none) into it. Each round takes the warp's largest new key;
// the loop ends as soon as that key would not make the list, which after the first few calls is
// at once for almost every call. Keys are distinct, so the owner of the round's key is unique.
__device__ __forceinline__ void warp_topk_insert(unsigned long long& mine, unsigned long long v, int k) {
  const int lane = threadIdx.x & 31;
  for (;;) {
    const unsigned long long m = warp_max_u64(v);
    const unsigned long long kth = __shfl_sync(0xFFFFFFFFu, mine, k - 1);
    if (m <= kth) break;
    const int pos = __popc(__ballot_sync(0xFFFFFFFFu, mine > m));  // entries that stay ahead of m
    const unsigned long long up = __shfl_up_sync(0xFFFFFFFFu, mine, 1);
    if (lane == pos) mine = m;
    else if (lane > pos && lane < k) mine = up;
    if (v == m) v = 0ull;
  }
}

// The k largest of the block's keys (N per thread), descending, into s_list[0..k).
// Two levels: every warp first ranks its own keys (k rounds of warp-wide max, no block barrier;
// a warp that runs out of keys stops), then warp 0 merges the warps' sorted lists: lane w holds
// the head of warp w's list, a round takes the largest head and its lane moves on to the next
// entry. Equal keys (the same candidate listed twice) leave in the same round, so they are
// reported once. All threads of the block must call; s_warp needs n_warps * KS_MAX_K slots.
template <int N>
__device__ __forceinline__ void block_topk(const unsigned long long (&keys)[N], int k,
                                           unsigned long long* s_warp, unsigned long long* s_list) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  unsigned long long prev = ~0ull;
  for (int j = 0; j < k; ++j) {
    unsigned long long best = 0ull;
#pragma unroll
    for (int q = 0; q < N; ++q) {
      const unsigned long long v = keys[q];
      if (v < prev && v > best) best = v;
    }
    best = warp_max_u64(best);
    if (best == 0ull) {  // nothing left in this warp
      if (lane < k - j) s_warp[warp * k + j + lane] = 0ull;
      break;
    }
    if (lane == 0) s_warp[warp * k + j] = best;
    prev = best;
  }
  __syncthreads();
  if (warp == 0) {
    int next = 1;
    unsigned long long head = lane < n_warps ? s_warp[lane * k] : 0ull;
    for (int j = 0; j < k; ++j) {
      const unsigned long long m = warp_max_u64(head);
      if (lane == 0) s_list[j] = m;
      if (m == 0ull) {
        if (lane > j && lane < k) s_list[lane] = 0ull;
        break;
      }
      if (head == m) {
        head = next < k ? s_warp[lane * k + next] : 0ull;
        ++next;
      }
    }
  }
  __syncthreads();
}

}  // namespace ks
