// Classes of candidates that look alike to the per-pair columns (sections "Work Decomposition
// and Wave Quantization", "Memory Behavior", "Pipeline Balance"): those columns see a candidate
// only through (T_M, T_N, T_K, S, c_M, c_N) and its resident-block count, and a cross-product
// catalogue holds far fewer such classes than candidates (the schedules and the instruction
// shape do not enter). Per call every candidate is given its class: a slot of a hash table per
// element-type combination, filled with atomicCAS and linear probing; the slot also remembers
// one member. Whatever depends on (problem, per-pair columns) can then be evaluated once per
// (problem, class) from the member and looked up per pair. A candidate whose fields do not fit
// the key, or whose probe sequence runs out (more classes than slots), has no class and is
// evaluated in place.
#pragma once

#include <cstddef>
#include <cstdint>

#include <cuda_runtime.h>

#include "ks.h"

namespace ks {

constexpr int kMemoCombos = 16;  // dtype_ab x dtype_d
constexpr int kMemoCap = 8192;   // slots per type combination (a power of two)
constexpr int kMemoMinProblems = 32;
constexpr int kMemoMaxProblems = 8192;
constexpr unsigned kNoClass = 0xFFFFFFFFu;

struct MemoView {
  unsigned long long* keys;  // [kMemoCombos][kMemoCap], 0 = empty
  int* count;                // [kMemoCombos] occupied slots
  int* dense;                // [kMemoCombos][kMemoCap] the occupied slots, packed
  int* reps;                 // [kMemoCombos][kMemoCap] one member of the class
  unsigned* cls;             // [kMemoCombos][C]
  void* tab;                 // [P][kMemoCap] records of the caller's size
};

// bytes of everything but the per-problem records, and the view over a block of that size
// followed by the records
size_t memo_fixed_bytes(int C);
MemoView memo_view(void* mem, int C);
// zeroes the tables (before the kernel that assigns classes) / packs the occupied slots (after it)
cudaError_t memo_clear(const MemoView& memo, cudaStream_t stream);
cudaError_t memo_compact(const MemoView& memo, cudaStream_t stream);

#ifdef __CUDACC__
// Class of candidate i (of type combination `combo`, resident-block count b_eff), creating the
// slot when the candidate is the first of its class.
__device__ __forceinline__ unsigned memo_assign(const MemoView& memo, int combo, int i, const ks_candidate& cand,
                                                long long b_eff) {
  if (!(cand.tile_m < 4096 && cand.tile_n < 4096 && cand.tile_k < 4096 && cand.cluster_m < 32 &&
        cand.cluster_n < 32 && b_eff >= 0 && b_eff < 64))
    return kNoClass;
  const unsigned long long key =
      (1ull << 63) | cand.tile_m | (static_cast<unsigned long long>(cand.tile_n) << 12) |
      (static_cast<unsigned long long>(cand.tile_k) << 24) | (static_cast<unsigned long long>(cand.stages) << 36) |
      (static_cast<unsigned long long>(cand.cluster_m) << 44) | (static_cast<unsigned long long>(cand.cluster_n) << 49) |
      (static_cast<unsigned long long>(b_eff) << 54);
  unsigned long long* K = memo.keys + static_cast<size_t>(combo) * kMemoCap;
  unsigned h = static_cast<unsigned>((key * 0x9E3779B97F4A7C15ull) >> 40) & (kMemoCap - 1);
  for (int probe = 0; probe < 64; ++probe) {
    const unsigned long long prev = atomicCAS(K + h, 0ull, key);
    if (prev == 0ull) memo.reps[static_cast<size_t>(combo) * kMemoCap + h] = i;  // this thread made the slot
    if (prev == 0ull || prev == key) return h;
    h = (h + 1) & (kMemoCap - 1);
  }
  return kNoClass;
}
#endif

}  // namespace ks
