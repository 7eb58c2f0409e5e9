// Similarity order of a candidate catalogue.
//
// The quantised tree kernel keeps the four candidates of a tile word in one thread and can share
// one walk among them for as long as they take the same turns. They do so the more often the
// more alike they are, so the catalogue is ranked in an order in which neighbours differ in as
// few knobs as possible: sorted by (T_M, T_N, T_K, stages, c_M, c_N, kernel schedule, epilogue
// schedule, tile scheduler, instruction shape), most significant first. In a cross-product
// catalogue the four candidates of a word then differ only in the tile scheduler and the
// instruction shape. The order changes nothing in the results: ranking keys carry the pool index.
//
// The sort itself is a library primitive (cub::DeviceRadixSort) outside the hot loop: about
// 0.1 % of a batch step, and done once for a prepared catalogue.
#include <cub/device/device_radix_sort.cuh>

#include "ks_features.cuh"
#include "ks_internal.h"

namespace ks {

namespace {

__global__ void order_keys_kernel(const ks_candidate* __restrict__ c, int C, unsigned long long* __restrict__ keys,
                                  int* __restrict__ idx) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= C) return;
  const ks_candidate k = load_candidate(c + i);
  unsigned long long key = k.tile_m & 0xFFFu;
  key = (key << 12) | (k.tile_n & 0xFFFu);
  key = (key << 12) | (k.tile_k & 0xFFFu);
  key = (key << 4) | (k.stages & 0xFu);
  key = (key << 5) | (k.cluster_m & 0x1Fu);
  key = (key << 5) | (k.cluster_n & 0x1Fu);
  key = (key << 2) | (k.kernel_sched & 3u);
  key = (key << 2) | (k.epi_sched & 3u);
  key = (key << 1) | (k.tile_sched & 1u);
  key = (key << 1) | (k.instr_n != k.tile_n ? 1u : 0u);
  keys[i] = key;
  idx[i] = i;
}

constexpr int kKeyBits = 56;

size_t align256(size_t v) { return (v + 255) / 256 * 256; }

size_t cub_temp_bytes(int C) {
  size_t bytes = 0;
  cub::DeviceRadixSort::SortPairs(nullptr, bytes, static_cast<const unsigned long long*>(nullptr),
                                  static_cast<unsigned long long*>(nullptr), static_cast<const int*>(nullptr),
                                  static_cast<int*>(nullptr), C, 0, kKeyBits);
  return bytes;
}

}  // namespace

// scratch layout: order (the result, first) | keys in | keys out | indices in | sort workspace
size_t order_scratch_bytes(int C) {
  if (C < 1) return 0;
  return align256(sizeof(int) * C) + 2 * align256(sizeof(unsigned long long) * C) + align256(sizeof(int) * C) +
         align256(cub_temp_bytes(C));
}

// Writes the catalogue positions in similarity order to the front of `scratch` (C int32).
cudaError_t launch_catalogue_order(const ks_candidate* d_c, int C, void* scratch, cudaStream_t stream,
                                   int64_t* launches) {
  char* base = static_cast<char*>(scratch);
  int* order = reinterpret_cast<int*>(base);
  base += align256(sizeof(int) * C);
  unsigned long long* keys_in = reinterpret_cast<unsigned long long*>(base);
  base += align256(sizeof(unsigned long long) * C);
  unsigned long long* keys_out = reinterpret_cast<unsigned long long*>(base);
  base += align256(sizeof(unsigned long long) * C);
  int* idx_in = reinterpret_cast<int*>(base);
  base += align256(sizeof(int) * C);
  size_t temp = cub_temp_bytes(C);
  order_keys_kernel<<<(C + 255) / 256, 256, 0, stream>>>(d_c, C, keys_in, idx_in);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  e = cub::DeviceRadixSort::SortPairs(base, temp, keys_in, keys_out, idx_in, order, C, 0, kKeyBits, stream);
  *launches += 1;  // the key kernel (the sort launches the library's own kernels)
  return e;
}

}  // namespace ks
