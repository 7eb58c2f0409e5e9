// ks_select_trees_static: the fused tree select for callers that must not allocate.
//
// Who cannot allocate: a runtime that hands all device memory to its own pool at start-up (a
// later cudaMalloc simply fails), a caller in the middle of stream capture or of a latency
// critical stream-ordered pipeline (cudaMalloc and cudaFree synchronise the whole device),
// or a host that forbids driver allocations after initialisation. Those callers cannot
// create a ks_ctx or a ks_model either, since both own device buffers, so this entry point
// takes everything as plain device pointers and keeps the one piece of scratch the kernels
// need -- the per-block partial top-k lists -- in a fixed array inside the library image.
#include <mutex>

#include "ks_internal.h"

namespace ks {
int64_t select_generic_partial_keys(int P, int C, int k);
cudaError_t launch_select_generic_trees(const ks_gpu_desc& desc, const DevNode* d_nodes, const int* d_roots,
                                        int n_trees, float base, const ks_problem* d_p, int P,
                                        const ks_candidate* d_c, int C, int k, unsigned long long* partial,
                                        int32_t* d_topk_idx, float* d_topk_score, cudaStream_t stream);
}  // namespace ks

namespace {

// Partial top-k lists of every (problem, candidate block): 524,288 keys = 4 MiB, held by every
// GPU that loads the library until the process exits.
constexpr int64_t kStaticKeys = KS_STATIC_MAX_KEYS;
static __device__ __align__(256) unsigned long long g_static_keys[kStaticKeys];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
unsigned long long* g_keys_ptr[kMaxDevices] = {nullptr};

// The array's name is only a host-side stand-in: the device address has to be asked for, once
// per device, with that device current.
cudaError_t static_keys_address(int device, unsigned long long** out) {
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_keys_ptr[device]) {
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_keys);
    if (e != cudaSuccess) return e;
    g_keys_ptr[device] = static_cast<unsigned long long*>(p);
  }
  *out = g_keys_ptr[device];
  return cudaSuccess;
}

}  // namespace

extern "C" ks_status ks_select_trees_static(int cuda_device, const ks_gpu_desc* desc, const ks_problem* d_p, int P,
                                            const ks_candidate* d_c, int C, const ks_node_dev* d_nodes,
                                            const int32_t* d_tree_offsets, int n_trees, float base_score, int k,
                                            int32_t* d_topk_idx, float* d_topk_score, void* stream) {
  static_assert(sizeof(ks_node_dev) == sizeof(ks::DevNode), "device node layout");
  if (!desc || P < 0 || C < 0 || n_trees < 0 || k < 1 || k > KS_MAX_K) return KS_ERR_INVALID_ARG;
  if (cuda_device < 0 || cuda_device >= kMaxDevices) return KS_ERR_INVALID_ARG;
  if (!ks::valid_desc(*desc)) return KS_ERR_INVALID_ARG;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess) {
    cudaGetLastError();
    return KS_ERR_CUDA;
  }
  if (cuda_device >= n_dev) return KS_ERR_INVALID_ARG;
  if (P == 0) return KS_OK;
  if (!d_p || !d_topk_idx || !d_topk_score || (C > 0 && !d_c) || (n_trees > 0 && (!d_nodes || !d_tree_offsets)))
    return KS_ERR_INVALID_ARG;
  // sizes beyond the fixed scratch are refused before anything is launched
  if (ks::select_generic_partial_keys(P, C, k) > kStaticKeys) return KS_ERR_UNSUPPORTED;

  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return KS_ERR_CUDA;
  if (prev != cuda_device && cudaSetDevice(cuda_device) != cudaSuccess) {
    cudaGetLastError();
    return KS_ERR_CUDA;
  }
  unsigned long long* keys = nullptr;
  cudaError_t e = static_keys_address(cuda_device, &keys);
  if (e == cudaSuccess)
    e = ks::launch_select_generic_trees(*desc, reinterpret_cast<const ks::DevNode*>(d_nodes), d_tree_offsets, n_trees,
                                        base_score, d_p, P, d_c, C, k, keys, d_topk_idx, d_topk_score,
                                        static_cast<cudaStream_t>(stream));
  if (prev != cuda_device) cudaSetDevice(prev);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return KS_ERR_CUDA;
  }
  return KS_OK;
}
