// Host side of the C ABI: argument checks, model validation and repacking, workspace
// management, launches. No exception or abort crosses the boundary.
#include <cmath>
#include <mutex>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "ks_internal.h"

namespace {

const char* const kFeatureNames[KS_F] = {
    "log2_m", "log2_n", "log2_k", "a_col_major", "b_row_major", "dtype_code", "bytes_in",
    "bytes_out", "has_bias", "act_code", "tile_m", "tile_n", "tile_k", "instr_m", "instr_n",
    "instr_k", "stages", "kernel_sched", "epi_sched", "uses_streamk", "cluster_m", "cluster_n",
    "cluster_size", "n_m", "n_n", "n_k", "n_tiles", "w_m", "w_n", "sm_subscription", "waves",
    "eta_last", "streamk_applicability", "cluster_pad_waste", "tiles_per_cluster_m",
    "tiles_per_cluster_n", "cluster_overshoot", "i_problem", "i_mainloop", "r_stream",
    "ws_frac_l2", "panel_a_frac_l2", "panel_b_frac_l2", "traffic_in", "traffic_in_cluster",
    "traffic_epi", "bytes_per_stage", "smem_mainloop", "smem_epi", "smem_total", "f_smem",
    "fits_smem", "r_proxy", "b_smem", "b_reg", "b_res", "occupancy", "t_producer_us",
    "t_consumer_us", "r_pc", "f_fill", "a_stage", "stages_x_fsmem"};

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
    if (prev != dev) ok = cudaSetDevice(dev) == cudaSuccess;
  }
  ~DeviceGuard() {
    int cur = -1;
    if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
  }
};

ks_status cuda_fail(ks_ctx* ctx, cudaError_t e, const char* what) {
  if (ctx) std::snprintf(ctx->err, sizeof(ctx->err), "%s: %s", what, cudaGetErrorString(e));
  cudaGetLastError();  // clear the sticky-free error state
  return e == cudaErrorMemoryAllocation ? KS_ERR_OOM : KS_ERR_CUDA;
}

ks_status ensure_workspace(ks_ctx* ctx, size_t bytes) {
  if (bytes <= ctx->ws_bytes) return KS_OK;
  if (ctx->ws) {
    cudaError_t e = cudaFree(ctx->ws);  // synchronises: nothing in flight still uses it
    ctx->ws = nullptr;
    ctx->ws_bytes = 0;
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaFree(workspace)");
  }
  const size_t want = bytes + bytes / 2 + (1u << 20);
  cudaError_t e = cudaMalloc(&ctx->ws, want);
  if (e != cudaSuccess) {
    ctx->ws = nullptr;
    return cuda_fail(ctx, e, "cudaMalloc(workspace)");
  }
  ctx->ws_bytes = want;
  return KS_OK;
}

}  // namespace

namespace ks {
bool valid_desc(const ks_gpu_desc& d) {
  if (!d.num_sms || !d.smem_per_sm || !d.smem_per_cta_max || !d.regs_per_sm || !d.max_threads_per_sm ||
      !d.max_ctas_per_sm || !d.l2_bytes || !d.tma_bytes_per_us || d.reserved0)
    return false;
  if (d.max_threads_per_sm < 384) return false;
  for (int i = 0; i < 4; ++i)
    if (!d.tc_flops_per_us_per_sm[i]) return false;
  return true;
}

cudaError_t ensure_dynamic_smem(const void* kernel, size_t bytes) {
  struct Entry {
    const void* kernel;
    int device;
    size_t bytes;
  };
  static Entry table[256];
  static int used = 0;
  static std::mutex mu;
  int device = 0;
  cudaError_t e = cudaGetDevice(&device);
  if (e != cudaSuccess) return e;
  std::lock_guard<std::mutex> lock(mu);
  Entry* hit = nullptr;
  for (int i = 0; i < used; ++i)
    if (table[i].kernel == kernel && table[i].device == device) hit = &table[i];
  if (hit && hit->bytes >= bytes) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes));
  if (e != cudaSuccess) return e;
  if (hit) hit->bytes = bytes;
  else if (used < 256) table[used++] = Entry{kernel, device, bytes};
  return cudaSuccess;
}
}  // namespace ks

namespace {

// Reads (and clears) the device status word; the stream must have been synchronised.
ks_status read_status(ks_ctx* ctx) {
  const int v = *static_cast<volatile int*>(ctx->h_status);
  if (v != 0) {
    *ctx->h_status = 0;
    // a failed launch may have left arrival counters of the slice mode behind
    if (ctx->d_counters) cudaMemset(ctx->d_counters, 0, sizeof(int) * (ks::kMaxSliceBlocks + 1));
    return static_cast<ks_status>(v);
  }
  return KS_OK;
}

inline size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }

template <typename T>
cudaError_t upload(T** dst, const T* src, size_t n) {
  *dst = nullptr;
  if (n == 0) return cudaSuccess;
  cudaError_t e = cudaMalloc(reinterpret_cast<void**>(dst), n * sizeof(T));
  if (e != cudaSuccess) return e;
  return cudaMemcpy(*dst, src, n * sizeof(T), cudaMemcpyHostToDevice);
}

// Checks one tree; returns its depth or -1.
int validate_tree(const ks_node_host* t, int64_t n) {
  if (n < 1 || n > 65535) return -1;
  std::vector<int> depth(n, -1);
  depth[0] = 0;
  int max_depth = 0;
  int64_t reached = 1;
  for (int64_t i = 0; i < n; ++i) {
    const ks_node_host& nd = t[i];
    if (depth[i] < 0) return -1;  // parents precede children, so an unreached node is an orphan
    if (nd.kind > KS_NODE_PARTITION) return -1;
    if (nd.kind == KS_NODE_PARTITION) {
      if (nd.feat == 0xFFFF) return -1;
      const int levels = ks::categorical_levels(nd.feat);
      uint32_t mask;
      std::memcpy(&mask, &nd.thr_or_leaf, 4);
      if (levels == 0 || mask == 0 || (mask >> levels) != 0) return -1;
    } else if (!std::isfinite(nd.thr_or_leaf)) {
      return -1;
    }
    if (nd.feat == 0xFFFF) continue;
    if (nd.feat >= KS_F) return -1;
    const int64_t l = nd.left;
    if (l <= i || l + 1 >= n) return -1;
    if (depth[l] >= 0 || depth[l + 1] >= 0) return -1;  // a node has exactly one parent
    depth[l] = depth[l + 1] = depth[i] + 1;
    reached += 2;
    if (depth[i] + 1 > max_depth) max_depth = depth[i] + 1;
  }
  if (reached != n || max_depth > KS_MAX_DEPTH) return -1;
  return max_depth;
}

void free_model(ks_model* m) {
  if (!m) return;
  DeviceGuard g(m->device);  // not m->ctx: a model may be destroyed after its context
  cudaFree(m->gbdt.d_nodes);
  cudaFree(m->gbdt.d_roots);
  cudaFree(m->gbdt.d_qnodes);
  cudaFree(m->gbdt.d_qthr);
  cudaFree(m->gbdt.d_qfeat);
  ks::free_fast_gbdt(m->gbdt);
  for (int l = 0; l < KS_MLP_MAX_LAYERS; ++l) {
    cudaFree(m->mlp.d_w[l]);
    cudaFree(m->mlp.d_b[l]);
  }
  cudaFree(m->mlp.d_mu);
  cudaFree(m->mlp.d_sigma);
  cudaFree(m->mlp.d_tc_image);
  cudaFree(m->mlp.d_w1_prob);
  ks::free_fast_mlp(m->mlp);
  ks::free_ridge(m->mlp);
  delete m;
}

ks_status check_pairs(int P, int C, const void* seg_off, const void* seg_idx, int64_t pairs) {
  if (P < 0 || C < 0 || pairs < 0) return KS_ERR_INVALID_ARG;
  if ((seg_off == nullptr) != (seg_idx == nullptr) && pairs > 0) return KS_ERR_INVALID_ARG;
  if (!seg_off && pairs != static_cast<int64_t>(P) * C) return KS_ERR_INVALID_ARG;
  return KS_OK;
}

// problem and candidate records are fetched with 128-bit loads
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" {

const char* ks_status_string(ks_status s) {
  switch (s) {
    case KS_OK: return "ok";
    case KS_ERR_INVALID_ARG: return "invalid argument";
    case KS_ERR_UNSUPPORTED: return "unsupported";
    case KS_ERR_CUDA: return "CUDA error";
    case KS_ERR_TIMEOUT: return "device-side wait timed out";
    case KS_ERR_OOM: return "out of memory";
    default: return "unknown status";
  }
}

int ks_feature_count(void) { return KS_F; }

const char* ks_feature_name(int index) {
  return (index >= 0 && index < KS_F) ? kFeatureNames[index] : nullptr;
}

ks_status ks_create(ks_ctx** out_ctx, int cuda_device, const ks_gpu_desc* desc) {
  if (!out_ctx) return KS_ERR_INVALID_ARG;
  *out_ctx = nullptr;
  if (!desc || !ks::valid_desc(*desc)) return KS_ERR_INVALID_ARG;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess) {
    cudaGetLastError();
    return KS_ERR_CUDA;
  }
  if (cuda_device < 0 || cuda_device >= n_dev) return KS_ERR_INVALID_ARG;
  DeviceGuard g(cuda_device);
  if (!g.ok) return KS_ERR_CUDA;
  ks_ctx* ctx = new (std::nothrow) ks_ctx();
  if (!ctx) return KS_ERR_OOM;
  ctx->device = cuda_device;
  ctx->desc = *desc;
  ctx->pinned_bytes = KS_MAX_K * (sizeof(int32_t) + sizeof(float)) + 64;  // results + the sequence word
  // result staging of ks_select_one: mapped pinned memory, so the kernel's last block can
  // write the k results where the host reads them, with no copy in between
  void* d_pin = nullptr;
  if (cudaHostAlloc(&ctx->pinned, ctx->pinned_bytes, cudaHostAllocMapped) != cudaSuccess ||
      cudaHostGetDevicePointer(&d_pin, ctx->pinned, 0) != cudaSuccess) {
    cudaGetLastError();
    if (ctx->pinned) cudaFreeHost(ctx->pinned);
    delete ctx;
    return KS_ERR_OOM;
  }
  std::memset(ctx->pinned, 0, ctx->pinned_bytes);
  ctx->d_pinned_idx = static_cast<int32_t*>(d_pin);
  ctx->d_pinned_score = reinterpret_cast<float*>(ctx->d_pinned_idx + KS_MAX_K);
  if (cudaMalloc(reinterpret_cast<void**>(&ctx->d_counters), sizeof(int) * (ks::kMaxSliceBlocks + 1)) != cudaSuccess ||
      cudaMemset(ctx->d_counters, 0, sizeof(int) * (ks::kMaxSliceBlocks + 1)) != cudaSuccess) {
    cudaGetLastError();
    cudaFree(ctx->d_counters);
    cudaFreeHost(ctx->pinned);
    delete ctx;
    return KS_ERR_OOM;
  }
  ks_status s = ensure_workspace(ctx, 1u << 20);
  // status word in mapped pinned host memory: kernels write it through d_status, the host
  // reads h_status after a synchronisation without issuing a copy
  if (s == KS_OK && (cudaHostAlloc(reinterpret_cast<void**>(&ctx->h_status), sizeof(int), cudaHostAllocMapped) != cudaSuccess ||
                     cudaHostGetDevicePointer(reinterpret_cast<void**>(&ctx->d_status), ctx->h_status, 0) != cudaSuccess)) {
    cudaGetLastError();
    s = KS_ERR_OOM;
  }
  if (s == KS_OK) *ctx->h_status = 0;
  if (s != KS_OK) {
    cudaFree(ctx->ws);
    cudaFree(ctx->d_counters);
    if (ctx->h_status) cudaFreeHost(ctx->h_status);
    cudaFreeHost(ctx->pinned);
    delete ctx;
    return s;
  }
  *out_ctx = ctx;
  return KS_OK;
}

ks_status ks_destroy(ks_ctx* ctx) {
  if (!ctx) return KS_OK;
  DeviceGuard g(ctx->device);
  if (ctx->ev_begin) cudaEventDestroy(ctx->ev_begin);
  if (ctx->ev_end) cudaEventDestroy(ctx->ev_end);
  cudaFree(ctx->ws);
  cudaFree(ctx->d_counters);
  cudaFreeHost(ctx->h_status);
  cudaFreeHost(ctx->pinned);
  delete ctx;
  return KS_OK;
}

const char* ks_last_cuda_error(const ks_ctx* ctx) { return ctx ? ctx->err : ""; }

int64_t ks_launch_count(const ks_ctx* ctx) { return ctx ? ctx->launches : 0; }

ks_status ks_device_status(ks_ctx* ctx) {
  if (!ctx) return KS_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "ks_device_status");
  return read_status(ctx);
}

ks_status ks_profile_enable(ks_ctx* ctx, int on) {
  if (!ctx) return KS_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (on && !ctx->ev_begin) {
    cudaError_t e = cudaEventCreate(&ctx->ev_begin);
    if (e == cudaSuccess) e = cudaEventCreate(&ctx->ev_end);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "ks_profile_enable");
  }
  ctx->profile = on != 0;
  ctx->profile_valid = false;
  return KS_OK;
}

ks_status ks_profile_last_ms(ks_ctx* ctx, float* out_ms) {
  if (!ctx || !out_ms || !ctx->profile_valid) return KS_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  cudaError_t e = cudaEventSynchronize(ctx->ev_end);
  if (e == cudaSuccess) e = cudaEventElapsedTime(out_ms, ctx->ev_begin, ctx->ev_end);
  return e == cudaSuccess ? KS_OK : cuda_fail(ctx, e, "ks_profile_last_ms");
}

ks_status ks_merge_topk(ks_ctx* ctx, const int32_t* d_idx, const float* d_score, int P, int n, int k,
                        int32_t* d_topk_idx, float* d_topk_score, void* stream) {
  if (!ctx || P < 0 || n < 0 || k < 1 || k > KS_MAX_K) return KS_ERR_INVALID_ARG;
  if (P == 0) return KS_OK;
  if (!d_topk_idx || !d_topk_score || (n > 0 && (!d_idx || !d_score))) return KS_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  cudaError_t e = ks::launch_merge_lists(d_idx, d_score, P, n, k, d_topk_idx, d_topk_score,
                                         static_cast<cudaStream_t>(stream), &ctx->launches);
  return e == cudaSuccess ? KS_OK : cuda_fail(ctx, e, "ks_merge_topk");
}

ks_status ks_model_describe(const ks_model* model, char* buf, int len) {
  if (!model || !buf || len < 1) return KS_ERR_INVALID_ARG;
  if (model->kind == 0 && model->gbdt.fast) {
    const ks::GbdtModel& g = model->gbdt;
    std::snprintf(buf, len,
                  "select_fast_kernel threads=%d block=%d rows=%d thresholds=%d top_levels=%d%s trees=%d depth=%d "
                  "chunks=%d chunk_trees=%d",
                  g.fast_threads, g.block_cands, g.n_qrows, g.n_qthr, g.top_levels, g.top_compact ? "c" : "",
                  g.n_trees, g.fast_depth, g.n_chunks, g.tpc);
  } else if (model->kind == 0) {
    std::snprintf(buf, len, "select_generic_kernel trees=%d depth=%d", model->gbdt.n_trees, model->gbdt.max_depth);
  } else if (model->kind == 1 && model->mlp.tc) {
    std::snprintf(buf, len, "select_mlp_tc_kernel");
  } else if (model->kind == 1 && model->mlp.h_ridge) {
    std::snprintf(buf, len, "select_ridge_kernel");
  } else if (model->kind == 1) {
    std::snprintf(buf, len, "select_generic_kernel mlp layers=%d", model->mlp.n_layers);
  } else {
    std::snprintf(buf, len, "select_generic_kernel static score");
  }
  return KS_OK;
}

ks_status ks_debug_set_wait(ks_ctx* ctx, int probe_limit, int starve) {
  if (!ctx || probe_limit < 0) return KS_ERR_INVALID_ARG;
  ctx->wait.limit = probe_limit;
  ctx->wait.starve = starve != 0;
  return KS_OK;
}

int ks_debug_bounds_line(void) {
  cudaDeviceSynchronize();
  return ks::fast_bounds_line();
}

void ks_debug_bounds_clear(void) {
  cudaDeviceSynchronize();
  ks::fast_bounds_clear();
}

ks_status ks_model_create_gbdt(ks_ctx* ctx, int n_trees, const int64_t* h_tree_offsets,
                               const ks_node_host* h_nodes, float base_score, ks_model** out_model) {
  if (!out_model) return KS_ERR_INVALID_ARG;
  *out_model = nullptr;
  if (!ctx || n_trees < 0 || !h_tree_offsets || (n_trees > 0 && !h_nodes) || !std::isfinite(base_score))
    return KS_ERR_INVALID_ARG;
  if (h_tree_offsets[0] != 0) return KS_ERR_INVALID_ARG;
  const int64_t total = h_tree_offsets[n_trees];
  if (total < 0 || total > (1ll << 31) - 1) return KS_ERR_INVALID_ARG;
  int max_depth = 0;
  for (int t = 0; t < n_trees; ++t) {
    const int64_t lo = h_tree_offsets[t], hi = h_tree_offsets[t + 1];
    if (hi <= lo) return KS_ERR_INVALID_ARG;
    const int d = validate_tree(h_nodes + lo, hi - lo);
    if (d < 0) return KS_ERR_INVALID_ARG;
    if (d > max_depth) max_depth = d;
  }
  std::vector<ks::DevNode> dev(static_cast<size_t>(total));
  for (int64_t i = 0; i < total; ++i) {
    dev[i].v = h_nodes[i].thr_or_leaf;
    dev[i].feat = h_nodes[i].kind == KS_NODE_PARTITION ? static_cast<uint16_t>(h_nodes[i].feat | 0x8000u)
                                                       : h_nodes[i].feat;
    dev[i].left = h_nodes[i].feat == 0xFFFF ? 0 : static_cast<uint16_t>(h_nodes[i].left);
  }
  std::vector<int> roots(n_trees + 1);
  for (int t = 0; t <= n_trees; ++t) roots[t] = static_cast<int>(h_tree_offsets[t]);

  DeviceGuard g(ctx->device);
  ks_model* m = new (std::nothrow) ks_model();
  if (!m) return KS_ERR_OOM;
  m->ctx = ctx;
  m->device = ctx->device;
  m->kind = 0;
  m->gbdt.n_trees = n_trees;
  m->gbdt.max_depth = max_depth;
  m->gbdt.n_nodes = total;
  m->gbdt.base = base_score;
  cudaError_t e = upload(&m->gbdt.d_nodes, dev.data(), dev.size());
  if (e == cudaSuccess) e = upload(&m->gbdt.d_roots, roots.data(), roots.size());
  if (e == cudaSuccess) e = ks::build_fast_gbdt(m->gbdt, n_trees, h_tree_offsets, h_nodes);
  if (e != cudaSuccess) {
    ks_status s = cuda_fail(ctx, e, "ks_model_create_gbdt");
    free_model(m);
    return s;
  }
  *out_model = m;
  return KS_OK;
}

ks_status ks_model_create_mlp(ks_ctx* ctx, int n_layers, const int* h_widths,
                              const uint16_t* const* h_w_bf16, const float* const* h_bias,
                              const float* h_mu, const float* h_sigma, ks_model** out_model) {
  if (!out_model) return KS_ERR_INVALID_ARG;
  *out_model = nullptr;
  if (!ctx || !h_widths || !h_w_bf16 || !h_bias || !h_mu || !h_sigma) return KS_ERR_INVALID_ARG;
  if (n_layers < 1 || n_layers > KS_MLP_MAX_LAYERS) return KS_ERR_INVALID_ARG;
  const int in0 = h_widths[0];
  if ((in0 != KS_F_PAD && in0 != KS_F_ONEHOT) || h_widths[n_layers] != 1) return KS_ERR_INVALID_ARG;
  int max_width = in0;
  for (int l = 1; l < n_layers; ++l) {
    if (h_widths[l] < 64 || h_widths[l] > KS_MLP_MAX_WIDTH || h_widths[l] % 64) return KS_ERR_INVALID_ARG;
    if (h_widths[l] > max_width) max_width = h_widths[l];
  }
  for (int l = 0; l < n_layers; ++l)
    if (!h_w_bf16[l] || !h_bias[l]) return KS_ERR_INVALID_ARG;
  for (int j = 0; j < in0; ++j)
    if (!std::isfinite(h_mu[j]) || !std::isfinite(h_sigma[j]) || h_sigma[j] == 0.0f) return KS_ERR_INVALID_ARG;

  DeviceGuard g(ctx->device);
  ks_model* m = new (std::nothrow) ks_model();
  if (!m) return KS_ERR_OOM;
  m->ctx = ctx;
  m->device = ctx->device;
  m->kind = 1;
  m->mlp.n_layers = n_layers;
  m->mlp.max_width = max_width;
  for (int l = 0; l <= n_layers; ++l) m->mlp.widths[l] = h_widths[l];
  cudaError_t e = cudaSuccess;
  for (int l = 0; l < n_layers && e == cudaSuccess; ++l) {
    const size_t n = static_cast<size_t>(h_widths[l]) * h_widths[l + 1];
    e = upload(&m->mlp.d_w[l], h_w_bf16[l], n);
    if (e == cudaSuccess) e = upload(&m->mlp.d_b[l], h_bias[l], static_cast<size_t>(h_widths[l + 1]));
  }
  if (e == cudaSuccess) e = upload(&m->mlp.d_mu, h_mu, static_cast<size_t>(in0));
  if (e == cudaSuccess) e = upload(&m->mlp.d_sigma, h_sigma, static_cast<size_t>(in0));
  if (e == cudaSuccess) e = ks::build_fast_mlp(m->mlp, h_w_bf16, h_bias, h_mu, h_sigma);
  if (e == cudaSuccess) e = ks::build_ridge(m->mlp, h_w_bf16[0], h_bias[0], h_mu, h_sigma);
  if (e != cudaSuccess) {
    ks_status s = cuda_fail(ctx, e, "ks_model_create_mlp");
    free_model(m);
    return s;
  }
  *out_model = m;
  return KS_OK;
}

ks_status ks_model_create_static(ks_ctx* ctx, ks_model** out_model) {
  if (!out_model) return KS_ERR_INVALID_ARG;
  *out_model = nullptr;
  if (!ctx) return KS_ERR_INVALID_ARG;
  ks_model* m = new (std::nothrow) ks_model();
  if (!m) return KS_ERR_OOM;
  m->ctx = ctx;
  m->device = ctx->device;
  m->kind = 2;
  *out_model = m;
  return KS_OK;
}

ks_status ks_model_destroy(ks_model* model) {
  free_model(model);
  return KS_OK;
}

ks_status ks_enumerate(ks_ctx* ctx, int64_t first, int64_t count, ks_candidate* d_out, void* stream) {
  if (!ctx || first < 0 || count < 0 || first > KS_CATALOGUE_SIZE || count > KS_CATALOGUE_SIZE - first)
    return KS_ERR_INVALID_ARG;
  if (count == 0) return KS_OK;
  if (!d_out || (reinterpret_cast<uintptr_t>(d_out) & 15u)) return KS_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  cudaError_t e = ks::launch_enumerate(first, count, d_out, static_cast<cudaStream_t>(stream), &ctx->launches);
  return e == cudaSuccess ? KS_OK : cuda_fail(ctx, e, "ks_enumerate");
}

ks_status ks_valid_catalogue(ks_ctx* ctx, const ks_problem* problem, unsigned flags,
                             const ks_candidate* d_candidates, int C, ks_candidate* d_out,
                             int32_t* d_out_index, int32_t* d_count, int32_t* h_count, void* stream) {
  if (!ctx || !problem || !d_count || C < 0) return KS_ERR_INVALID_ARG;
  if (flags & ~(KS_VALID_COUPLED | KS_VALID_WASTEFUL | KS_VALID_PRINTED_CAPACITY)) return KS_ERR_INVALID_ARG;
  if (problem->layout > 3 || problem->dtype_ab > 3 || problem->dtype_d > 3) return KS_ERR_INVALID_ARG;
  if (!d_candidates && C > KS_CATALOGUE_SIZE) return KS_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_candidates) & 15u) || (reinterpret_cast<uintptr_t>(d_out) & 15u))
    return KS_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ks_status s = ensure_workspace(ctx, ks::valid_catalogue_scratch_bytes(C));
  if (s != KS_OK) return s;
  cudaError_t e = ks::launch_valid_catalogue(ctx->desc, *problem, flags, d_candidates, C, ctx->ws, d_out,
                                             d_out_index, d_count, st, &ctx->launches);
  if (e == cudaSuccess && h_count) {
    e = cudaMemcpyAsync(h_count, d_count, sizeof(int32_t), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  }
  return e == cudaSuccess ? KS_OK : cuda_fail(ctx, e, "ks_valid_catalogue");
}

ks_status ks_remap_indices(ks_ctx* ctx, int32_t* d_idx, int64_t n, const int32_t* d_map, int map_len,
                           void* stream) {
  if (!ctx || n < 0 || map_len < 0) return KS_ERR_INVALID_ARG;
  if (n == 0) return KS_OK;
  if (!d_idx || (map_len > 0 && !d_map)) return KS_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  cudaError_t e = ks::launch_remap_indices(d_idx, n, d_map, map_len, static_cast<cudaStream_t>(stream),
                                           &ctx->launches);
  return e == cudaSuccess ? KS_OK : cuda_fail(ctx, e, "ks_remap_indices");
}

ks_status ks_featurize(ks_ctx* ctx, const ks_problem* d_p, int P, const ks_candidate* d_c, int C,
                       const int64_t* d_seg_offsets, const int32_t* d_seg_index, int64_t pairs,
                       float* d_features, void* stream) {
  if (!ctx) return KS_ERR_INVALID_ARG;
  ks_status s = check_pairs(P, C, d_seg_offsets, d_seg_index, pairs);
  if (s != KS_OK) return s;
  if (pairs == 0) return KS_OK;
  if (!d_p || !d_c || !d_features || !aligned16(d_p) || !aligned16(d_c)) return KS_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  s = ensure_workspace(ctx, ks::featurize_scratch_bytes(P));
  if (s != KS_OK) return s;
  cudaError_t e = ks::launch_featurize(ctx->desc, d_p, P, d_c, C, d_seg_offsets, d_seg_index, pairs,
                                       d_features, ctx->ws, static_cast<cudaStream_t>(stream), &ctx->launches);
  return e == cudaSuccess ? KS_OK : cuda_fail(ctx, e, "ks_featurize");
}

ks_status ks_debug_walk_floor(ks_ctx* ctx, const float* d_features, int64_t rows, const ks_model* model,
                              int repeat, float* d_scores, void* stream) {
  if (!ctx || !model || model->ctx != ctx || rows < 1 || repeat < 1 || repeat > 4096) return KS_ERR_INVALID_ARG;
  if (!d_features || !d_scores) return KS_ERR_INVALID_ARG;
  if (model->kind != 0 || !model->gbdt.fast) return KS_ERR_UNSUPPORTED;
  DeviceGuard g(ctx->device);
  ks_status s = ensure_workspace(ctx, ks::score_fast_scratch_bytes(model->gbdt, rows));
  if (s != KS_OK) return s;
  cudaError_t e = ks::launch_score_fast(ctx->desc, model->gbdt, d_features, rows, d_scores, ctx->ws, ctx->d_status,
                                        static_cast<cudaStream_t>(stream), &ctx->launches, &ctx->wait, repeat);
  if (e == cudaErrorNotSupported) return KS_ERR_UNSUPPORTED;
  return e == cudaSuccess ? KS_OK : cuda_fail(ctx, e, "ks_debug_walk_floor");
}

ks_status ks_score(ks_ctx* ctx, const float* d_features, int64_t rows, const ks_model* model,
                   float* d_scores, uint16_t* d_leaf_idx, void* stream) {
  if (!ctx || !model || model->ctx != ctx || rows < 0) return KS_ERR_INVALID_ARG;
  if (rows == 0) return KS_OK;
  if (!d_features || !d_scores) return KS_ERR_INVALID_ARG;
  if (model->kind == 2) return KS_ERR_UNSUPPORTED;  // the static score is a function of (p, c), not of x
  if (model->kind == 1 && d_leaf_idx) return KS_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (model->kind == 0 && model->gbdt.fast && !d_leaf_idx) {
    // quantised path: the same walk as ks_select, on tiles built from the given rows
    ks_status s = ensure_workspace(ctx, ks::score_fast_scratch_bytes(model->gbdt, rows));
    if (s != KS_OK) return s;
    cudaError_t e = ks::launch_score_fast(ctx->desc, model->gbdt, d_features, rows, d_scores, ctx->ws,
                                          ctx->d_status, static_cast<cudaStream_t>(stream), &ctx->launches,
                                          &ctx->wait);
    return e == cudaSuccess ? KS_OK : cuda_fail(ctx, e, "ks_score");
  }
  if (model->kind == 1 && ks::score_mlp_tc_ok(model->mlp)) {
    cudaError_t e = ks::launch_score_mlp_tc(ctx->desc, model->mlp, d_features, rows, d_scores, ctx->d_status,
                                            static_cast<cudaStream_t>(stream), &ctx->launches, &ctx->wait);
    return e == cudaSuccess ? KS_OK : cuda_fail(ctx, e, "ks_score");
  }
  cudaError_t e =
      model->kind == 0
          ? ks::launch_score_gbdt(model->gbdt, d_features, rows, d_scores, d_leaf_idx,
                                  static_cast<cudaStream_t>(stream), &ctx->launches)
          : ks::launch_score_mlp(model->mlp, d_features, rows, d_scores,
                                 static_cast<cudaStream_t>(stream), &ctx->launches);
  return e == cudaSuccess ? KS_OK : cuda_fail(ctx, e, "ks_score");
}

ks_status ks_select(ks_ctx* ctx, const ks_problem* d_p, int P, const ks_candidate* d_c, int C,
                    const int64_t* d_seg_offsets, const int32_t* d_seg_index, int64_t pairs,
                    const ks_model* model, int k, int32_t* d_topk_idx, float* d_topk_score,
                    void* stream) {
  if (!ctx || !model || model->ctx != ctx || k < 1 || k > KS_MAX_K) return KS_ERR_INVALID_ARG;
  ks_status s = check_pairs(P, C, d_seg_offsets, d_seg_index, pairs);
  if (s != KS_OK) return s;
  if (P == 0) return KS_OK;
  if (!d_p || !d_topk_idx || !d_topk_score || (pairs > 0 && !d_c)) return KS_ERR_INVALID_ARG;
  if (!aligned16(d_p) || !aligned16(d_c)) return KS_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  s = ensure_workspace(ctx, ks::select_partial_bytes(*model, P, C, pairs, d_seg_offsets != nullptr, k));
  if (s != KS_OK) return s;
  cudaError_t e = ks::launch_select(ctx->desc, *model, d_p, nullptr, P, d_c, C, d_seg_offsets,
                                    d_seg_index, pairs, k, ctx->ws, d_topk_idx, d_topk_score,
                                    static_cast<cudaStream_t>(stream), &ctx->launches, ctx->d_status,
                                    ctx->profile ? ctx->ev_begin : nullptr,
                                    ctx->profile ? ctx->ev_end : nullptr, ctx->d_counters, &ctx->wait);
  ctx->profile_valid = ctx->profile && e == cudaSuccess;
  return e == cudaSuccess ? KS_OK : cuda_fail(ctx, e, "ks_select");
}

ks_status ks_select_one(ks_ctx* ctx, ks_problem p, const ks_candidate* d_c, int C, const ks_model* model,
                        int k, int32_t* h_topk_idx, float* h_topk_score, void* stream) {
  if (!ctx || !model || model->ctx != ctx || k < 1 || k > KS_MAX_K || C < 0) return KS_ERR_INVALID_ARG;
  if (!h_topk_idx || !h_topk_score || (C > 0 && !d_c) || !aligned16(d_c)) return KS_ERR_INVALID_ARG;
  if (p.m < 1 || p.n < 1 || p.k < 1 || p.m > KS_MAX_DIM || p.n > KS_MAX_DIM || p.k > KS_MAX_DIM ||
      p.layout > 3 || p.dtype_ab > 3 || p.dtype_d > 3 || p.epi_flags > 5)
    return KS_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t* pin_idx = static_cast<int32_t*>(ctx->pinned);
  float* pin_sc = reinterpret_cast<float*>(pin_idx + KS_MAX_K);

  // Latency path for a qualifying tree model: the trees are split over several CTAs per
  // candidate block, the last block writes the k results straight into mapped host memory.
  if (model->kind == 0 && model->gbdt.fast && C > 0) {
    const int NC = model->gbdt.block_cands;
    const int nblk = (C + NC - 1) / NC;
    const int S = ks::fast_slices(model->gbdt, nblk);
    if (S > 1) {
      const size_t b_part = align_up(sizeof(unsigned long long) * nblk * k);
      // scratch of this path: the prepared tiles, one per candidate block (no per-call table)
      const size_t b_scratch = align_up(static_cast<size_t>(nblk) * model->gbdt.n_qrows * NC);
      const size_t b_scores = align_up(sizeof(float) * static_cast<size_t>(S) * C);
      ks_status s = ensure_workspace(ctx, b_part + b_scratch + b_scores);
      if (s != KS_OK) return s;
      char* base = static_cast<char*>(ctx->ws);
      ks::FastSlice sl;
      sl.n_slices = S;
      sl.pairs = C;
      sl.scores = reinterpret_cast<float*>(base + b_part + b_scratch);
      sl.counters = ctx->d_counters;
      sl.out_idx = ctx->d_pinned_idx;
      sl.out_score = ctx->d_pinned_score;
      sl.tiles = reinterpret_cast<uint8_t*>(base + b_part);
      // the kernel stores this call's sequence number after the results; polling that word
      // returns a few microseconds before the stream reports completion
      int* h_seq = reinterpret_cast<int*>(pin_sc + KS_MAX_K);
      sl.out_seq = reinterpret_cast<int*>(ctx->d_pinned_score + KS_MAX_K);
      sl.seq = ++ctx->select_one_seq;
      cudaError_t e = ks::launch_select_fast(ctx->desc, model->gbdt, nullptr, &p, 1, d_c, C, nblk, NC,
                                             nullptr, nullptr, k, reinterpret_cast<unsigned long long*>(base),
                                             base + b_part, ctx->d_status, st, &ctx->launches, nullptr, &sl, nullptr,
                                             &ctx->wait);
      if (e == cudaSuccess) {
        bool seen = false;
        for (int spin = 0; spin < (1 << 22) && !seen; ++spin) seen = *static_cast<volatile int*>(h_seq) == sl.seq;
        // not seen within a few milliseconds (a failed launch never writes it): wait the regular way
        if (!seen) e = cudaStreamSynchronize(st);
      }
      if (e != cudaSuccess) return cuda_fail(ctx, e, "ks_select_one");
      s = read_status(ctx);
      if (s != KS_OK) {
        cudaMemset(ctx->d_counters, 0, sizeof(int) * (ks::kMaxSliceBlocks + 1));
        return s;
      }
      std::memcpy(h_topk_idx, pin_idx, k * sizeof(int32_t));
      std::memcpy(h_topk_score, pin_sc, k * sizeof(float));
      return KS_OK;
    }
  }

  // every other model: the general path with one problem; its merge kernel writes the k results
  // straight into the mapped host block, so there is no copy between the kernel and the caller
  const size_t part = align_up(ks::select_partial_bytes(*model, 1, C, C, false, k));
  ks_status s = ensure_workspace(ctx, part);
  if (s != KS_OK) return s;
  cudaError_t e = ks::launch_select(ctx->desc, *model, nullptr, &p, 1, d_c, C, nullptr, nullptr, C, k,
                                    ctx->ws, ctx->d_pinned_idx, ctx->d_pinned_score, st, &ctx->launches,
                                    ctx->d_status, nullptr, nullptr, nullptr, &ctx->wait);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "ks_select_one");
  std::memcpy(h_topk_idx, pin_idx, k * sizeof(int32_t));
  std::memcpy(h_topk_score, pin_sc, k * sizeof(float));
  return read_status(ctx);
}

ks_status ks_catalogue_prepare(ks_ctx* ctx, const ks_candidate* d_c, int C, const ks_model* model,
                               ks_catalogue** out_catalogue, void* stream) {
  if (!out_catalogue) return KS_ERR_INVALID_ARG;
  *out_catalogue = nullptr;
  if (!ctx || !model || model->ctx != ctx || C < 0 || (C > 0 && !d_c) || !aligned16(d_c)) return KS_ERR_INVALID_ARG;
  ks_catalogue* cat = new (std::nothrow) ks_catalogue();
  if (!cat) return KS_ERR_OOM;
  cat->ctx = ctx;
  cat->model = model;
  cat->d_c = d_c;
  cat->C = C;
  cat->device = ctx->device;
  const ks::GbdtModel& g = model->gbdt;
  if (model->kind == 0 && g.fast && C > 0) {
    const int nblk = (C + g.block_cands - 1) / g.block_cands;
    const int S = ks::fast_slices(g, nblk);
    const size_t b_memo = ks::fast_prepared_memo_bytes(g, C);
    if (S > 1 && b_memo > 0) {
      DeviceGuard guard(ctx->device);
      const size_t b_rows = align_up(ks::fast_prepared_rows_bytes(g, C));
      const size_t b_part = align_up(sizeof(unsigned long long) * nblk * KS_MAX_K);
      const size_t b_scores = align_up(sizeof(float) * static_cast<size_t>(S) * C);
      cat->off_memo = b_rows;
      cat->off_part = b_rows + align_up(b_memo);
      cat->off_scores = cat->off_part + b_part;
      cat->off_order = cat->off_scores + b_scores;
      cudaError_t e = cudaMalloc(&cat->d_mem, cat->off_order + ks::order_scratch_bytes(C));
      if (e == cudaSuccess)
        e = ks::fast_prepare(ctx->desc, g, d_c, C, cat->d_mem, static_cast<char*>(cat->d_mem) + cat->off_memo,
                             static_cast<cudaStream_t>(stream), &ctx->launches);
      // the catalogue is ranked in similarity order (neighbouring candidates take similar paths)
      if (e == cudaSuccess)
        e = ks::launch_catalogue_order(d_c, C, static_cast<char*>(cat->d_mem) + cat->off_order,
                                       static_cast<cudaStream_t>(stream), &ctx->launches);
      if (e == cudaSuccess) e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
      if (e != cudaSuccess) {
        cudaFree(cat->d_mem);
        delete cat;
        return cuda_fail(ctx, e, "ks_catalogue_prepare");
      }
      cat->nblk = nblk;
      cat->slices = S;
      cat->prepared = true;
    }
  }
  *out_catalogue = cat;
  return KS_OK;
}

ks_status ks_catalogue_destroy(ks_catalogue* cat) {
  if (!cat) return KS_OK;
  DeviceGuard g(cat->device);
  cudaFree(cat->d_mem);
  delete cat;
  return KS_OK;
}

ks_status ks_select_one_prepared(ks_ctx* ctx, const ks_catalogue* cat, ks_problem p, int k, int32_t* h_topk_idx,
                                 float* h_topk_score, void* stream) {
  if (!ctx || !cat || cat->ctx != ctx || k < 1 || k > KS_MAX_K || !h_topk_idx || !h_topk_score)
    return KS_ERR_INVALID_ARG;
  if (!cat->prepared) return ks_select_one(ctx, p, cat->d_c, cat->C, cat->model, k, h_topk_idx, h_topk_score, stream);
  if (p.m < 1 || p.n < 1 || p.k < 1 || p.m > KS_MAX_DIM || p.n > KS_MAX_DIM || p.k > KS_MAX_DIM ||
      p.layout > 3 || p.dtype_ab > 3 || p.dtype_d > 3 || p.epi_flags > 5)
    return KS_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t* pin_idx = static_cast<int32_t*>(ctx->pinned);
  float* pin_sc = reinterpret_cast<float*>(pin_idx + KS_MAX_K);
  char* base = static_cast<char*>(cat->d_mem);
  const ks::GbdtModel& gm = cat->model->gbdt;
  ks::FastSlice sl{};
  sl.n_slices = cat->slices;
  sl.pairs = cat->C;
  sl.scores = reinterpret_cast<float*>(base + cat->off_scores);
  sl.counters = ctx->d_counters;
  sl.out_idx = ctx->d_pinned_idx;
  sl.out_score = ctx->d_pinned_score;
  sl.tiles = nullptr;
  int* h_seq = reinterpret_cast<int*>(pin_sc + KS_MAX_K);
  sl.out_seq = reinterpret_cast<int*>(ctx->d_pinned_score + KS_MAX_K);
  sl.seq = ++ctx->select_one_seq;
  ks::FastPrepared prep{reinterpret_cast<const uint8_t*>(base), base + cat->off_memo};
  cudaError_t e = ks::launch_select_fast(ctx->desc, gm, nullptr, &p, 1, cat->d_c, cat->C, cat->nblk, gm.block_cands,
                                         nullptr, nullptr, k, reinterpret_cast<unsigned long long*>(base + cat->off_part),
                                         nullptr, ctx->d_status, st, &ctx->launches, nullptr, &sl, nullptr, &ctx->wait,
                                         &prep, reinterpret_cast<const int32_t*>(base + cat->off_order));
  if (e == cudaSuccess) {
    bool seen = false;
    for (int spin = 0; spin < (1 << 22) && !seen; ++spin) seen = *static_cast<volatile int*>(h_seq) == sl.seq;
    if (!seen) e = cudaStreamSynchronize(st);  // a failed launch never writes the word: wait the regular way
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e, "ks_select_one_prepared");
  ks_status s = read_status(ctx);
  if (s != KS_OK) return s;
  std::memcpy(h_topk_idx, pin_idx, k * sizeof(int32_t));
  std::memcpy(h_topk_score, pin_sc, k * sizeof(float));
  return KS_OK;
}

ks_status ks_select_host(ks_ctx* ctx, const ks_problem* h_p, int P, const ks_candidate* h_c, int C,
                         const int64_t* h_seg_offsets, const int32_t* h_seg_index, int64_t pairs,
                         const ks_model* model, int k, int32_t* h_topk_idx, float* h_topk_score,
                         void* stream) {
  if (!ctx || !model || model->ctx != ctx || k < 1 || k > KS_MAX_K) return KS_ERR_INVALID_ARG;
  ks_status s = check_pairs(P, C, h_seg_offsets, h_seg_index, pairs);
  if (s != KS_OK) return s;
  if (P == 0) return KS_OK;
  if (!h_p || !h_topk_idx || !h_topk_score || (pairs > 0 && !h_c)) return KS_ERR_INVALID_ARG;
  const bool seg = h_seg_offsets != nullptr;
  if (seg && (h_seg_offsets[0] != 0 || h_seg_offsets[P] != pairs)) return KS_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t b_part = align_up(ks::select_partial_bytes(*model, P, C, pairs, seg, k));
  const size_t b_p = align_up(sizeof(ks_problem) * P), b_c = align_up(sizeof(ks_candidate) * C);
  const size_t b_so = seg ? align_up(sizeof(int64_t) * (P + 1)) : 0;
  const size_t b_si = seg ? align_up(sizeof(int32_t) * pairs) : 0;
  const size_t b_oi = align_up(sizeof(int32_t) * P * k), b_os = align_up(sizeof(float) * P * k);
  s = ensure_workspace(ctx, b_part + b_p + b_c + b_so + b_si + b_oi + b_os);
  if (s != KS_OK) return s;
  char* q = static_cast<char*>(ctx->ws) + b_part;
  ks_problem* d_p = reinterpret_cast<ks_problem*>(q); q += b_p;
  ks_candidate* d_c = reinterpret_cast<ks_candidate*>(q); q += b_c;
  int64_t* d_so = seg ? reinterpret_cast<int64_t*>(q) : nullptr; q += b_so;
  int32_t* d_si = seg ? reinterpret_cast<int32_t*>(q) : nullptr; q += b_si;
  int32_t* d_oi = reinterpret_cast<int32_t*>(q); q += b_oi;
  float* d_os = reinterpret_cast<float*>(q);
  cudaError_t e = cudaMemcpyAsync(d_p, h_p, sizeof(ks_problem) * P, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess && C > 0) e = cudaMemcpyAsync(d_c, h_c, sizeof(ks_candidate) * C, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess && seg) e = cudaMemcpyAsync(d_so, h_seg_offsets, sizeof(int64_t) * (P + 1), cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess && seg && pairs > 0) e = cudaMemcpyAsync(d_si, h_seg_index, sizeof(int32_t) * pairs, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess)
    e = ks::launch_select(ctx->desc, *model, d_p, nullptr, P, d_c, C, d_so, d_si, pairs, k, ctx->ws, d_oi,
                          d_os, st, &ctx->launches, ctx->d_status, nullptr, nullptr, ctx->d_counters, &ctx->wait);
  if (e == cudaSuccess) e = cudaMemcpyAsync(h_topk_idx, d_oi, sizeof(int32_t) * P * k, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaMemcpyAsync(h_topk_score, d_os, sizeof(float) * P * k, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  return e == cudaSuccess ? read_status(ctx) : cuda_fail(ctx, e, "ks_select_host");
}

}  // extern "C"
