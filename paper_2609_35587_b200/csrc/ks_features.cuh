// Device-side feature map x = phi(p, c, h) (Table "Feature groups").
//
// Integer quantities are exact in 64-bit arithmetic; every float column is a fixed short
// sequence of individually rounded binary32 operations issued through the round-to-nearest
// intrinsics (__ll2float_rn, __fdiv_rn, __fmul_rn, __fsub_rn), which the compiler neither
// contracts into FMAs nor replaces by approximations, so the bits do not depend on
// optimisation flags. The split into problem-only, candidate-only and per-pair terms lets a
// kernel hoist the first two out of its pair loop.
#pragma once

#include <cstdint>

#include "ks.h"

namespace ks {

constexpr int kRow = KS_F_PAD;

// What a feature column depends on (Table "Feature groups"): 0 problem only, 1 candidate only
// (given the element types), 2 both.
__host__ __device__ constexpr int feat_class(int col) {
  return (col <= 9 || col == 37 || col == 40 || col == 45) ? 0
         : ((col >= 10 && col <= 22) || col == 38 || (col >= 46 && col <= 59) || col == 62) ? 1
                                                                                            : 2;
}

// Descriptor fetch: a problem or candidate record is 16 bytes and sits on a 16-byte boundary
// (checked where the arrays enter the library), so it is one 128-bit load.
__device__ __forceinline__ ks_problem load_problem(const ks_problem* p) {
  const uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
  ks_problem r;
  r.m = v.x;
  r.n = v.y;
  r.k = v.z;
  r.layout = static_cast<uint8_t>(v.w);
  r.dtype_ab = static_cast<uint8_t>(v.w >> 8);
  r.dtype_d = static_cast<uint8_t>(v.w >> 16);
  r.epi_flags = static_cast<uint8_t>(v.w >> 24);
  return r;
}
__device__ __forceinline__ ks_candidate load_candidate(const ks_candidate* p) {
  const uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
  ks_candidate r;
  r.tile_m = static_cast<uint16_t>(v.x);
  r.tile_n = static_cast<uint16_t>(v.x >> 16);
  r.tile_k = static_cast<uint16_t>(v.y);
  r.instr_n = static_cast<uint16_t>(v.y >> 16);
  r.stages = static_cast<uint8_t>(v.z);
  r.cluster_m = static_cast<uint8_t>(v.z >> 8);
  r.cluster_n = static_cast<uint8_t>(v.z >> 16);
  r.kernel_sched = static_cast<uint8_t>(v.z >> 24);
  r.epi_sched = static_cast<uint8_t>(v.w);
  r.tile_sched = static_cast<uint8_t>(v.w >> 8);
  r.instr_m = static_cast<uint8_t>(v.w >> 16);
  r.instr_k = static_cast<uint8_t>(v.w >> 24);
  return r;
}

__device__ __forceinline__ float F64i(long long v) { return __ll2float_rn(v); }
__device__ __forceinline__ float F32i(int v) { return __int2float_rn(v); }
__device__ __forceinline__ unsigned cdiv_u32(unsigned a, unsigned b) { return (a + b - 1u) / b; }
__device__ __forceinline__ long long cdiv_i64(long long a, long long b) { return (a + b - 1) / b; }

__device__ __forceinline__ int bytes_ab(int dt) { return dt == 2 ? 1 : (dt == 3 ? 4 : 2); }
__device__ __forceinline__ int bytes_d(int dt) { return dt == 2 ? 1 : (dt == 3 ? 4 : 2); }

// Problem-only terms (section "Structural Core", "Memory Behavior"): computed once per problem.
struct ProblemTerms {
  unsigned M, N, K;
  int bA, bD, dtype_ab, dtype_d, layout, has_bias, act;
  long long bytesA, bytesB, Q_epi;  // b_A M K, b_B K N, Q_epilogue
  float log2m, log2n, log2k;
  float i_problem, ws_frac_l2, f_bytes_in, f_traffic_epi;
  unsigned long long tc_rate;  // tensor rate of this problem's input type
};

__device__ __forceinline__ float log2_dim(unsigned v) {
  return __double2float_rn(log2(static_cast<double>(v)));
}

__device__ inline void problem_terms(const ks_problem& p, const ks_gpu_desc& h, ProblemTerms& t) {
  t.M = p.m; t.N = p.n; t.K = p.k;
  t.dtype_ab = p.dtype_ab & 3;
  t.dtype_d = p.dtype_d & 3;
  t.layout = p.layout;
  t.bA = bytes_ab(t.dtype_ab);
  t.bD = bytes_d(t.dtype_d);
  t.has_bias = p.epi_flags & 1;
  t.act = (p.epi_flags >> 1) & 3;
  const long long M = t.M, N = t.N, K = t.K;
  t.bytesA = t.bA * M * K;
  t.bytesB = t.bA * K * N;
  t.Q_epi = t.bD * M * N + (t.has_bias ? t.bD * M : 0);
  t.log2m = log2_dim(t.M);
  t.log2n = log2_dim(t.N);
  t.log2k = log2_dim(t.K);
  t.i_problem = __fdiv_rn(F64i(2 * M * N * K), F64i(t.bytesA + t.bytesB + t.Q_epi));
  t.ws_frac_l2 = __fdiv_rn(F64i(t.bytesA + t.bytesB), F64i(static_cast<long long>(h.l2_bytes)));
  t.f_traffic_epi = F64i(t.Q_epi);
  t.tc_rate = h.tc_flops_per_us_per_sm[t.dtype_ab];
}

// a / b rounded up for non-negative operands; takes the 32-bit path when both fit (same value)
__device__ __forceinline__ long long cdiv_fit(long long a, long long b) {
  if (((a | b) >> 32) == 0)
    return static_cast<long long>(cdiv_u32(static_cast<unsigned>(a), static_cast<unsigned>(b)));
  return cdiv_i64(a, b);
}
__device__ __forceinline__ long long div_fit(long long a, long long b) {
  if (((a | b) >> 32) == 0) return static_cast<long long>(static_cast<unsigned>(a) / static_cast<unsigned>(b));
  return a / b;
}

// kExact: IEEE round-to-nearest division (bit-identical to the CPU definition). !kExact: the
// fast approximate division, for consumers that round the result to bf16 anyway.
template <bool kExact>
__device__ __forceinline__ float fdiv(float a, float b) {
  return kExact ? __fdiv_rn(a, b) : __fdividef(a, b);
}

// Candidate-side resource terms (section "Resource Pressure and Occupancy"); they depend on the
// problem only through its element sizes.
// Shared-memory footprint of one CTA: mainloop stages, epilogue staging, and their total.
// The warp-specialised (and the basic) mainloop may reuse the mainloop buffers for the
// epilogue; ping-pong and cooperative hold both at once.
struct SmemTerms {
  long long B_stage, smem_main, B_epi, both, B_smem;
};

__device__ __forceinline__ SmemTerms smem_terms(int bA, int bD, const ks_candidate& c, const ks_gpu_desc& h) {
  SmemTerms s;
  const int TM = c.tile_m, TN = c.tile_n, TK = c.tile_k, S = c.stages;
  const int ks = c.kernel_sched & 3;
  s.B_stage = static_cast<long long>(TK) * (TM * bA + TN * bA);
  s.smem_main = S * s.B_stage;
  const int E = (ks == 2) ? 128 : 64;
  s.B_epi = (c.epi_sched == 0) ? 0 : 2ll * min(TM, E) * min(TN, 32) * bD;
  s.both = s.smem_main + s.B_epi + h.smem_reserved;
  s.B_smem = (ks == 0 || ks == 3) ? max(s.smem_main, s.B_epi) + h.smem_reserved : s.both;
  return s;
}

struct Resources {
  long long B_stage, smem_main, B_epi, B_smem, area, b_smem, b_reg, b_res, b_eff;
  int T_block, n_cons, fits;
  float f_smem;
};

__device__ __forceinline__ Resources resources(const ProblemTerms& t, const ks_candidate& c,
                                               const ks_gpu_desc& h) {
  Resources r;
  const int TM = c.tile_m, TN = c.tile_n;
  const int ks = c.kernel_sched & 3;
  // (consumer warpgroups in the mainloop, threads per block): WS, Pingpong, Cooperative, basic
  r.n_cons = (ks == 2) ? 2 : 1;
  r.T_block = (ks == 0) ? 256 : (ks == 3 ? 128 : 384);
  const SmemTerms sm = smem_terms(t.bA, t.bD, c, h);
  r.B_stage = sm.B_stage;
  r.smem_main = sm.smem_main;
  r.B_epi = sm.B_epi;
  const long long both = sm.both;
  r.B_smem = sm.B_smem;
  r.f_smem = __fdiv_rn(F64i(r.B_smem), F64i(h.smem_per_sm));
  r.fits = both <= static_cast<long long>(h.smem_per_cta_max);
  r.area = static_cast<long long>(TM) * TN;
  r.b_smem = div_fit(static_cast<long long>(h.smem_per_sm), r.B_smem);
  const long long regs = min(255ll, 32 + cdiv_fit(r.area, r.T_block));
  r.b_reg = div_fit(static_cast<long long>(h.regs_per_sm), regs * r.T_block);
  const long long b_arch =
      min(static_cast<long long>(h.max_ctas_per_sm), static_cast<long long>(h.max_threads_per_sm / r.T_block));
  r.b_res = min(r.b_smem, min(r.b_reg, b_arch));
  r.b_eff = max(1ll, r.b_res);
  return r;
}

// The columns that depend on both the problem and the candidate (sections "Work Decomposition
// and Wave Quantization", "Memory Behavior", "Pipeline Balance"), given the candidate's
// effective resident-block count b_eff.
template <bool kExact, typename Put>
__device__ __forceinline__ void pair_columns(const ProblemTerms& t, const ks_candidate& c, const ks_gpu_desc& h,
                                             long long b_eff, Put put) {
  const int TM = c.tile_m, TN = c.tile_n, TK = c.tile_k, S = c.stages;
  const int cM = c.cluster_m, cN = c.cluster_n;
  const int bA = t.bA;
  const long long n_m = cdiv_u32(t.M, TM), n_n = cdiv_u32(t.N, TN), n_k = cdiv_u32(t.K, TK);
  const long long n_tiles = n_m * n_n;
  put(23, F64i(n_m));
  put(24, F64i(n_n));
  put(25, F64i(n_k));
  put(26, F64i(n_tiles));
  put(27, fdiv<kExact>(F64i(n_m * TM - t.M), F64i(t.M)));
  put(28, fdiv<kExact>(F64i(n_n * TN - t.N), F64i(t.N)));
  put(29, fdiv<kExact>(F64i(n_tiles), F64i(h.num_sms)));
  const long long resident = static_cast<long long>(h.num_sms) * b_eff;
  const long long waves = cdiv_fit(n_tiles, resident);
  put(30, F64i(waves));
  const float eta = fdiv<kExact>(F64i(n_tiles), F64i(waves * resident));
  put(31, eta);
  put(32, fmaxf(0.0f, __fsub_rn(1.0f, eta)));
  const long long n_c = cdiv_fit(t.M, static_cast<long long>(cM) * TM) * cdiv_fit(t.N, static_cast<long long>(cN) * TN);
  put(33, fdiv<kExact>(F64i(n_c * cM * cN - n_tiles), F64i(n_tiles)));
  put(34, fdiv<kExact>(F64i(n_m), F64i(cM)));
  put(35, fdiv<kExact>(F64i(n_n), F64i(cN)));
  put(36, F32i(cM > n_m || cN > n_n));
  const long long restream = n_n * t.bytesA + n_m * t.bytesB;
  put(39, fdiv<kExact>(F64i(restream), F64i(t.bytesA + t.bytesB)));
  const float fl2 = F64i(static_cast<long long>(h.l2_bytes));
  put(41, fdiv<kExact>(F64i(static_cast<long long>(bA) * TM * t.K), fl2));
  put(42, fdiv<kExact>(F64i(static_cast<long long>(bA) * TN * t.K), fl2));
  put(43, F64i(restream));
  put(44, F64i(cdiv_fit(n_n, cN) * t.bytesA + cdiv_fit(n_m, cM) * t.bytesB));
  put(60, fdiv<kExact>(F64i(min(static_cast<long long>(S), n_k)), F32i(S)));
  put(61, fdiv<kExact>(F64i(n_k), F32i(S)));
}

// ---- per-pair columns for consumers that round them to bf16 ------------------------------------
// Same quantities as pair_columns, evaluated in 32-bit integer and single-precision arithmetic:
// the integer counts (tiles, waves, clusters) stay exact, the ratios and byte counts carry
// float rounding (relative error ~1e-7, far below the bf16 rounding that follows). Valid when
// the tile counts are small enough for that (ok == true); otherwise the caller falls back to
// pair_columns.
struct PairFastTerms {
  float inv_M, inv_N, inv_sms, f_bytesA, f_bytesB, inv_bytes, k_bytes_over_l2;
};

__device__ inline void pair_fast_terms(const ProblemTerms& t, const ks_gpu_desc& h, PairFastTerms& f) {
  f.inv_M = __fdividef(1.0f, F64i(t.M));
  f.inv_N = __fdividef(1.0f, F64i(t.N));
  f.inv_sms = __fdividef(1.0f, F64i(h.num_sms));
  f.f_bytesA = F64i(t.bytesA);
  f.f_bytesB = F64i(t.bytesB);
  f.inv_bytes = __fdividef(1.0f, F64i(t.bytesA + t.bytesB));
  f.k_bytes_over_l2 = __fdividef(F64i(static_cast<long long>(t.bA) * t.K), F64i(static_cast<long long>(h.l2_bytes)));
}

// floor(a / b) for a < 2^24, 0 < b, given rb ~ 1 / b: the float quotient is within one of the
// answer and one multiply-back settles it
__device__ __forceinline__ unsigned udiv_small(unsigned a, unsigned b, float rb) {
  unsigned q = __float2uint_rz(__fmul_rz(__uint2float_rz(a), rb));
  const int r = static_cast<int>(a - q * b);
  q += (r >= static_cast<int>(b)) ? 1u : 0u;
  q -= (r < 0) ? 1u : 0u;
  return q;
}
__device__ __forceinline__ unsigned cdiv_small(unsigned a, unsigned b, float rb) {
  return udiv_small(a + b - 1u, b, rb);
}

template <typename Put>
__device__ __forceinline__ bool pair_columns_bf16(const ProblemTerms& t, const PairFastTerms& f,
                                                  const ks_candidate& c, const ks_gpu_desc& h, unsigned b_eff,
                                                  Put put) {
  const unsigned TM = c.tile_m, TN = c.tile_n, TK = c.tile_k, S = c.stages;
  const unsigned cM = c.cluster_m, cN = c.cluster_n;
  const float fTM = __uint2float_rn(TM), fTN = __uint2float_rn(TN);
  const float rTM = __fdividef(1.0f, fTM), rTN = __fdividef(1.0f, fTN);
  const float rTK = __fdividef(1.0f, __uint2float_rn(TK)), rS = __fdividef(1.0f, __uint2float_rn(S));
  const float rcM = __fdividef(1.0f, __uint2float_rn(cM)), rcN = __fdividef(1.0f, __uint2float_rn(cN));
  const unsigned n_m = cdiv_small(t.M, TM, rTM), n_n = cdiv_small(t.N, TN, rTN), n_k = cdiv_small(t.K, TK, rTK);
  if (n_m > 2048u || n_n > 2048u) return false;  // keeps every integer below 2^23
  const unsigned n_tiles = n_m * n_n;
  const float fn_m = __uint2float_rn(n_m), fn_n = __uint2float_rn(n_n), fn_k = __uint2float_rn(n_k);
  const float fn_tiles = __uint2float_rn(n_tiles);
  put(23, fn_m);
  put(24, fn_n);
  put(25, fn_k);
  put(26, fn_tiles);
  put(27, __uint2float_rn(n_m * TM - t.M) * f.inv_M);
  put(28, __uint2float_rn(n_n * TN - t.N) * f.inv_N);
  put(29, fn_tiles * f.inv_sms);
  const unsigned resident = h.num_sms * b_eff;
  const unsigned waves = cdiv_small(n_tiles, resident, __fdividef(1.0f, __uint2float_rn(resident)));
  put(30, __uint2float_rn(waves));
  const float eta = __fdividef(fn_tiles, __uint2float_rn(waves * resident));
  put(31, eta);
  put(32, fmaxf(0.0f, 1.0f - eta));
  const unsigned cmtm = cM * TM, cntn = cN * TN;
  const unsigned n_cm = cmtm >= t.M ? 1u : cdiv_small(t.M, cmtm, rcM * rTM);
  const unsigned n_cn = cntn >= t.N ? 1u : cdiv_small(t.N, cntn, rcN * rTN);
  const float r_tiles = __fdividef(1.0f, fn_tiles);
  put(33, __uint2float_rn(n_cm * cM * n_cn * cN - n_tiles) * r_tiles);
  put(34, fn_m * rcM);
  put(35, fn_n * rcN);
  put(36, (cM > n_m || cN > n_n) ? 1.0f : 0.0f);
  const float restream = fmaf(fn_n, f.f_bytesA, fn_m * f.f_bytesB);
  put(39, restream * f.inv_bytes);
  put(41, fTM * f.k_bytes_over_l2);
  put(42, fTN * f.k_bytes_over_l2);
  put(43, restream);
  put(44, fmaf(__uint2float_rn(cdiv_small(n_n, cN, rcN)), f.f_bytesA,
               __uint2float_rn(cdiv_small(n_m, cM, rcM)) * f.f_bytesB));
  put(60, __uint2float_rn(min(S, n_k)) * rS);
  put(61, fn_k * rS);
  return true;
}

// Static sampling score (the paper's sampling policy): n_c clusters, W = ceil(n_c / S_SM)
// cluster waves, s = n_c / (W S_SM c_M c_N) * S * sqrt(T_M T_N T_K), each step rounded to fp32.
__device__ __forceinline__ float static_score(const ProblemTerms& t, const ks_candidate& c, const ks_gpu_desc& h) {
  const long long TM = c.tile_m, TN = c.tile_n, TK = c.tile_k, cM = c.cluster_m, cN = c.cluster_n;
  const long long n_c = cdiv_fit(t.M, cM * TM) * cdiv_fit(t.N, cN * TN);
  const long long W = cdiv_fit(n_c, h.num_sms);
  float s = __fdiv_rn(F64i(n_c), F64i(W * h.num_sms * cM * cN));
  s = __fmul_rn(s, F32i(c.stages));
  return __fmul_rn(s, __fsqrt_rn(F64i(TM * TN * TK)));
}

// The columns that depend on the problem alone (class 0 of feat_class), straight from its terms.
template <typename Put>
__device__ __forceinline__ void problem_columns(const ProblemTerms& t, Put put) {
  put(0, t.log2m);
  put(1, t.log2n);
  put(2, t.log2k);
  put(3, F32i(t.layout == 2 || t.layout == 3));
  put(4, F32i(t.layout == 1 || t.layout == 3));
  put(5, F32i(t.dtype_ab));
  put(6, F32i(t.bA));
  put(7, F32i(t.bD));
  put(8, F32i(t.has_bias));
  put(9, F32i(t.act));
  put(37, t.i_problem);
  put(40, t.ws_frac_l2);
  put(45, t.f_traffic_epi);
}

// Writes the 64 columns of one pair through `put(column, value)`.
template <typename Put>
__device__ __forceinline__ void featurize_pair(const ProblemTerms& t, const ks_candidate& c,
                                               const ks_gpu_desc& h, Put put) {
  const int TM = c.tile_m, TN = c.tile_n, TK = c.tile_k, S = c.stages;
  const int cM = c.cluster_m, cN = c.cluster_n;
  const int bA = t.bA;

  // ---- structural core ------------------------------------------------------------------
  problem_columns(t, put);
  put(10, F32i(TM));
  put(11, F32i(TN));
  put(12, F32i(TK));
  put(13, F32i(c.instr_m));
  put(14, F32i(c.instr_n));
  put(15, F32i(c.instr_k));
  put(16, F32i(S));
  put(17, F32i(c.kernel_sched));
  put(18, F32i(c.epi_sched));
  put(19, F32i(c.tile_sched));
  put(20, F32i(cM));
  put(21, F32i(cN));
  put(22, F32i(cM * cN));

  const Resources r = resources(t, c, h);
  pair_columns<true>(t, c, h, r.b_eff, put);

  // ---- memory behaviour (candidate-only column) -----------------------------------------------
  put(38, __fdiv_rn(F64i(2 * r.area), F64i(static_cast<long long>(TM) * bA + static_cast<long long>(TN) * bA)));

  // ---- resource pressure columns ------------------------------------------------------------
  put(46, F64i(r.B_stage));
  put(47, F64i(r.smem_main));
  put(48, F64i(r.B_epi));
  put(49, F64i(r.B_smem));
  put(50, r.f_smem);
  put(51, F32i(r.fits));
  put(52, __fdiv_rn(F64i(r.area), F32i(r.T_block)));
  put(53, F64i(r.b_smem));
  put(54, F64i(r.b_reg));
  put(55, F64i(r.b_res));
  put(56, __fdiv_rn(F64i(r.b_eff * r.T_block), F64i(h.max_threads_per_sm)));

  // ---- pipeline balance (candidate-only columns) ----------------------------------------------
  const float t_prod = __fdiv_rn(F64i(static_cast<long long>(h.num_sms) * r.B_stage),
                                 F64i(static_cast<long long>(h.tma_bytes_per_us)));
  const float t_cons = __fdiv_rn(F64i(2 * r.area * TK), F64i(r.n_cons * static_cast<long long>(t.tc_rate)));
  put(57, t_prod);
  put(58, t_cons);
  put(59, __fdiv_rn(t_cons, t_prod));
  put(62, __fmul_rn(F32i(S), r.f_smem));
  put(63, 0.0f);
}

}  // namespace ks
