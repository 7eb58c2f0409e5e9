// Tensor-core path of the fused select kernel for the feed-forward ranker (Model B) of shape
// 64 -> 256 -> 256 -> 1: bf16 operands, fp32 accumulation in tensor memory.
//
// One CTA (512 threads: four first-epilogue warps, four second-epilogue warps, eight feature-row
// warps in two groups that take alternate tiles) ranks one problem against its share of the
// candidates, 128 at a time, as one continuous pipeline of tiles:
//   F    the 128 feature rows are written straight into shared memory as the bf16 A operand
//        (candidate-only columns come standardised from a per-call table, problem-only columns
//        are constant per CTA, the per-pair columns are computed in registers);
//   L1   4 x tcgen05.mma (M 128, N 256, K 16) against W1, accumulator in TMEM;
//   E1   TMEM -> registers, + bias, ReLU, round to bf16, written back to shared memory as the A
//        operand of the next layer (it overwrites the feature tile);
//   L2   16 x tcgen05.mma against W2 into the same TMEM columns;
//   E2   TMEM -> registers, + bias, ReLU, round to bf16, dot with w3 on the CUDA cores, + b3:
//        the score; one ranking key per row, merged into the warp's running top-k list (one
//        entry per lane), so ranking costs a warp-wide max per tile and nothing per pass.
// The four lists are merged once, when the CTA has walked all its tiles.
// Both weight matrices stay resident in shared memory for the CTA's lifetime; they arrive by
// bulk async copies (cp.async.bulk, no multicast) of an image the host prepared in the
// operand layout. All waits are bounded and report through the status word.
//
// Operand layout (no swizzle, K-major): element (row, k) of a [rows x K] operand lives at
// (k / 8) * rows * 16 + row * 16 + (k % 8) * 2 bytes: planes of eight K-columns, 16 bytes per
// row. In descriptor terms the two 8-column halves of one K = 16 step are `rows * 16` bytes
// apart (leading offset) and groups of eight rows 128 bytes apart (stride offset).
#include <cuda_bf16.h>

#include <cmath>
#include <cstring>
#include <new>
#include <vector>

#include "ks_features.cuh"
#include "ks_internal.h"
#include "ks_topk.cuh"

namespace ks {

namespace {

constexpr int kT = kMlpThreads;
constexpr int kTileRows = 128;
constexpr int kH = 256;                               // hidden width
constexpr int kW1Bytes = kH * 64 * 2;                 // 32 KB
constexpr int kW2Bytes = kH * kH * 2;                 // 128 KB
constexpr int kABytes = kTileRows * kH * 2;           // 64 KB: H1 tile (the feature tile aliases its start)
constexpr int kOffW1 = 0;
constexpr int kOffW2 = kW1Bytes;
constexpr int kOffA = kW1Bytes + kW2Bytes;
constexpr int kSmemBytes = kOffA + kABytes;           // 224 KB
constexpr int kPlaneA = kTileRows * 16;               // bytes per 8-column plane of an A operand
constexpr int kPlaneB = kH * 16;                      // ... of a B operand
constexpr int kCandRec = 64;                          // bytes per (combination, candidate) record
constexpr int kCombos = 16;
constexpr int kNC = 29, kNPair = 21;                  // candidate-only and per-pair columns (13 are problem-only)

// position of feature column `col` along K: candidate-only columns first, then per-pair, then
// problem-only, each class in ascending column order; position 63 is the zero pad
__host__ __device__ constexpr int kpos(int col) {
  int pos = 0;
  const int cls = feat_class(col);
  const int base = cls == 1 ? 0 : (cls == 2 ? kNC : kNC + kNPair);
  for (int c = 0; c < col; ++c)
    if (feat_class(c) == cls) ++pos;
  return base + pos;
}

// One-hot input form: the candidate-only columns other than kernel / epilogue schedule at 0..26,
// the per-pair columns where they always are (29..49), the seven schedule-level indicators at
// 50..56; everything else is zero. The problem-only inputs do not enter the MMA (-1): they are
// folded into a per-CTA bias.
__host__ __device__ constexpr int kpos_oh(int col) {
  const int cls = feat_class(col);
  if (cls == 0 || col == 17 || col == 18) return -1;
  if (cls == 2) return kpos(col);
  int pos = 0;
  for (int c = 0; c < col; ++c)
    if (feat_class(c) == 1 && c != 17 && c != 18) ++pos;
  return pos;
}
constexpr int kIndPos = 50;  // K position of the first level indicator
// the folded inputs in order: problem-only columns other than operand type (5) and activation (9),
// then the four operand-type indicators, then the three activation indicators
__host__ __device__ constexpr int kfold(int col) {
  if (feat_class(col) != 0 || col == 5 || col == 9) return -1;
  int pos = 0;
  for (int c = 0; c < col; ++c)
    if (feat_class(c) == 0 && c != 5 && c != 9) ++pos;
  return pos;
}
constexpr int kFoldCols = 11, kFold = 18;

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
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// shared-memory matrix descriptor: no swizzle, K-major, version 1
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lead_bytes, uint32_t stride_bytes) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr >> 4) & 0x3FFFu);
  d |= static_cast<uint64_t>((lead_bytes >> 4) & 0x3FFFu) << 16;
  d |= static_cast<uint64_t>((stride_bytes >> 4) & 0x3FFFu) << 32;
  d |= 1ull << 46;
  return d;
}

// instruction descriptor: D fp32, A and B bf16, both K-major, N = 256, M = 128
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(tmem_d),
      "l"(a_desc), "l"(b_desc), "r"(kIdesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&t);
}
// (max(lo, 0), max(hi, 0)) rounded to bf16 and packed, one instruction
__device__ __forceinline__ uint32_t pack_bf16_relu(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}

// ------------------------------------------------------------------------------------------
// candidate-only columns, standardised and rounded to bf16, once per call
// ------------------------------------------------------------------------------------------

// Raised by a CTA whose bounded wait ran out, so that the CTAs after it leave at once; cleared by
// the per-call table kernel that precedes every launch. (The status word itself lives in mapped
// host memory: reading it from every CTA would cost a PCIe round trip each.)
__device__ int g_mlp_abort;

// the scoring call has no per-call table kernel in front: this clears the abort flag instead
__global__ void mlp_reset_abort_kernel() { g_mlp_abort = 0; }

__global__ void mlp_combo_mask_kernel(const ks_problem* __restrict__ p, int P, unsigned* __restrict__ mask) {
  unsigned m = 0;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < P; i += gridDim.x * blockDim.x)
    m |= 1u << ((p[i].dtype_ab & 3) * 4 + (p[i].dtype_d & 3));
  m = __reduce_or_sync(0xFFFFFFFFu, m);
  if ((threadIdx.x & 31) == 0 && m) atomicOr(mask, m);
}

__global__ void __launch_bounds__(256)
mlp_cand_cols_kernel(ks_gpu_desc desc, const ks_candidate* __restrict__ c, int C, const unsigned* mask_ptr,
                     unsigned mask_value, const __grid_constant__ MlpTcParams prm, uint8_t* __restrict__ out) {
  const int combo = blockIdx.y;
  if (blockIdx.x == 0 && combo == 0 && threadIdx.x == 0) g_mlp_abort = 0;
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
  float x[32];
#pragma unroll
  for (int q = 0; q < 32; ++q) x[q] = 0.0f;
  const ks_candidate cand = c[i];
  if (prm.onehot) {
    featurize_pair(t, cand, desc, [&](int col, float v) {
      if (feat_class(col) != 1 || col == 17 || col == 18) return;
      const int k = kpos_oh(col);
      x[k] = fmaf(v, prm.scale[k], prm.shift[k]);
    });
  } else {
    featurize_pair(t, cand, desc, [&](int col, float v) {
      if (feat_class(col) != 1) return;
      const int k = kpos(col);
      x[k] = fmaf(v, prm.scale[k], prm.shift[k]);
    });
  }
  uint32_t w[16];
#pragma unroll
  for (int q = 0; q < 16; ++q) w[q] = pack_bf16(x[2 * q], x[2 * q + 1]);
  // the last word (positions 30, 31 belong to per-pair columns) carries the candidate's
  // effective resident-block count for the per-pair wave columns
  w[15] = static_cast<uint32_t>(resources(t, cand, desc).b_eff) & 0xFFFFu;
  uint4* dst = reinterpret_cast<uint4*>(out + (static_cast<size_t>(combo) * C + i) * kCandRec);
#pragma unroll
  for (int q = 0; q < 4; ++q) dst[q] = make_uint4(w[4 * q], w[4 * q + 1], w[4 * q + 2], w[4 * q + 3]);
}

// ------------------------------------------------------------------------------------------
// epilogues (H = which half of the 256 columns this warp owns)
// ------------------------------------------------------------------------------------------

// 32 consecutive fp32 columns of this thread's TMEM lane, without waiting for them
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
// Waits for this thread's outstanding TMEM loads. The registers of the load being waited for
// pass through as read-write operands, so that no use of them is scheduled above the wait.
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]),
                 "+r"(r[15]), "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]),
                 "+r"(r[22]), "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]),
                 "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}

// two fp32 lanes per 64-bit register: (lo, hi) + (lo, hi), and a * b + c, each lane rounded as
// the scalar instruction would
__device__ __forceinline__ unsigned long long pack2(uint32_t lo, uint32_t hi) {
  unsigned long long d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(lo), "r"(hi));
  return d;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& lo, float& hi) {
  uint32_t a, b;
  asm("mov.b64 {%0, %1}, %2;" : "=r"(a), "=r"(b) : "l"(v));
  lo = __uint_as_float(a);
  hi = __uint_as_float(b);
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ unsigned long long const2(const float* p) {  // two consecutive floats, 8-byte aligned
  return *reinterpret_cast<const unsigned long long*>(p);
}

// E1: h1 = bf16(relu(acc + b1)) for the 256 columns of this thread's row, written as A-operand
// planes. The TMEM load of the next 32 columns is in flight while the current ones are processed.
// kSmemBias: the bias comes from shared memory (per-CTA vector of the one-hot form) instead of the
// constant bank.
template <int H, bool kSmemBias>
__device__ __forceinline__ void epilogue1(uint32_t tmem_row, uint32_t sA_row, const MlpTcParams& prm,
                                          const float* s_b1) {
  uint32_t ra[32], rb[32];
  tmem_ld32_issue(tmem_row + H * 128, ra);
#pragma unroll
  for (int blk = 0; blk < 8; ++blk) {
    uint32_t(&cur)[32] = (blk & 1) ? rb : ra;
    uint32_t(&nxt)[32] = (blk & 1) ? ra : rb;
    tmem_ld_wait(cur);
    if (blk < 7) tmem_ld32_issue(tmem_row + H * 128 + (blk + 1) * 32, nxt);
#pragma unroll
    for (int g = 0; g < 4; ++g) {  // eight columns = one plane
      uint32_t w[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int j = H * 128 + blk * 32 + g * 8 + 2 * q;
        float lo, hi;
        unpack2(add2(pack2(cur[g * 8 + 2 * q], cur[g * 8 + 2 * q + 1]), const2(kSmemBias ? &s_b1[j] : &prm.b1[j])),
                lo, hi);
        w[q] = pack_bf16_relu(lo, hi);
      }
      const int plane = (H * 128 + blk * 32 + g * 8) / 8;
      asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(sA_row + plane * kPlaneA), "r"(w[0]), "r"(w[1]),
                   "r"(w[2]), "r"(w[3])
                   : "memory");
    }
  }
}

// E2: dot of bf16(relu(acc + b2)) with w3 over the 256 columns of this thread's row; even and
// odd columns accumulate in the two lanes of one packed register
template <int H>
__device__ __forceinline__ float epilogue2(uint32_t tmem_row, const MlpTcParams& prm) {
  unsigned long long s0 = 0ull, s1 = 0ull;  // (0.0f, 0.0f)
  uint32_t ra[32], rb[32];
  tmem_ld32_issue(tmem_row + H * 128, ra);
#pragma unroll
  for (int blk = 0; blk < 8; ++blk) {
    uint32_t(&cur)[32] = (blk & 1) ? rb : ra;
    uint32_t(&nxt)[32] = (blk & 1) ? ra : rb;
    tmem_ld_wait(cur);
    if (blk < 7) tmem_ld32_issue(tmem_row + H * 128 + (blk + 1) * 32, nxt);
#pragma unroll
    for (int q = 0; q < 16; ++q) {
      const int j = H * 128 + blk * 32 + 2 * q;
      float lo, hi;
      unpack2(add2(pack2(cur[2 * q], cur[2 * q + 1]), const2(&prm.b2[j])), lo, hi);
      const uint32_t pk = pack_bf16_relu(lo, hi);
      const unsigned long long h2 = pack2(pk << 16, pk & 0xFFFF0000u);
      if (q & 1) s1 = fma2(h2, const2(&prm.w3[j]), s1);
      else s0 = fma2(h2, const2(&prm.w3[j]), s0);
    }
  }
  float a, b, c, d;
  unpack2(s0, a, b);
  unpack2(s1, c, d);
  return (a + b) + (c + d);
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// barrier among the four warps of the first-epilogue group
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// ------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------

// kForm 0: ordinal input form (K positions as kpos); 1: one-hot form (kpos_oh + folded bias);
// 2: scoring call - the rows of `feat_rows` (ordinal form) are the input, every score is written to
// `score_out`, nothing is ranked (one "problem" whose candidates are the rows).
template <int kForm>
__global__ void __launch_bounds__(kT, 1)
select_mlp_tc_kernel(ks_gpu_desc desc, const ks_problem* __restrict__ p, ks_problem p_value, int use_value,
                     const ks_candidate* __restrict__ c, int P, int C, int nblk,
                     const int64_t* __restrict__ seg_off, const int32_t* __restrict__ seg_idx,
                     const uint8_t* __restrict__ w_image, const uint8_t* __restrict__ cand_cols, int k,
                     unsigned long long* __restrict__ partial, int* __restrict__ status,
                     const float* __restrict__ feat_rows, float* __restrict__ score_out,
                     const __grid_constant__ MlpTcParams prm) {
  constexpr bool kOneHot = kForm == 1, kRows = kForm == 2;
  extern __shared__ __align__(1024) unsigned char smem[];
  __shared__ ProblemTerms s_pt;
  __shared__ PairFastTerms s_pf;
  // weights; L2 first group; L2 done; L1 done; feature rows stored; accumulator 0 / 1 read out
  __shared__ __align__(8) unsigned long long s_bar[10];
  __shared__ uint32_t s_tmem;
  __shared__ uint32_t s_pwords[7];   // problem-only columns (positions 50..63) as packed bf16
  // the second-epilogue warps' final lists; until they are written (after the last tile) the
  // same kilobyte holds the per-CTA first-layer bias of the one-hot form
  __shared__ __align__(16) unsigned long long s_merge[4][32];
  float* s_b1 = reinterpret_cast<float*>(&s_merge[0][0]);
  __shared__ float s_xp[kFold];  // one-hot form: the folded inputs, standardised and rounded to bf16
  __shared__ int s_fail, s_abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) s_abort = *reinterpret_cast<volatile int*>(&g_mlp_abort);
  __syncthreads();
  if (s_abort) {  // a wait ran out in an earlier CTA of this launch: the call fails, leave at once
    if (!kRows && tid < k) partial[static_cast<size_t>(blockIdx.x) * k + tid] = 0ull;
    return;
  }
  const bool is_epi = tid < 256;  // warps 0..7 read the accumulators; warps 8..15 produce feature rows
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
  const uint32_t bar_w = smem_u32(&s_bar[0]), bar_a0 = smem_u32(&s_bar[1]), bar_b0 = smem_u32(&s_bar[2]),
                 bar_c = smem_u32(&s_bar[3]), bar_x0 = smem_u32(&s_bar[4]), bar_f0 = smem_u32(&s_bar[5]),
                 bar_f1 = smem_u32(&s_bar[6]), bar_a1 = smem_u32(&s_bar[7]), bar_x1 = smem_u32(&s_bar[8]),
                 bar_b1 = smem_u32(&s_bar[9]);

  if (tid == 0 && !kRows) {
    problem_terms(use_value ? p_value : p[prob], desc, s_pt);
    pair_fast_terms(s_pt, desc, s_pf);
    ks_candidate dummy{};
    dummy.tile_m = dummy.tile_n = dummy.tile_k = 64;
    dummy.stages = dummy.cluster_m = dummy.cluster_n = 1;
    float pv[16];
#pragma unroll
    for (int q = 0; q < 16; ++q) pv[q] = 0.0f;
    featurize_pair(s_pt, dummy, desc, [&](int col, float v) {
      if (feat_class(col) != 0) return;
      const int kk = kpos(col);
      pv[kk - (kNC + kNPair)] = fmaf(v, prm.scale[kk], prm.shift[kk]);
    });
#pragma unroll
    for (int q = 0; q < 7; ++q) s_pwords[q] = pack_bf16(pv[2 * q], q == 6 ? 0.0f : pv[2 * q + 1]);
    if (kOneHot) {
      featurize_pair(s_pt, dummy, desc, [&](int col, float v) {
        const int q = kfold(col);
        if (q < 0) return;
        s_xp[q] = __bfloat162float(__float2bfloat16_rn(fmaf(v, prm.p_scale[q], prm.p_shift[q])));
      });
      for (int l = 0; l < 4; ++l)
        s_xp[kFoldCols + l] = __bfloat162float(__float2bfloat16_rn(
            fmaf(s_pt.dtype_ab == l ? 1.0f : 0.0f, prm.p_scale[kFoldCols + l], prm.p_shift[kFoldCols + l])));
      for (int l = 0; l < 3; ++l)
        s_xp[kFoldCols + 4 + l] = __bfloat162float(__float2bfloat16_rn(
            fmaf(s_pt.act == l ? 1.0f : 0.0f, prm.p_scale[kFoldCols + 4 + l], prm.p_shift[kFoldCols + 4 + l])));
    }
  }
  if (tid == 0) {
    mbar_init(bar_w, 1);
    mbar_init(bar_a0, 1);
    mbar_init(bar_a1, 1);
    mbar_init(bar_b0, 1);
    mbar_init(bar_b1, 1);
    mbar_init(bar_c, 1);
    mbar_init(bar_x0, kTileRows);
    mbar_init(bar_x1, kTileRows);
    mbar_init(bar_f0, kTileRows);
    mbar_init(bar_f1, kTileRows);
    s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // both weight matrices, resident for the CTA's lifetime
    fence_async_proxy();
    mbar_expect_tx(bar_w, kW1Bytes + kW2Bytes);
    if (!prm.starve)  // test hook: without the copies the wait on this barrier runs out
      for (int off = 0; off < kW1Bytes + kW2Bytes; off += 32768)
        bulk_copy_g2s(sbase + kOffW1 + off, w_image + off, 32768, bar_w);
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  const uint32_t sA = sbase + kOffA;
  if (kOneHot) {  // per-CTA bias: b1 + the folded problem-only inputs through their weights
    if (tid < kH) {
      float acc = prm.b1[tid];
      for (int q = 0; q < kFold; ++q) acc = fmaf(__ldg(prm.w1_prob + q * kH + tid), s_xp[q], acc);
      s_b1[tid] = acc;
    }
    __syncthreads();
  }
  const int combo = kRows ? 0 : s_pt.dtype_ab * 4 + s_pt.dtype_d;
  bool failed = false;
  // Bounded wait. After the first one that runs out, every later wait of the CTA gives up after a
  // few probes, and the CTAs that start later leave at once (device flag).
  auto wait_ok = [&](uint32_t bar, uint32_t parity) {
    for (int i = 0; i < prm.wait_limit; ++i) {
      if (mbar_try_wait(bar, parity)) return true;
      if ((i & 255) == 255 && *reinterpret_cast<volatile int*>(&s_fail)) break;
    }
    *reinterpret_cast<volatile int*>(&s_fail) = 1;
    atomicExch(&g_mlp_abort, 1);
    return false;
  };
  if (!wait_ok(bar_w, 0)) failed = true;
  // Each role tracks the phase of the barriers it waits on. A parity wait can only tell adjacent
  // phases apart, so every barrier here is consumed before it can complete again; that is why
  // the barriers of alternating tiles come in pairs.
  uint32_t ph_a = 0, ph_b[2] = {0, 0}, ph_c = 0, ph_x = 0, ph_f = 0;

  // This CTA's tiles: an equal share (to within one) of the problem's 128-row tiles, contiguous.
  // The tile pipeline runs through all of them without draining in between.
  const int64_t problem_tiles = (len + kTileRows - 1) / kTileRows;
  const int64_t tile_first = problem_tiles * chunk / nblk;
  // a CTA whose weights never arrived runs no tile at all: nothing is issued to the tensor cores
  const int total_tiles = failed ? 0 : static_cast<int>(problem_tiles * (chunk + 1) / nblk - tile_first);
  auto tile_row0 = [&](int tile) { return (tile_first + tile) * kTileRows; };
  unsigned long long top = 0ull;  // second-epilogue warps: lane j holds the warp's j-th best key

  // Roles (tile t uses accumulator t & 1):
  //   feature rows  two groups of four warps take alternate tiles: compute row(t) in registers at
  //                 any time; once L2(t-1)'s first group has released planes 0..7 store it there;
  //                 the group's first warp then issues L1(t) as soon as all rows are stored and
  //                 accumulator t & 1 has been read out (E2(t-2));
  //   warps 0..3    wait L2(t-1) and L1(t) -> E1(t) -> issue L2(t) in two groups;
  //   warps 4..7    wait L2(t) -> E2(t) -> key -> the warp's running top-k list, so E2(t) runs
  //                 beside E1(t+1) and L2(t+1).
  if (!is_epi) {
    // ---------------------------------- feature rows ------------------------------------------------
    const int pg = (tid - 256) >> 7, prow = (tid - 256) & 127;
    const uint32_t dst = sA + prow * 16;
    const uint32_t bar_a_prev = pg ? bar_a0 : bar_a1;  // first group of L2 of the other parity's tiles
    const uint32_t bar_x = pg ? bar_x1 : bar_x0, bar_f = pg ? bar_f1 : bar_f0;
#pragma unroll 1
    for (int tile = pg; tile < total_tiles; tile += 2) {
      const int64_t row = tile_row0(tile) + prow;
      const bool live = row < len;
      uint32_t w[32];
#pragma unroll
      for (int q = 0; q < 32; ++q) w[q] = 0u;
      if (kRows) {
        if (live) {
          // the given row: non-finite entries count as 0, every column standardised and rounded
          const float4* src = reinterpret_cast<const float4*>(feat_rows + row * KS_F_PAD);
          float x[64];
          x[63] = 0.0f;
#pragma unroll
          for (int q4 = 0; q4 < KS_F_PAD / 4; ++q4) {
            const float4 v4 = __ldg(src + q4);
            const float v[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              if (4 * q4 + j >= KS_F) continue;
              const int kk = kpos(4 * q4 + j);
              const float f = (fabsf(v[j]) <= 3.402823466e38f) ? v[j] : 0.0f;
              x[kk] = fmaf(f, prm.scale[kk], prm.shift[kk]);
            }
          }
#pragma unroll
          for (int q = 0; q < 32; ++q) w[q] = pack_bf16(x[2 * q], x[2 * q + 1]);
        }
      } else if (live) {
        const int idx = seg_off ? seg_idx[lo + row] : static_cast<int>(row);
        const ks_candidate cand = c[idx];
        const uint4* rec = reinterpret_cast<const uint4*>(cand_cols + (static_cast<size_t>(combo) * C + idx) * kCandRec);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint4 r = __ldg(rec + q);
          w[4 * q] = r.x; w[4 * q + 1] = r.y; w[4 * q + 2] = r.z; w[4 * q + 3] = r.w;
        }
        float x[64];
        auto put = [&](int col, float v) {
          const int kk = kpos(col);  // the per-pair columns sit at the same positions in both forms
          x[kk] = fmaf(v, prm.scale[kk], prm.shift[kk]);
        };
        // single-precision evaluation (the values are rounded to bf16 next); the exact
        // 64-bit form only for tile counts beyond its range
        if (!pair_columns_bf16(s_pt, s_pf, cand, desc, w[15] & 0xFFFFu, put))
          pair_columns<false>(s_pt, cand, desc, static_cast<long long>(w[15] & 0xFFFFu), put);
        // positions 0..28 came from the table; 29..49 are the per-pair columns
        w[14] = (w[14] & 0xFFFFu) | (pack_bf16(0.0f, x[29]) & 0xFFFF0000u);
#pragma unroll
        for (int q = 15; q < 25; ++q) w[q] = pack_bf16(x[2 * q], x[2 * q + 1]);
        if (kOneHot) {
          // positions 50..56: the level indicators of kernel schedule (4) and epilogue schedule (3)
          const unsigned ks = cand.kernel_sched, es = cand.epi_sched;
          auto ind = [&](int q, bool on) { return static_cast<uint32_t>(on ? prm.ind1[q] : prm.ind0[q]); };
          w[25] = ind(0, ks == 0) | (ind(1, ks == 1) << 16);
          w[26] = ind(2, ks == 2) | (ind(3, ks == 3) << 16);
          w[27] = ind(4, es == 0) | (ind(5, es == 1) << 16);
          w[28] = ind(6, es == 2);
        } else {
#pragma unroll
          for (int q = 0; q < 7; ++q) w[25 + q] = s_pwords[q];
        }
      }
      if (tile > 0) {  // planes 0..7 are free once the first group of L2(tile - 1) is done
        if (!wait_ok(bar_a_prev, ph_a)) failed = true;
        ph_a ^= 1;
      }
#pragma unroll
      for (int pl = 0; pl < 8; ++pl)
        asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst + pl * kPlaneA), "r"(w[4 * pl]),
                     "r"(w[4 * pl + 1]), "r"(w[4 * pl + 2]), "r"(w[4 * pl + 3])
                     : "memory");
      fence_async_proxy();
      mbar_arrive(bar_x);
      if ((warp & 3) == 0) {
        // the group's first warp issues L1; its lanes wait together
        if (!wait_ok(bar_x, ph_x)) failed = true;  // every row of the tile is stored
        ph_x ^= 1;
        if (tile >= 2) {  // accumulator tile & 1 was read out by E2(tile - 2)
          if (!wait_ok(bar_f, ph_f)) failed = true;
          ph_f ^= 1;
        }
        if (lane == 0) {
          tc_fence_after();
#pragma unroll
          for (int ks16 = 0; ks16 < 4; ++ks16)
            umma(tmem + (tile & 1) * 256, make_desc(sA + ks16 * 2 * kPlaneA, kPlaneA, 128),
                 make_desc(sbase + kOffW1 + ks16 * 2 * kPlaneB, kPlaneB, 128), ks16 > 0);
          umma_commit(bar_c);
        }
        __syncwarp();
      }
    }
  } else {
    // ---------------------------------- epilogue warps ----------------------------------------------
    // warps 0..3: first epilogue + L2 issue; warps 4..7: second epilogue + ranking keys. Thread
    // (quarter, lane) of either group owns row quarter * 32 + lane and all 256 columns.
    const int quarter = warp & 3, group = warp >> 2;
    const int trow = quarter * 32 + lane;
    const uint32_t tmem_row = tmem + (static_cast<uint32_t>(quarter * 32) << 16);
    if (group == 0) {
#pragma unroll 1
      for (int tile = 0; tile < total_tiles; ++tile) {
        const uint32_t acc = tmem + (tile & 1) * 256, acc_row = tmem_row + (tile & 1) * 256;
        if (tile > 0) {  // the A buffer is free once L2(tile - 1) is complete
          if (!wait_ok((tile & 1) ? bar_b0 : bar_b1, ph_b[(tile - 1) & 1])) failed = true;
          ph_b[(tile - 1) & 1] ^= 1;
        }
        if (!wait_ok(bar_c, ph_c)) failed = true;  // L1(tile) is complete
        ph_c ^= 1;
        tc_fence_after();
        if (kOneHot) epilogue1<0, true>(acc_row, sA + trow * 16, prm, s_b1);
        else epilogue1<0, false>(acc_row, sA + trow * 16, prm, s_b1);
        fence_async_proxy();
        tc_fence_before();
        epi_sync();
        if (tid == 0) {
          tc_fence_after();
#pragma unroll
          for (int ks16 = 0; ks16 < 4; ++ks16)
            umma(acc, make_desc(sA + ks16 * 2 * kPlaneA, kPlaneA, 128),
                 make_desc(sbase + kOffW2 + ks16 * 2 * kPlaneB, kPlaneB, 128), ks16 > 0);
          umma_commit((tile & 1) ? bar_a1 : bar_a0);
#pragma unroll
          for (int ks16 = 4; ks16 < 16; ++ks16)
            umma(acc, make_desc(sA + ks16 * 2 * kPlaneA, kPlaneA, 128),
                 make_desc(sbase + kOffW2 + ks16 * 2 * kPlaneB, kPlaneB, 128), 1u);
          umma_commit((tile & 1) ? bar_b1 : bar_b0);
        }
      }
    } else {
#pragma unroll 1
      for (int tile = 0; tile < total_tiles; ++tile) {
        const uint32_t acc_row = tmem_row + (tile & 1) * 256;
        const int64_t row = tile_row0(tile) + trow;
        int idx = -1;  // fetched before the wait, so that its latency hides behind it
        if (row < len) idx = (!kRows && seg_off) ? __ldg(seg_idx + lo + row) : static_cast<int>(row);
        if (!wait_ok((tile & 1) ? bar_b1 : bar_b0, ph_b[tile & 1])) failed = true;  // L2(tile) is complete
        ph_b[tile & 1] ^= 1;
        tc_fence_after();
        const float score = epilogue2<0>(acc_row, prm) + prm.b3;
        tc_fence_before();
        mbar_arrive((tile & 1) ? bar_f1 : bar_f0);
        if (kRows) {
          if (idx >= 0) score_out[row] = score + 0.0f;
        } else {
          warp_topk_insert(top, idx >= 0 ? make_key(score + 0.0f, idx) : 0ull, k);
        }
      }
      s_merge[quarter][lane] = top;
    }
  }
  // merge the four warps' lists: the j-th best is the largest key below the (j-1)-th
  if (__syncthreads_or(failed)) {
    if (tid == 0 && status) atomicExch(status, KS_ERR_TIMEOUT);
    failed = true;
  }
  if (warp == 0 && !kRows) {
    unsigned long long mine[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) mine[q] = s_merge[q][lane];
    unsigned long long prev = ~0ull;
    for (int j = 0; j < k; ++j) {
      unsigned long long best = 0ull;
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (mine[q] < prev && mine[q] > best) best = mine[q];
      best = warp_max_u64(best);
      if (lane == 0) partial[(static_cast<size_t>(prob) * nblk + chunk) * k + j] = failed ? 0ull : best;
      prev = best;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512) : "memory");
  }
}

}  // namespace

// ------------------------------------------------------------------------------------------
// host
// ------------------------------------------------------------------------------------------

static float bf16_bits_to_float_host(uint16_t b) {
  const uint32_t u = static_cast<uint32_t>(b) << 16;
  float f;
  std::memcpy(&f, &u, 4);
  return f;
}

cudaError_t build_fast_mlp(MlpModel& m, const uint16_t* const* h_w_in, const float* const* h_b_in,
                           const float* h_mu, const float* h_sigma) {
  m.tc = false;
  const int in0 = m.widths[0];
  // One or two hidden layers of at most kH units each: narrower layers are padded with units
  // whose weights and bias are zero (they stay zero through ReLU and contribute nothing), and a
  // single hidden layer gets an identity second layer (its activations are non-negative bf16
  // values, which ReLU and the rounding leave unchanged). Other shapes stay on the generic kernel.
  if ((m.n_layers != 2 && m.n_layers != 3) || (in0 != KS_F_PAD && in0 != KS_F_ONEHOT)) return cudaSuccess;
  for (int l = 1; l < m.n_layers; ++l)
    if (m.widths[l] > kH) return cudaSuccess;
  const bool onehot = in0 == KS_F_ONEHOT;
  const int h1 = m.widths[1], h2 = m.n_layers == 3 ? m.widths[2] : m.widths[1];
  std::vector<uint16_t> pw1(static_cast<size_t>(kH) * in0, 0), pw2(static_cast<size_t>(kH) * kH, 0), pw3(kH, 0);
  std::vector<float> pb1(kH, 0.0f), pb2(kH, 0.0f);
  for (int n = 0; n < h1; ++n) {
    std::memcpy(&pw1[static_cast<size_t>(n) * in0], &h_w_in[0][static_cast<size_t>(n) * in0], sizeof(uint16_t) * in0);
    pb1[n] = h_b_in[0][n];
  }
  if (m.n_layers == 3) {
    for (int n = 0; n < h2; ++n) {
      for (int kk = 0; kk < h1; ++kk) pw2[static_cast<size_t>(n) * kH + kk] = h_w_in[1][static_cast<size_t>(n) * h1 + kk];
      pb2[n] = h_b_in[1][n];
    }
  } else {
    for (int n = 0; n < h1; ++n) pw2[static_cast<size_t>(n) * kH + n] = 0x3F80;  // bf16 1.0
  }
  for (int n = 0; n < h2; ++n) pw3[n] = h_w_in[m.n_layers - 1][n];
  const uint16_t* h_w[3] = {pw1.data(), pw2.data(), pw3.data()};
  const float b3v = h_b_in[m.n_layers - 1][0];
  const float* h_b[3] = {pb1.data(), pb2.data(), &b3v};
  // source of every K position: the model's input position that feeds it (-1: zero), and the
  // folded standardisation x' = x * scale + shift
  int src_at[64];
  for (int q = 0; q < 64; ++q) src_at[q] = -1;
  int oh_pos[KS_F];  // one-hot form: input position of every kept feature column
  {
    int pos = 0;
    for (int col = 0; col < KS_F; ++col) oh_pos[col] = (col == 5 || col == 9 || col == 17 || col == 18) ? -1 : pos++;
  }
  if (!onehot) {
    for (int col = 0; col < KS_F; ++col) src_at[kpos(col)] = col;
  } else {
    for (int col = 0; col < KS_F; ++col)
      if (kpos_oh(col) >= 0) src_at[kpos_oh(col)] = oh_pos[col];
    for (int q = 0; q < 7; ++q) src_at[kIndPos + q] = 66 + q;  // kernel schedule 66..69, epilogue schedule 70..72
  }
  MlpTcParams* prm = new (std::nothrow) MlpTcParams();
  if (!prm) return cudaErrorMemoryAllocation;
  std::memset(prm, 0, sizeof(*prm));
  auto fold = [&](int src, float& scale, float& shift) {
    const double s = 1.0 / static_cast<double>(h_sigma[src]);
    scale = static_cast<float>(s);
    shift = static_cast<float>(-static_cast<double>(h_mu[src]) * s);
  };
  for (int kk = 0; kk < 64; ++kk)
    if (src_at[kk] >= 0) fold(src_at[kk], prm->scale[kk], prm->shift[kk]);
  for (int j = 0; j < kH; ++j) {
    prm->b1[j] = h_b[0][j];
    prm->b2[j] = h_b[1][j];
    prm->w3[j] = bf16_bits_to_float_host(h_w[2][j]);
  }
  prm->b3 = h_b[2][0];
  prm->onehot = onehot ? 1 : 0;
  std::vector<float> w1p;
  if (onehot) {
    auto bf16_of = [](float v) {
      const __nv_bfloat16 b = __float2bfloat16_rn(v);
      uint16_t u;
      std::memcpy(&u, &b, 2);
      return u;
    };
    for (int q = 0; q < 7; ++q) {
      prm->ind0[q] = bf16_of(fmaf(0.0f, prm->scale[kIndPos + q], prm->shift[kIndPos + q]));
      prm->ind1[q] = bf16_of(fmaf(1.0f, prm->scale[kIndPos + q], prm->shift[kIndPos + q]));
    }
    // the folded inputs: their input positions, standardisation and first-layer weights
    int fold_src[kFold];
    for (int col = 0; col < KS_F; ++col)
      if (kfold(col) >= 0) fold_src[kfold(col)] = oh_pos[col];
    for (int l = 0; l < 7; ++l) fold_src[kFoldCols + l] = 59 + l;  // operand type 59..62, activation 63..65
    w1p.resize(static_cast<size_t>(kFold) * kH);
    for (int q = 0; q < kFold; ++q) {
      fold(fold_src[q], prm->p_scale[q], prm->p_shift[q]);
      for (int n = 0; n < kH; ++n)
        w1p[static_cast<size_t>(q) * kH + n] = bf16_bits_to_float_host(h_w[0][static_cast<size_t>(n) * in0 + fold_src[q]]);
    }
  }
  // operand images: plane (k / 8), 16 bytes per output unit
  std::vector<uint16_t> img((kW1Bytes + kW2Bytes) / 2, 0);
  for (int n = 0; n < kH; ++n)
    for (int kk = 0; kk < 64; ++kk)
      if (src_at[kk] >= 0)
        img[(kk / 8) * (kPlaneB / 2) + n * 8 + (kk % 8)] = h_w[0][static_cast<size_t>(n) * in0 + src_at[kk]];
  uint16_t* w2 = img.data() + kW1Bytes / 2;
  for (int n = 0; n < kH; ++n)
    for (int kk = 0; kk < kH; ++kk) w2[(kk / 8) * (kPlaneB / 2) + n * 8 + (kk % 8)] = h_w[1][static_cast<size_t>(n) * kH + kk];
  cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&m.d_tc_image), img.size() * 2);
  if (e == cudaSuccess) e = cudaMemcpy(m.d_tc_image, img.data(), img.size() * 2, cudaMemcpyHostToDevice);
  if (e == cudaSuccess && onehot) {
    e = cudaMalloc(reinterpret_cast<void**>(&m.d_w1_prob), w1p.size() * sizeof(float));
    if (e == cudaSuccess) e = cudaMemcpy(m.d_w1_prob, w1p.data(), w1p.size() * sizeof(float), cudaMemcpyHostToDevice);
    prm->w1_prob = m.d_w1_prob;
  }
  if (e != cudaSuccess) {
    delete prm;
    return e;
  }
  m.h_tc_params = prm;
  m.tc = true;
  return cudaSuccess;
}

void free_fast_mlp(MlpModel& m) {
  delete m.h_tc_params;
  m.h_tc_params = nullptr;
}

// CTAs per problem. A CTA's set-up (160 KB of weights, TMEM, problem terms) is worth about 128
// tiles; with few problems the tiles are spread over one CTA per SM instead.
int mlp_tc_blocks_per_problem(int P, int64_t per_problem) {
  int64_t tiles = (per_problem + kTileRows - 1) / kTileRows;
  if (tiles < 1) tiles = 1;
  int64_t nblk = (tiles + 127) / 128;
  const int64_t fill = (148 + P - 1) / (P > 0 ? P : 1);  // CTAs per problem that fill the machine once
  if (nblk < fill) nblk = fill < tiles ? fill : tiles;
  return static_cast<int>(nblk);
}

size_t mlp_tc_scratch_bytes(int C) { return 256 + static_cast<size_t>(kCombos) * C * kCandRec; }

cudaError_t launch_select_mlp_tc(const ks_gpu_desc& desc, const MlpModel& m, const ks_problem* d_p,
                                 const ks_problem* p_by_value, int P, const ks_candidate* d_c, int C, int nblk,
                                 const int64_t* seg_off, const int32_t* seg_idx, int k,
                                 unsigned long long* partial, void* scratch, int* status, cudaStream_t stream,
                                 int64_t* launches, cudaEvent_t ev_begin, const FastWait* wait) {
  m.h_tc_params->wait_limit = wait && wait->limit > 0 ? wait->limit : kMlpWaitLimit;
  m.h_tc_params->starve = wait ? wait->starve : 0;
  ks_problem pv{};
  if (p_by_value) pv = *p_by_value;
  const int uv = p_by_value != nullptr;
  unsigned* d_mask = static_cast<unsigned*>(scratch);
  uint8_t* d_cols = static_cast<uint8_t*>(scratch) + 256;
  unsigned mask_value = 0;
  cudaError_t e;
  if (uv) {
    mask_value = 1u << ((pv.dtype_ab & 3) * 4 + (pv.dtype_d & 3));
  } else {
    e = cudaMemsetAsync(d_mask, 0, sizeof(unsigned), stream);
    if (e != cudaSuccess) return e;
    mlp_combo_mask_kernel<<<P >= 4096 ? 16 : 1, 256, 0, stream>>>(d_p, P, d_mask);
    ++*launches;
  }
  if (C > 0) {
    mlp_cand_cols_kernel<<<dim3((C + 255) / 256, kCombos), 256, 0, stream>>>(desc, d_c, C, uv ? nullptr : d_mask,
                                                                             mask_value, *m.h_tc_params, d_cols);
    ++*launches;
  }
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (ev_begin) cudaEventRecord(ev_begin, stream);
  const unsigned grid = static_cast<unsigned>(static_cast<int64_t>(P) * nblk);
  const uint8_t* image = reinterpret_cast<const uint8_t*>(m.d_tc_image);
  if (m.h_tc_params->onehot) {
    e = ensure_dynamic_smem(reinterpret_cast<const void*>(&select_mlp_tc_kernel<1>), kSmemBytes);
    if (e != cudaSuccess) return e;
    select_mlp_tc_kernel<1><<<grid, kT, kSmemBytes, stream>>>(desc, d_p, pv, uv, d_c, P, C, nblk, seg_off, seg_idx, image,
                                                              d_cols, k, partial, status, nullptr, nullptr,
                                                              *m.h_tc_params);
  } else {
    e = ensure_dynamic_smem(reinterpret_cast<const void*>(&select_mlp_tc_kernel<0>), kSmemBytes);
    if (e != cudaSuccess) return e;
    select_mlp_tc_kernel<0><<<grid, kT, kSmemBytes, stream>>>(desc, d_p, pv, uv, d_c, P, C, nblk, seg_off, seg_idx, image,
                                                              d_cols, k, partial, status, nullptr, nullptr,
                                                              *m.h_tc_params);
  }
  ++*launches;
  return cudaGetLastError();
}

// ks_score on the tensor-core kernel (ordinal input form): one CTA per SM, each with an equal
// share of the 128-row tiles; rows in batches that fit the kernel's 32-bit row count.
bool score_mlp_tc_ok(const MlpModel& m) { return m.tc && m.h_tc_params && !m.h_tc_params->onehot; }

cudaError_t launch_score_mlp_tc(const ks_gpu_desc& desc, const MlpModel& m, const float* d_feat, int64_t rows,
                                float* d_scores, int* status, cudaStream_t stream, int64_t* launches,
                                const FastWait* wait) {
  m.h_tc_params->wait_limit = wait && wait->limit > 0 ? wait->limit : kMlpWaitLimit;
  m.h_tc_params->starve = wait ? wait->starve : 0;
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(&select_mlp_tc_kernel<2>), kSmemBytes);
  if (e != cudaSuccess) return e;
  const uint8_t* image = reinterpret_cast<const uint8_t*>(m.d_tc_image);
  const ks_problem pv{};
  constexpr int64_t kBatch = int64_t{1} << 30;
  mlp_reset_abort_kernel<<<1, 1, 0, stream>>>();
  ++*launches;
  for (int64_t first = 0; first < rows; first += kBatch) {
    const int64_t n = rows - first < kBatch ? rows - first : kBatch;
    const int64_t tiles = (n + kTileRows - 1) / kTileRows;
    const int nblk = static_cast<int>(tiles < 148 ? tiles : 148);
    select_mlp_tc_kernel<2><<<nblk, kT, kSmemBytes, stream>>>(desc, nullptr, pv, 1, nullptr, 1, static_cast<int>(n), nblk,
                                                              nullptr, nullptr, image, nullptr, 0, nullptr, status,
                                                              d_feat + first * KS_F_PAD, d_scores + first,
                                                              *m.h_tc_params);
    ++*launches;
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace ks

