// Dense attention partials over the uncompressed tail (Sec. 4 "Implementation details": tokens generated
// during decoding are not compressed).  One CTA per (128-row split of the tail, problem) writes, per query head,
// (acc[d_h], m, l): the unnormalised output, the running maximum of the scaled logits in log2 units and the sum
// of 2^(z - m).  The segment merge of the fused kernel folds these in.  Two kernels: `tail_tc_kernel` (d_h = 128)
// forms the tile's logits and value sums on the tensor core; `tail_partial_kernel` is the CUDA-core version
// (thread = tail row for the logits, thread = output column for the weighted sum of value rows), used for
// d_h = 64 and when the handle was created with XKV_TAIL_IMPL=c.
#include <math.h>

#include "xkv_internal.cuh"
#include "xkv_ptx.cuh"

namespace xkv {

namespace {

constexpr int kTailThreads = 128;   // = rows per tile
constexpr float kLog2e = 1.4426950408889634f;

// NR: query heads per KV head rounded up to 4, 8 or 16 (the loops over heads are unrolled to NR, not to the
// largest supported count: the unrolled code has to stay inside the instruction cache).
// One CTA = one 128-row tile (kTailSplitRows == kTailThreads): its K and V rows are brought into shared memory
// with one burst of 16-byte cp.async copies, so the CTA pays one memory round trip.
template <int DH>
constexpr int tail_k_stride() { return DH * 2 + 16; }   // bytes per staged key row: padded against bank conflicts, 16-byte multiple

template <int DH, int NR>
constexpr size_t tail_smem_bytes() {
  return (size_t)kTailThreads * tail_k_stride<DH>() + (size_t)kTailThreads * DH * 2 + sizeof(float) * (NR * DH + NR * kTailThreads);
}

template <int DH, int NR>
__global__ void __launch_bounds__(kTailThreads)
tail_partial_kernel(GroupDev dev, int l0, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ tail_k,
                    const __nv_bfloat16* __restrict__ tail_v, const int32_t* __restrict__ tail_len, int tail_cap,
                    int n_split, float* __restrict__ part) {
  static_assert(kTailSplitRows == kTailThreads, "one tile per CTA");
  extern __shared__ __align__(16) uint8_t tail_smem[];
  constexpr int KS = tail_k_stride<DH>();
  uint8_t* k_s = tail_smem;                                           // [128][KS]
  __nv_bfloat16* v_s = reinterpret_cast<__nv_bfloat16*>(k_s + kTailThreads * KS);     // [128][DH]
  float* q_s = reinterpret_cast<float*>(v_s + kTailThreads * DH);     // [DH][NR]
  float* p_s = q_s + NR * DH;                                         // [128][NR] weights of the tile
  __shared__ float red_s[NR * (kTailThreads / 32)];
  __shared__ float m_s[NR];
  __shared__ float fold_s[kTailThreads];               // d_h = 64: the two halves of the row range meet here
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int py = blockIdx.x, split = blockIdx.y;
  const int per_layer = dev.batch * dev.H_kv, n_rep = dev.n_rep;
  const int g = py % dev.H_kv, b = (py / dev.H_kv) % dev.batch, l = l0 + py / per_layer;
  const float scale2 = dev.att_scale * kLog2e;

  ptx::grid_dependency_wait();                         // q (and the tail rows) may come from the kernel before
  ptx::grid_dependency_launch();
  int len = tail_len ? tail_len[b] : tail_cap;
  if (len < 0 || len > tail_cap) {
    if (tid == 0 && split == 0) atomicOr(dev.flags, XKV_FLAG_INDEX_RANGE);
    len = len < 0 ? 0 : tail_cap;
  }
  const int r_begin = split * kTailSplitRows;
  const int rows = max(0, min(len - r_begin, kTailSplitRows));

  // ---- stage the tile: 16-byte pieces, consecutive threads take consecutive pieces of a row
  const size_t head_rows = (((size_t)l * dev.batch + b) * dev.H_kv + g) * (size_t)tail_cap + r_begin;
  const __nv_bfloat16* Kh = tail_k + head_rows * DH;
  const __nv_bfloat16* Vh = tail_v + head_rows * DH;
  constexpr int PPR = DH / 8;                          // 16-byte pieces per row
  // two copy groups: the logits start as soon as the keys are in, the values land meanwhile
  for (int i = tid; i < rows * PPR; i += kTailThreads) {
    const int r = i / PPR, c = i % PPR;
    ptx::cp_async16(ptx::smem_u32(k_s + r * KS + c * 16), Kh + (size_t)r * DH + c * 8, 16u);
  }
  ptx::cp_async_commit();
  for (int i = tid; i < rows * PPR; i += kTailThreads) {
    const int r = i / PPR, c = i % PPR;
    ptx::cp_async16(ptx::smem_u32(v_s + r * DH + c * 8), Vh + (size_t)r * DH + c * 8, 16u);
  }
  ptx::cp_async_commit();
  const __nv_bfloat16* qg = q + (((long long)l * dev.batch + b) * dev.H_q + (long long)g * n_rep) * DH;
  // queries head-minor, [dim][head]: one 16-byte load gives one dimension of four heads, which pair up in the
  // packed multiply-adds below
  for (int i = tid; i < NR * DH; i += kTailThreads) {
    const int h = i / DH, dd = i - h * DH;
    q_s[dd * NR + h] = h < n_rep ? __bfloat162float(qg[i]) : 0.0f;
  }
  ptx::cp_async_wait<1>();                             // the keys of this thread's copies are in
  __syncthreads();

  // ---- logits of row `tid` against every head
  const bool valid = tid < rows;
  float z[NR];
  {
    // two heads per fma.rn.f32x2 (each half is an ordinary fused multiply-add: same sums, half the instructions
    // of a kernel that is bound by their number)
    float2 z2[NR / 2];
#pragma unroll
    for (int hp = 0; hp < NR / 2; ++hp) z2[hp] = make_float2(0.0f, 0.0f);
    if (valid) {
      const uint4* kr = reinterpret_cast<const uint4*>(k_s + tid * KS);
#pragma unroll 2
      for (int cc = 0; cc < DH / 8; ++cc) {
        const uint4 v = kr[cc];
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        float kf[8];
#pragma unroll
        for (int e = 0; e < 4; ++e) { kf[2 * e] = __uint_as_float(w[e] << 16); kf[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u); }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float2 kk = make_float2(kf[e], kf[e]);
#pragma unroll
          for (int h4 = 0; h4 < NR / 4; ++h4) {
            const float4 q4 = *reinterpret_cast<const float4*>(q_s + (cc * 8 + e) * NR + h4 * 4);
            z2[2 * h4] = __ffma2_rn(make_float2(q4.x, q4.y), kk, z2[2 * h4]);
            z2[2 * h4 + 1] = __ffma2_rn(make_float2(q4.z, q4.w), kk, z2[2 * h4 + 1]);
          }
        }
      }
    }
#pragma unroll
    for (int hp = 0; hp < NR / 2; ++hp) { z[2 * hp] = z2[hp].x; z[2 * hp + 1] = z2[hp].y; }
  }
  // ---- tile maximum per head
#pragma unroll
  for (int h = 0; h < NR; ++h) {
    z[h] = valid ? z[h] * scale2 : -INFINITY;
    float v = z[h];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    if (lane == 0) red_s[h * (kTailThreads / 32) + warp] = v;
  }
  __syncthreads();
  if (tid < NR) {
    float tm = red_s[tid * (kTailThreads / 32)];
#pragma unroll
    for (int w = 1; w < kTailThreads / 32; ++w) tm = fmaxf(tm, red_s[tid * (kTailThreads / 32) + w]);
    m_s[tid] = tm;
  }
  __syncthreads();
  // ---- weights (kept in fp32: the CUDA-core value phase has no operand format to round to), row-major and
  // head-minor like the queries, and their sums per head
#pragma unroll
  for (int h = 0; h < NR; ++h) {
    const float mn = m_s[h];
    const float p = (valid && mn != -INFINITY) ? exp2f(z[h] - mn) : 0.0f;
    p_s[tid * NR + h] = p;
    float v = p;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane == 0) red_s[h * (kTailThreads / 32) + warp] = v;      // (the maxima in red_s were consumed before the last barrier)
  }
  ptx::cp_async_wait<0>();                             // the values too
  __syncthreads();
  // ---- value phase: thread -> output column d and, for d_h = 64, one half of the tile's rows
  constexpr int PARTS = kTailThreads / DH;
  const int d = tid % DH, vpart = tid / DH;
  float acc[NR];
  {
    float2 a2[NR / 2];
#pragma unroll
    for (int hp = 0; hp < NR / 2; ++hp) a2[hp] = make_float2(0.0f, 0.0f);
    const int row_lo = vpart * (kTailThreads / PARTS), row_hi = min(rows, row_lo + kTailThreads / PARTS);
#pragma unroll 4
    for (int jj = row_lo; jj < row_hi; ++jj) {
      const float vv = __bfloat162float(v_s[jj * DH + d]);
      const float2 v2 = make_float2(vv, vv);
#pragma unroll
      for (int h4 = 0; h4 < NR / 4; ++h4) {
        const float4 p4 = *reinterpret_cast<const float4*>(p_s + jj * NR + h4 * 4);
        a2[2 * h4] = __ffma2_rn(make_float2(p4.x, p4.y), v2, a2[2 * h4]);
        a2[2 * h4 + 1] = __ffma2_rn(make_float2(p4.z, p4.w), v2, a2[2 * h4 + 1]);
      }
    }
#pragma unroll
    for (int hp = 0; hp < NR / 2; ++hp) { acc[2 * hp] = a2[hp].x; acc[2 * hp + 1] = a2[hp].y; }
  }

  // ---- write the partial: [py][split][head][DH + 2]
  float* dst = part + (((size_t)py * n_split + split) * n_rep) * (DH + 2);
#pragma unroll
  for (int h = 0; h < NR; ++h) {
    if (h < n_rep) {
      float a = acc[h];
      float ls = 0.0f;
#pragma unroll
      for (int w = 0; w < kTailThreads / 32; ++w) ls += red_s[h * (kTailThreads / 32) + w];
      if (PARTS > 1) {                                   // d_h = 64: add the other half of the rows
        if (vpart == 1) fold_s[d] = a;
        __syncthreads();
        if (vpart == 0) a += fold_s[d];
        __syncthreads();
      }
      if (vpart == 0) {
        dst[(size_t)h * (DH + 2) + d] = a;
        if (d == 0) { dst[(size_t)h * (DH + 2) + DH] = m_s[h]; dst[(size_t)h * (DH + 2) + DH + 1] = ls; }
      }
    }
  }
}


// ---------------------------------------------------------------------------------------------
// The same partials on the tensor core, for d_h = 128.  Per 128-row tile: logits S[row][head] = K q^T
// (tcgen05.mma, M = rows, N = 16 heads, K = d_h, both operands K-major), softmax statistics and weights by
// thread = row = TMEM lane, then O^T[d][head] = V^T P^T (A = the value tile read along its rows, MN-major,
// B = the bf16 weights), read back by thread = d = TMEM lane.  The sixteen small MMAs replace ~2 k multiply-adds
// per thread, so a CTA spends its time on its loads.  Weights are rounded to bf16 for the MMA; the denominator
// sums the rounded weights, like the reconstructed rows' path does.
constexpr int kTcSlab = kTailThreads * 128;           // 128 rows x 64 bf16, 128-byte swizzle
constexpr uint32_t kTcWaitLimit = 1u << 22;

template <int NR>
constexpr size_t tail_tc_smem_bytes() {
  return 1024 + 4 * (size_t)kTcSlab + 2 * 2048 + 4096 + 64;   // K and V tiles (two slabs each), q operand, weights, barriers
}

__device__ __forceinline__ bool tc_wait_bounded(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < kTcWaitLimit; ++i) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
  }
  return false;
}

template <int NR>
__global__ void __launch_bounds__(kTailThreads)
tail_tc_kernel(GroupDev dev, int l0, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ tail_k,
               const __nv_bfloat16* __restrict__ tail_v, const int32_t* __restrict__ tail_len, int tail_cap,
               int n_split, int tiles_per_split, float* __restrict__ part) {
  using namespace ptx;
  constexpr int DH = 128;
  extern __shared__ uint8_t tc_smem[];
  __shared__ float red_s[NR * (kTailThreads / 32)];
  __shared__ float m_s[2][NR];                         // running maximum per head, before and after the current tile
  const uint32_t base = (smem_u32(tc_smem) + 1023u) & ~1023u;
  uint8_t* gen = tc_smem + (base - smem_u32(tc_smem));
  const uint32_t k_addr = base, v_addr = base + 2 * kTcSlab, q_addr = base + 4 * kTcSlab, p_addr = q_addr + 4096;
  uint8_t* q_gen = gen + 4 * kTcSlab;
  uint8_t* p_gen = q_gen + 4096;
  uint64_t* bars = reinterpret_cast<uint64_t*>(p_gen + 4096);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2);
  const uint32_t bar_s = smem_u32(bars), bar_o = bar_s + 8;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int py = blockIdx.x, split = blockIdx.y;
  const int per_layer = dev.batch * dev.H_kv, n_rep = dev.n_rep;
  const int g = py % dev.H_kv, b = (py / dev.H_kv) % dev.batch, l = l0 + py / per_layer;
  const float scale2 = dev.att_scale * kLog2e;

  if (tid == 0) {
    mbar_init(bar_s, 1);
    mbar_init(bar_o, 1);
    fence_mbar_init();
  }
  // operands that stay zero: heads that do not exist (q rows, weight rows)
  for (int i = tid; i < 8192 / 4; i += kTailThreads) reinterpret_cast<uint32_t*>(q_gen)[i] = 0u;
  if (tid < NR) { m_s[0][tid] = -INFINITY; m_s[1][tid] = -INFINITY; }
  if (warp == 0) {
    tmem_alloc(smem_u32(tmem_slot), 32);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  grid_dependency_wait();                              // q (and the tail rows) may come from the kernel before
  grid_dependency_launch();
  int len = tail_len ? tail_len[b] : tail_cap;
  if (len < 0 || len > tail_cap) {
    if (tid == 0 && split == 0) atomicOr(dev.flags, XKV_FLAG_INDEX_RANGE);
    len = len < 0 ? 0 : tail_cap;
  }
  // q as the B operand of the logits: [16 heads][128 dims], K-major, 64-column slabs, 128-byte swizzle
  const __nv_bfloat16* qg = q + (((long long)l * dev.batch + b) * dev.H_q + (long long)g * n_rep) * DH;
  for (int i = tid; i < n_rep * 16; i += kTailThreads) {
    const int h = i >> 4, c = i & 15;
    const uint4 v = *reinterpret_cast<const uint4*>(qg + h * DH + c * 8);
    *reinterpret_cast<uint4*>(q_gen + (c >> 3) * 2048 + h * 128 + (((c & 7) ^ (h & 7)) << 4)) = v;
  }
  const uint64_t desc_hi = smem_desc_sw128(0, 0) & 0xFFFFFFFF00000000ull;
  constexpr uint32_t idesc_s = idesc_bf16_f32(128, 16);
  constexpr uint32_t idesc_o = idesc_bf16_f32(128, 16) | (1u << 15);          // A read along its rows (MN-major)
  const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
  const size_t head_rows = (((size_t)l * dev.batch + b) * dev.H_kv + g) * (size_t)tail_cap;

  // running results of the split: thread = output column d for acc, thread = row for the weight sums
  float acc[NR], l_thr[NR];
#pragma unroll
  for (int h = 0; h < NR; ++h) { acc[h] = 0.0f; l_thr[h] = 0.0f; }
  bool ok = true;
  int issued = 0;                                      // MMA group committed and not yet known to have retired: 0 none, 1 logits, 2 values
  uint32_t issued_par = 0;                             // barrier phase that group completes
  // A split is `tiles_per_split` consecutive 128-row tiles, walked with a running softmax (one tile for tails up
  // to XKV_TAIL_MAX_ROWS; more for the long caches of xkv_dense_attend, so that the merge sees a bounded number
  // of partial results).
  for (int t = 0; t < tiles_per_split; ++t) {
    const int r_begin = (split * tiles_per_split + t) * kTailSplitRows;
    const int rows = max(0, min(len - r_begin, kTailSplitRows));
    if (rows == 0 && t > 0) break;                     // CTA-uniform: the split ends inside the cache
    const int cur = t & 1, nxt = cur ^ 1;
    const uint32_t par = (uint32_t)(t & 1);
    // ---- stage K and V in the tensor core's layout: 64-column slabs, 128-byte rows, 16-byte units swizzled by
    // the row; rows beyond `rows` are zero-filled (a weight of zero times garbage would still be garbage)
    const __nv_bfloat16* Kh = tail_k + (head_rows + r_begin) * DH;
    const __nv_bfloat16* Vh = tail_v + (head_rows + r_begin) * DH;
    for (int i = tid; i < kTailThreads * 16; i += kTailThreads) {
      const int r = i >> 4, c = i & 15;                // row, 16-byte piece of the 256-byte row
      const uint32_t off = (uint32_t)(c >> 3) * kTcSlab + (uint32_t)r * 128u + ((((uint32_t)c & 7u) ^ ((uint32_t)r & 7u)) << 4);
      const uint32_t nb = r < rows ? 16u : 0u;
      const size_t src = (size_t)(r < rows ? r : 0) * DH + c * 8;
      cp_async16(k_addr + off, Kh + src, nb);
      cp_async16(v_addr + off, Vh + src, nb);
    }
    cp_async_commit();
    cp_async_wait<0>();
    fence_proxy_async();                               // the tensor core reads what this thread wrote or copied
    __syncthreads();
    // ---- logits
    if (tid == 0) {
      const uint32_t k_lo = (uint32_t)(smem_desc_sw128(k_addr, 0) & 0xFFFFFFFFull);
      const uint32_t q_lo = (uint32_t)(smem_desc_sw128(q_addr, 0) & 0xFFFFFFFFull);
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {                 // 16 dims per step: 32 bytes along the row, next slab after four
        const uint32_t a = k_lo + (uint32_t)(kk >> 2) * (kTcSlab >> 4) + (uint32_t)(kk & 3) * 2u;
        const uint32_t bq = q_lo + (uint32_t)(kk >> 2) * (2048u >> 4) + (uint32_t)(kk & 3) * 2u;
        tc_mma_bf16(tmem, desc_hi | a, desc_hi | bq, idesc_s, kk ? 1u : 0u);
      }
      tc_commit(bar_s);
    }
    issued = 1; issued_par = par;
    // the outcome of a wait is made CTA-uniform (one thread's poll may run out a moment before another's succeeds)
    ok = __syncthreads_and(tc_wait_bounded(bar_s, par) ? 1 : 0) != 0;
    if (!ok) break;
    issued = 0;
    tc_fence_after();
    const bool valid = tid < rows;
    float z[NR];
    tmem_ld<NR>(tmem + lane_base, z);
    tc_wait_ld();
    // ---- tile maximum per head, folded into the running maximum
#pragma unroll
    for (int h = 0; h < NR; ++h) {
      z[h] = valid ? z[h] * scale2 : -INFINITY;
      float v = z[h];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
      if (lane == 0) red_s[h * (kTailThreads / 32) + warp] = v;
    }
    __syncthreads();
    if (tid < NR) {
      float tm = red_s[tid * (kTailThreads / 32)];
#pragma unroll
      for (int w = 1; w < kTailThreads / 32; ++w) tm = fmaxf(tm, red_s[tid * (kTailThreads / 32) + w]);
      m_s[nxt][tid] = fmaxf(m_s[cur][tid], tm);
    }
    __syncthreads();
    // ---- weights as the bf16 B operand [row block][head][64 rows]; the denominator sums the rounded values
    float alpha[NR];
    {
      uint8_t* Pw = p_gen + (tid >> 6) * 2048 + (tid & 7) * 2;
      const uint32_t p_unit = (uint32_t)((tid & 63) >> 3);
#pragma unroll
      for (int h = 0; h < NR; ++h) {
        const float mo = m_s[cur][h], mn = m_s[nxt][h];
        alpha[h] = (mo == -INFINITY) ? 0.0f : ex2_approx(mo - mn);
        const float p = (valid && mn != -INFINITY) ? ex2_approx(z[h] - mn) : 0.0f;
        const __nv_bfloat16 pb = __float2bfloat16(p);
        if (h < n_rep) *reinterpret_cast<__nv_bfloat16*>(Pw + h * 128 + ((p_unit ^ (uint32_t)(h & 7)) << 4)) = pb;
        l_thr[h] = l_thr[h] * alpha[h] + __bfloat162float(pb);
      }
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // ---- values: O^T[d][head] = V^T P^T
    if (tid == 0) {
      const uint32_t v_lo = ((uint32_t)(smem_desc_sw128(v_addr, 0) & 0xFFFFull)) | ((uint32_t)(kTcSlab >> 4) << 16);
      const uint32_t p_lo = (uint32_t)(smem_desc_sw128(p_addr, 0) & 0xFFFFFFFFull);
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {                 // 16 tile rows per step: 2048 bytes down the slab, 32 bytes along P
        const uint32_t bp = p_lo + (uint32_t)(kk >> 2) * (2048u >> 4) + (uint32_t)(kk & 3) * 2u;
        tc_mma_bf16(tmem + 16u, desc_hi | (v_lo + (uint32_t)kk * (2048u >> 4)), desc_hi | bp, idesc_o, kk ? 1u : 0u);
      }
      tc_commit(bar_o);
    }
    issued = 2; issued_par = par;
    ok = __syncthreads_and(tc_wait_bounded(bar_o, par) ? 1 : 0) != 0;
    if (!ok) break;
    issued = 0;
    tc_fence_after();
    float o[NR];
    tmem_ld<NR>(tmem + lane_base + 16u, o);
    tc_wait_ld();
#pragma unroll
    for (int h = 0; h < NR; ++h) acc[h] = fmaf(acc[h], alpha[h], o[h]);
    tc_fence_before();
    __syncthreads();                                   // the tile's memory and both accumulators may be reused
    tc_fence_after();
  }
  if (!ok) {
    if (tid == 0) {
      atomicOr(dev.flags, XKV_FLAG_TIMEOUT);
      // giving up: the MMAs issued above may still be running; wait once more (bounded) for the barrier that
      // their commit arrives on before the tensor memory is freed
      if (issued) (void)tc_wait_bounded(issued == 1 ? bar_s : bar_o, issued_par);
    }
#pragma unroll
    for (int h = 0; h < NR; ++h) { acc[h] = 0.0f; l_thr[h] = 0.0f; }
  }
  // ---- per head: sum of the weights over the rows (thread = row)
  __syncthreads();
#pragma unroll
  for (int h = 0; h < NR; ++h) {
    float v = l_thr[h];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane == 0) red_s[h * (kTailThreads / 32) + warp] = v;
  }
  __syncthreads();
  // ---- write the partial: [py][split][head][DH + 2].  The running maximum alternates between m_s[0] and m_s[1]
  // and never decreases, so the larger of the two is the final one.
  float* dst = part + (((size_t)py * n_split + split) * n_rep) * (DH + 2);
#pragma unroll
  for (int h = 0; h < NR; ++h) {
    if (h < n_rep) {
      dst[(size_t)h * (DH + 2) + tid] = acc[h];
      if (tid == 0) {
        float ls = 0.0f;
#pragma unroll
        for (int w = 0; w < kTailThreads / 32; ++w) ls += red_s[h * (kTailThreads / 32) + w];
        dst[(size_t)h * (DH + 2) + DH] = ok ? fmaxf(m_s[0][h], m_s[1][h]) : -INFINITY;
        dst[(size_t)h * (DH + 2) + DH + 1] = ls;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem, 32);
  }
}

// Merge of dense-attention partials (xkv_dense_attend): one CTA per (problem, query head); the splits are
// spread over 1024 / DH groups of DH threads, thread = output column.  m is in log2 units.
constexpr int kDenseMergeThreads = 1024;
template <int DH>
__global__ void __launch_bounds__(kDenseMergeThreads)
dense_merge_kernel(GroupDev dev, int l0, const float* __restrict__ part, int n_split, __nv_bfloat16* __restrict__ out,
                   float* __restrict__ lse) {
  __shared__ float twgt_s[kTailMaxSplit];
  __shared__ float ML_s[2];
  __shared__ float red[kDenseMergeThreads];
  constexpr int FOLD = kDenseMergeThreads / DH;
  const int tid = threadIdx.x, n_rep = dev.n_rep;
  const int h = blockIdx.x % n_rep, py = blockIdx.x / n_rep;
  const int per_layer = dev.batch * dev.H_kv;
  const int g = py % dev.H_kv, b = (py / dev.H_kv) % dev.batch, l = l0 + py / per_layer;
  ptx::grid_dependency_wait();                         // the partials come from the kernel launched before this one
  ptx::grid_dependency_launch();
  const int nts = min(n_split, kTailMaxSplit);
  const size_t tstride = (size_t)n_rep * (DH + 2);
  const float* tpart = part + ((size_t)py * n_split) * tstride + (size_t)h * (DH + 2);
  if (tid < 32) {
    float mx = -INFINITY;
    for (int s = tid; s < nts; s += 32) mx = fmaxf(mx, tpart[s * tstride + DH]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float Ls = 0.0f;
    for (int s = tid; s < nts; s += 32) {
      const float ms = tpart[s * tstride + DH];
      const float w = (ms == -INFINITY || mx == -INFINITY) ? 0.0f : exp2f(ms - mx);
      twgt_s[s] = w;
      Ls += w * tpart[s * tstride + DH + 1];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) Ls += __shfl_xor_sync(0xffffffffu, Ls, o);
    if (tid == 0) { ML_s[0] = mx; ML_s[1] = Ls; }
  }
  __syncthreads();
  const int d = tid % DH, f = tid / DH;
  float o = 0.0f;
#pragma unroll 4
  for (int s = f; s < nts; s += FOLD) o = fmaf(twgt_s[s], tpart[s * tstride + d], o);
  red[f * DH + d] = o;
  __syncthreads();
  if (tid < DH) {
    float v = 0.0f;
#pragma unroll
    for (int i = 0; i < FOLD; ++i) v += red[i * DH + tid];
    const float M = ML_s[0], L = ML_s[1];
    const long long qh = ((long long)l * dev.batch + b) * dev.H_q + (long long)g * n_rep + h;
    out[qh * DH + tid] = __float2bfloat16(L > 0.0f ? v / L : 0.0f);
    if (lse && tid == 0) lse[qh] = L > 0.0f ? (M + log2f(L)) * 0.6931471805599453f : -INFINITY;
  }
}

}  // namespace

// Tiles walked by one CTA of the tail kernels: one while the merge's table of partial results holds every tile,
// more for longer caches (dense attention).
int tail_tiles_per_split(int tail_cap) {
  const int tiles = (tail_cap + kTailSplitRows - 1) / kTailSplitRows;
  return (tiles + kTailMaxSplit - 1) / kTailMaxSplit;
}

int tail_splits(int tail_cap) {
  const int tiles = (tail_cap + kTailSplitRows - 1) / kTailSplitRows, tps = tail_tiles_per_split(tail_cap);
  return (tiles + tps - 1) / tps;
}

size_t tail_part_floats(const xkv_group* grp, int tail_cap) {
  const xkv_group_config& c = grp->cfg;
  return (size_t)c.G * c.batch * c.H_kv * tail_splits(tail_cap) * (size_t)(c.H_q / c.H_kv) * (c.d_h + 2);
}

cudaError_t launch_tail_partials(const xkv_group* grp, int l0, int l1, const __nv_bfloat16* q, const __nv_bfloat16* tail_k,
                                 const __nv_bfloat16* tail_v, const int32_t* tail_len, int tail_cap, float* part,
                                 cudaStream_t s) {
  const GroupDev& dev = grp->dev;
  const int problems = (l1 - l0) * dev.batch * dev.H_kv;
  const int n_split = tail_splits(tail_cap), tps = tail_tiles_per_split(tail_cap);
  cudaError_t e = cudaSuccess;
  const dim3 grid(problems, n_split), block(kTailThreads);
  // only the tensor-core kernel walks several tiles per CTA
  if (tps > 1 && !(dev.d_h == 128 && !grp->tail_impl)) return cudaErrorInvalidValue;
#define XKV_TAIL(DH, NR)                                                                                            \
  do {                                                                                                              \
    e = ensure_dyn_smem<tail_partial_kernel<DH, NR>>(tail_smem_bytes<DH, NR>(), grp->device);                       \
    if (e == cudaSuccess)                                                                                           \
      e = launch_pdl(tail_partial_kernel<DH, NR>, grid, block, tail_smem_bytes<DH, NR>(), s, dev, l0, q, tail_k,     \
                     tail_v, tail_len, tail_cap, n_split, part);                                                    \
  } while (0)
#define XKV_TAIL_TC(NR)                                                                                            \
  do {                                                                                                              \
    e = ensure_dyn_smem<tail_tc_kernel<NR>>(tail_tc_smem_bytes<NR>(), grp->device);                                 \
    if (e == cudaSuccess)                                                                                           \
      e = launch_pdl(tail_tc_kernel<NR>, grid, block, tail_tc_smem_bytes<NR>(), s, dev, l0, q, tail_k, tail_v,       \
                     tail_len, tail_cap, n_split, tps, part);                                                       \
  } while (0)
  if (dev.d_h == 128 && !grp->tail_impl) {
    if (dev.n_rep <= 4) XKV_TAIL_TC(4); else if (dev.n_rep <= 8) XKV_TAIL_TC(8); else XKV_TAIL_TC(16);
  } else if (dev.d_h == 128) {
    if (dev.n_rep <= 4) XKV_TAIL(128, 4); else if (dev.n_rep <= 8) XKV_TAIL(128, 8); else XKV_TAIL(128, 16);
  } else {
    if (dev.n_rep <= 4) XKV_TAIL(64, 4); else if (dev.n_rep <= 8) XKV_TAIL(64, 8); else XKV_TAIL(64, 16);
  }
#undef XKV_TAIL
#undef XKV_TAIL_TC
  count_launch((dev.d_h == 128 && !grp->tail_impl) ? kFamTailTc : kFamTailCuda);
  return e;
}

// Can xkv_dense_attend serve `cap` rows with this handle?  Longer caches than the tail limit need the multi-tile
// (tensor-core, d_h = 128) kernel.
bool dense_supported(const xkv_group* grp, int cap) {
  return tail_tiles_per_split(cap) == 1 || (grp->dev.d_h == 128 && !grp->tail_impl);
}

cudaError_t launch_dense_merge(const xkv_group* grp, int l0, int l1, const float* part, int cap, __nv_bfloat16* out,
                               float* lse, cudaStream_t s) {
  const GroupDev& dev = grp->dev;
  const int problems = (l1 - l0) * dev.batch * dev.H_kv;
  cudaError_t e;
  if (dev.d_h == 128)
    e = launch_pdl(dense_merge_kernel<128>, dim3(problems * dev.n_rep), dim3(kDenseMergeThreads), 0, s, dev, l0, part,
                   tail_splits(cap), out, lse);
  else
    e = launch_pdl(dense_merge_kernel<64>, dim3(problems * dev.n_rep), dim3(kDenseMergeThreads), 0, s, dev, l0, part,
                   tail_splits(cap), out, lse);
  count_launch(kFamDense);
  return e;
}

}  // namespace xkv
