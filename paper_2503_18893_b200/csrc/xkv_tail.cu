// Dense attention partials over the uncompressed tail (Sec. 4 "Implementation details": tokens generated
// during decoding are not compressed).  The tail is short next to the factorised context, so this is a plain
// CUDA-core kernel: one CTA per (128-row split of the tail, problem), thread = tail row for the logits,
// thread = output column for the weighted sum of value rows.
// Each CTA writes, per query head, (acc[d_h], m, l): the unnormalised output, the running maximum of the scaled
// logits in log2 units and the sum of 2^(z - m).  The segment merge of the fused kernel folds these in.
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

}  // namespace

int tail_splits(int tail_cap) { return (tail_cap + kTailSplitRows - 1) / kTailSplitRows; }

size_t tail_part_floats(const xkv_group* grp, int tail_cap) {
  const xkv_group_config& c = grp->cfg;
  return (size_t)c.G * c.batch * c.H_kv * tail_splits(tail_cap) * (size_t)(c.H_q / c.H_kv) * (c.d_h + 2);
}

cudaError_t launch_tail_partials(const xkv_group* grp, int l0, int l1, const __nv_bfloat16* q, const __nv_bfloat16* tail_k,
                                 const __nv_bfloat16* tail_v, const int32_t* tail_len, int tail_cap, float* part,
                                 cudaStream_t s) {
  const GroupDev& dev = grp->dev;
  const int problems = (l1 - l0) * dev.batch * dev.H_kv;
  const int n_split = tail_splits(tail_cap);
  cudaError_t e = cudaSuccess;
  const dim3 grid(problems, n_split), block(kTailThreads);
#define XKV_TAIL(DH, NR)                                                                                            \
  do {                                                                                                              \
    e = cudaFuncSetAttribute(tail_partial_kernel<DH, NR>, cudaFuncAttributeMaxDynamicSharedMemorySize,              \
                             (int)tail_smem_bytes<DH, NR>());                                                       \
    if (e == cudaSuccess)                                                                                           \
      e = launch_pdl(tail_partial_kernel<DH, NR>, grid, block, tail_smem_bytes<DH, NR>(), s, dev, l0, q, tail_k,     \
                     tail_v, tail_len, tail_cap, n_split, part);                                                    \
  } while (0)
  if (dev.d_h == 128) {
    if (dev.n_rep <= 4) XKV_TAIL(128, 4); else if (dev.n_rep <= 8) XKV_TAIL(128, 8); else XKV_TAIL(128, 16);
  } else {
    if (dev.n_rep <= 4) XKV_TAIL(64, 4); else if (dev.n_rep <= 8) XKV_TAIL(64, 8); else XKV_TAIL(64, 16);
  }
#undef XKV_TAIL
  count_launch();
  return e;
}

}  // namespace xkv
