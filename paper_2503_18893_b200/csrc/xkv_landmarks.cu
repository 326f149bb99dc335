// Landmark construction at prefill (App. B.1, Algorithm 1): chunk means of the post-RoPE keys and, optionally, the
// minimum within-chunk cosine similarity to the chunk mean, from which the static outlier chunks are taken.
// HBM bound: every key row is read once from DRAM (a second time from cache when the cosines are wanted, because
// they need the finished mean).
// One CTA handles up to 32 consecutive rows (whole chunks when c <= 32) of one (sequence, layer) for all KV heads.
// A thread owns 8 rotary pairs of one head (16-byte loads of the two halves of the row) and walks the rows of a
// chunk; the CTA's row groups work on different chunks.  The cos/sin of p * theta_i are formed in fp64 for the
// first row of the CTA (the angle reaches 2^24 rad; sincospi reduces it exactly) and advanced row by row with the
// fp64 rotation by theta_i; all heads share them through shared memory.
#include <math.h>

#include "xkv_internal.cuh"
#include "xkv_ptx.cuh"

namespace xkv {

namespace {

constexpr int kLmRows = 32;         // key rows per table (per CTA pass)
constexpr int kLmThreads = 256;

__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) { f[2 * e] = __uint_as_float(w[e] << 16); f[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u); }
}
__device__ __forceinline__ uint4 pack8(const float (&f)[8]) {
  uint4 v;
  __nv_bfloat162 t;
  t = __floats2bfloat162_rn(f[0], f[1]); v.x = *reinterpret_cast<uint32_t*>(&t);
  t = __floats2bfloat162_rn(f[2], f[3]); v.y = *reinterpret_cast<uint32_t*>(&t);
  t = __floats2bfloat162_rn(f[4], f[5]); v.z = *reinterpret_cast<uint32_t*>(&t);
  t = __floats2bfloat162_rn(f[6], f[7]); v.w = *reinterpret_cast<uint32_t*>(&t);
  return v;
}

// keys      bf16 [batch][G][T][H_kv*d_h], rows before rotation (use_rope) or already rotated
// landmarks bf16 [batch][G][H_kv][n_c][d_h]
// min_cos   fp32 [G][batch][H_kv][n_c] or nullptr
// grid = (ceil(n_c / chunks per CTA), G, batch), block = kLmThreads.  TPR = H_kv * d_h / 16 threads cover one row;
// TPR divides kLmThreads (checked on the host); the 8 or 4 threads of a head are consecutive lanes of one warp.
template <int DH>
__global__ void __launch_bounds__(kLmThreads, 3)
landmark_kernel(const __nv_bfloat16* __restrict__ keys, __nv_bfloat16* __restrict__ landmarks, float* __restrict__ min_cos,
                int G, int batch, int T, int H_kv, int c, int n_c, int chunks_per_cta, double rope_base, int use_rope) {
  constexpr int HALF = DH / 2;
  constexpr int APH = HALF / 8;                          // threads per head: each owns 8 rotary pairs
  __shared__ __align__(16) float2 cs_s[kLmRows * HALF];  // (cos, sin) of (row, pair) for the rows of the current pass
  __shared__ float comb_s[kLmThreads][17];               // long chunks only: partial results of the row groups
  const int tid = threadIdx.x;
  const int TPR = H_kv * APH, RG = kLmThreads / TPR;     // threads per row, row groups
  const int rg = tid / TPR, tr = tid % TPR;
  const int g = tr / APH, a = tr % APH;
  const int l = blockIdx.y, b = blockIdx.z;
  const int d = H_kv * DH;
  const __nv_bfloat16* K = keys + (((size_t)b * G + l) * T) * d + (size_t)g * DH + a * 8;
  const bool whole = c <= kLmRows;                        // all chunks of this CTA share one table
  const int R0 = blockIdx.x * chunks_per_cta * c;

  // cos/sin of rows [first, first + n): thread -> (pair, block of consecutive rows); the block's first row by
  // sincospi, then one fp64 rotation by theta per row
  auto fill_table = [&](int first, int n) {
    constexpr int BLKS = kLmThreads / HALF, RPB = kLmRows / BLKS;   // 4 blocks of 8 rows (d_h = 128), 8 of 4 (d_h = 64)
    const int ii = tid % HALF, r_begin = (tid / HALF) * RPB;
    if (r_begin < n) {
      const double th = pow(rope_base, -(double)ii / (double)HALF);
      double sn, cs, st, ct;
      sincospi((double)(first + r_begin) * (th / 3.14159265358979323846), &sn, &cs);
      sincos(th, &st, &ct);                               // theta <= 1: no range reduction needed
      const int r_end = min(n, r_begin + RPB);
      for (int r = r_begin; r < r_end; ++r) {
        cs_s[r * HALF + ii] = make_float2((float)cs, (float)sn);
        const double c2 = cs * ct - sn * st, s2 = sn * ct + cs * st;
        cs = c2; sn = s2;
      }
    }
  };
  // one row: this thread's 8 pairs -> x1[8] (dims a*8..), x2[8] (dims HALF + a*8..), rotated with table row `trow`
  auto load_row = [&](int row, uint4& u1, uint4& u2) {
    const __nv_bfloat16* kr = K + (size_t)row * d;
    u1 = __ldg(reinterpret_cast<const uint4*>(kr));
    u2 = __ldg(reinterpret_cast<const uint4*>(kr + HALF));
  };
  auto rotate = [&](const uint4& u1, const uint4& u2, int trow, float (&x1)[8], float (&x2)[8]) {
    unpack8(u1, x1); unpack8(u2, x2);
    if (use_rope) {
      const float4* t4 = reinterpret_cast<const float4*>(cs_s + trow * HALF + a * 8);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float4 t = t4[e];                           // (cos, sin) of pairs 2e and 2e+1
        const float y1 = x1[2 * e] * t.x - x2[2 * e] * t.y, y2 = x2[2 * e] * t.x + x1[2 * e] * t.y;
        const float z1 = x1[2 * e + 1] * t.z - x2[2 * e + 1] * t.w, z2 = x2[2 * e + 1] * t.z + x1[2 * e + 1] * t.w;
        x1[2 * e] = y1; x2[2 * e] = y2; x1[2 * e + 1] = z1; x2[2 * e + 1] = z2;
      }
    }
  };
  // sum over the APH threads of a head (consecutive lanes)
  // (only those lanes take part: the row groups of a warp may be in different chunks)
  const uint32_t hmask = ((1u << APH) - 1u) << ((tid & 31) & ~(APH - 1));
  auto head_sum = [&](float v) {
#pragma unroll
    for (int o = 1; o < APH; o <<= 1) v += __shfl_xor_sync(hmask, v, o);
    return v;
  };
  auto cosine = [&](const float (&x1)[8], const float (&x2)[8], const float (&m1)[8], const float (&m2)[8], float mn2) {
    float dot = 0.0f, nn = 0.0f;
#pragma unroll
    for (int e = 0; e < 8; ++e) { dot += x1[e] * m1[e] + x2[e] * m2[e]; nn += x1[e] * x1[e] + x2[e] * x2[e]; }
    dot = head_sum(dot); nn = head_sum(nn);
    const float den = sqrtf(nn) * sqrtf(mn2);
    return den > 0.0f ? dot / den : 0.0f;
  };

  if (whole) {
    if (use_rope) {
      fill_table(R0, min(chunks_per_cta * c, T - R0));
      __syncthreads();
    }
    // ---- chunks of at most 32 rows: row group rg takes chunks rg, rg + RG, ... of this CTA
    for (int jc = rg; jc < chunks_per_cta; jc += RG) {
      const int j = blockIdx.x * chunks_per_cta + jc;
      if (j >= n_c) break;
      const int row0 = j * c, rows = min(c, T - row0);
      float m1[8], m2[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) { m1[e] = 0.0f; m2[e] = 0.0f; }
      for (int rb = 0; rb < rows; rb += 4) {              // four rows' loads in flight
        uint4 u1[4], u2[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) load_row(row0 + min(rb + u, rows - 1), u1[u], u2[u]);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (rb + u < rows) {
            float x1[8], x2[8];
            rotate(u1[u], u2[u], row0 - R0 + rb + u, x1, x2);
#pragma unroll
            for (int e = 0; e < 8; ++e) { m1[e] += x1[e]; m2[e] += x2[e]; }
          }
        }
      }
      const float inv = 1.0f / (float)rows;
#pragma unroll
      for (int e = 0; e < 8; ++e) { m1[e] *= inv; m2[e] *= inv; }
      __nv_bfloat16* L = landmarks + ((((size_t)b * G + l) * H_kv + g) * n_c + j) * DH + a * 8;
      *reinterpret_cast<uint4*>(L) = pack8(m1);
      *reinterpret_cast<uint4*>(L + HALF) = pack8(m2);
      if (min_cos) {
        float mn2 = 0.0f;
#pragma unroll
        for (int e = 0; e < 8; ++e) mn2 += m1[e] * m1[e] + m2[e] * m2[e];
        mn2 = head_sum(mn2);
        float best = INFINITY;
        for (int rb = 0; rb < rows; rb += 4) {
          uint4 u1[4], u2[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) load_row(row0 + min(rb + u, rows - 1), u1[u], u2[u]);
#pragma unroll
          for (int u = 0; u < 4; ++u) {                    // a repeated last row changes no minimum
            float x1[8], x2[8];
            rotate(u1[u], u2[u], row0 - R0 + min(rb + u, rows - 1), x1, x2);
            best = fminf(best, cosine(x1, x2, m1, m2, mn2));
          }
        }
        if (a == 0) min_cos[(((size_t)l * batch + b) * H_kv + g) * n_c + j] = best;
      }
    }
    return;
  }

  // ---- a chunk longer than 32 rows: one chunk per CTA, passes of 32 rows, the row groups split the rows of a pass
  const int j = blockIdx.x;
  const int row0 = j * c, rows = min(c, T - row0);
  float m1[8], m2[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) { m1[e] = 0.0f; m2[e] = 0.0f; }
  float mn2 = 0.0f, best = INFINITY;
  for (int phase = 0; phase < (min_cos ? 2 : 1); ++phase) {
    for (int r0 = 0; r0 < rows; r0 += kLmRows) {
      const int nr = min(kLmRows, rows - r0);
      __syncthreads();                                    // the previous pass is done with the table
      if (use_rope) fill_table(row0 + r0, nr);
      __syncthreads();
      for (int r = rg; r < nr; r += RG) {
        uint4 u1, u2;
        load_row(row0 + r0 + r, u1, u2);
        float x1[8], x2[8];
        rotate(u1, u2, r, x1, x2);
        if (phase == 0) {
#pragma unroll
          for (int e = 0; e < 8; ++e) { m1[e] += x1[e]; m2[e] += x2[e]; }
        } else {
          best = fminf(best, cosine(x1, x2, m1, m2, mn2));
        }
      }
    }
    // combine the row groups: sums (phase 0) or minima (phase 1) of the same (head, pair group)
    __syncthreads();
    if (phase == 0) {
#pragma unroll
      for (int e = 0; e < 8; ++e) { comb_s[tid][e] = m1[e]; comb_s[tid][8 + e] = m2[e]; }
      __syncthreads();
#pragma unroll
      for (int e = 0; e < 8; ++e) { m1[e] = 0.0f; m2[e] = 0.0f; }
      for (int q = 0; q < RG; ++q) {
#pragma unroll
        for (int e = 0; e < 8; ++e) { m1[e] += comb_s[q * TPR + tr][e]; m2[e] += comb_s[q * TPR + tr][8 + e]; }
      }
      const float inv = 1.0f / (float)rows;
#pragma unroll
      for (int e = 0; e < 8; ++e) { m1[e] *= inv; m2[e] *= inv; }
      if (rg == 0) {
        __nv_bfloat16* L = landmarks + ((((size_t)b * G + l) * H_kv + g) * n_c + j) * DH + a * 8;
        *reinterpret_cast<uint4*>(L) = pack8(m1);
        *reinterpret_cast<uint4*>(L + HALF) = pack8(m2);
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) mn2 += m1[e] * m1[e] + m2[e] * m2[e];
      mn2 = head_sum(mn2);
    } else {
      comb_s[tid][16] = best;
      __syncthreads();
      for (int q = 0; q < RG; ++q) best = fminf(best, comb_s[q * TPR + tr][16]);
      if (rg == 0 && a == 0) min_cos[(((size_t)l * batch + b) * H_kv + g) * n_c + j] = best;
    }
  }
}

}  // namespace

cudaError_t launch_landmarks(const __nv_bfloat16* keys, __nv_bfloat16* landmarks, float* min_cos, int G, int batch, int T,
                             int H_kv, int d_h, int c, float rope_base, cudaStream_t s) {
  const int n_c = (T + c - 1) / c;
  const int tpr = H_kv * d_h / 16;                        // threads per key row
  if (tpr > kLmThreads || kLmThreads % tpr != 0) return cudaErrorInvalidValue;
  const int cpc = c >= kLmRows ? 1 : kLmRows / c;
  const dim3 grid((n_c + cpc - 1) / cpc, G, batch);
  const int use_rope = rope_base > 0.0f ? 1 : 0;
  if (d_h == 128)
    landmark_kernel<128><<<grid, kLmThreads, 0, s>>>(keys, landmarks, min_cos, G, batch, T, H_kv, c, n_c, cpc,
                                                     (double)rope_base, use_rope);
  else
    landmark_kernel<64><<<grid, kLmThreads, 0, s>>>(keys, landmarks, min_cos, G, batch, T, H_kv, c, n_c, cpc,
                                                    (double)rope_base, use_rope);
  count_launch(kFamLandmarks);
  return cudaGetLastError();
}

}  // namespace xkv
