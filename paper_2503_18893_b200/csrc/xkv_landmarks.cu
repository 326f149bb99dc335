// Landmark construction at prefill (App. B.1, Algorithm 1): chunk means of the post-RoPE keys and, optionally, the
// minimum within-chunk cosine similarity to the chunk mean, from which the static outlier chunks are taken.
// One pass over the keys (HBM bound: every key row is read once from DRAM, a second time from cache for the
// cosines).  One CTA handles a few consecutive chunks (32 rows) of one (sequence, layer) for all KV heads;
// thread = (KV head, rotary pair).  The rotation angles p * theta_i are formed in fp64 (p reaches 2^24) and their
// cos/sin are shared by the heads through shared memory.
#include <math.h>

#include "xkv_internal.cuh"
#include "xkv_ptx.cuh"

namespace xkv {

namespace {

constexpr int kLmRows = 32;         // key rows per CTA pass (a whole number of chunks when c divides it, else 1 chunk)

__device__ __forceinline__ float bf(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// keys      bf16 [batch][G][T][H_kv*d_h], rows before rotation (rope_base > 0) or already rotated (rope_base <= 0)
// landmarks bf16 [batch][G][H_kv][n_c][d_h]
// min_cos   fp32 [G][batch][H_kv][n_c] or nullptr
// grid = (ceil(n_c / chunks per CTA), G, batch), block = H_kv * d_h / 2 threads (at most 1024).
template <int DH>
__global__ void __launch_bounds__(1024)
landmark_kernel(const __nv_bfloat16* __restrict__ keys, __nv_bfloat16* __restrict__ landmarks, float* __restrict__ min_cos,
                int G, int batch, int T, int H_kv, int c, int n_c, int chunks_per_cta, double rope_base, int use_rope) {
  constexpr int HALF = DH / 2;
  extern __shared__ float2 cs_s[];                       // [rows of one chunk pass][HALF] (cos, sin)
  __shared__ float red_s[2][32];                         // per-warp partial sums of (dot, |k|^2)
  __shared__ double theta_s[HALF];                       // theta_i / pi, theta_i = base^(-2i/d_h)
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = tid / HALF, i = tid % HALF;
  const int l = blockIdx.y, b = blockIdx.z;
  const int d = H_kv * DH;
  const __nv_bfloat16* K = keys + (((size_t)b * G + l) * T) * d + (size_t)g * DH;
  if (use_rope && tid < HALF) theta_s[tid] = pow(rope_base, -(double)tid / (double)HALF) / 3.14159265358979323846;
  __syncthreads();
  constexpr int WPH = HALF / 32;                          // warps per head: 2 (d_h = 128) or 1 (d_h = 64)
  // When all chunks of this CTA fit one table (c <= 32), the cos/sin of their rows are computed once, up front.
  const bool whole = c <= kLmRows;
  const int R0 = blockIdx.x * chunks_per_cta * c;
  if (whole && use_rope) {
    const int nrows = min(chunks_per_cta * c, T - R0);
    for (int t = tid; t < nrows * HALF; t += blockDim.x) {
      const int r = t / HALF, ii = t % HALF;
      double sn, cs;
      sincospi((double)(R0 + r) * theta_s[ii], &sn, &cs);
      cs_s[r * HALF + ii] = make_float2((float)cs, (float)sn);
    }
    __syncthreads();
  }

  for (int jc = 0; jc < chunks_per_cta; ++jc) {
    const int j = blockIdx.x * chunks_per_cta + jc;
    if (j >= n_c) break;                                  // uniform over the CTA
    const int row0 = j * c, rows = min(c, T - row0);
    float m1 = 0.0f, m2 = 0.0f, best = INFINITY;
    // rows of a chunk are processed kLmRows at a time: first the sums, then (if asked) the cosines
    for (int phase = 0; phase < (min_cos ? 2 : 1); ++phase) {
      float s1 = 0.0f, s2 = 0.0f;
      float mn2 = 0.0f;                                   // |mean|^2 of this head (phase 1)
      if (phase == 1) {
        float v = m1 * m1 + m2 * m2;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        __syncthreads();
        if (lane == 0) red_s[0][warp] = v;
        __syncthreads();
        for (int w = 0; w < WPH; ++w) mn2 += red_s[0][g * WPH + w];
      }
      for (int r0 = 0; r0 < rows; r0 += kLmRows) {
        const int nr = min(kLmRows, rows - r0);
        const int toff = whole ? (row0 - R0) : 0;         // first table row of this pass
        if (!whole) __syncthreads();                      // the previous pass is done with cs_s
        if (use_rope && !whole) {
          // cos/sin of (row0 + r0 + r) * theta_i for the rows of this pass: each (r, i) once, shared by the heads
          for (int t = tid; t < nr * HALF; t += blockDim.x) {
            const int r = t / HALF, ii = t % HALF;
            double sn, cs;
            sincospi((double)(row0 + r0 + r) * theta_s[ii], &sn, &cs);   // exact range reduction: the angle reaches 2^24 rad
            cs_s[r * HALF + ii] = make_float2((float)cs, (float)sn);
          }
          __syncthreads();
        }
        for (int rb = 0; rb < nr; rb += 8) {
         // eight rows at a time: their loads are issued together (each thread only reads 4 bytes of a row)
         float xa[8], xb[8];
#pragma unroll
         for (int u = 0; u < 8; ++u) {
           const __nv_bfloat16* kr = K + (size_t)(row0 + r0 + min(rb + u, nr - 1)) * d;
           xa[u] = bf(kr + i); xb[u] = bf(kr + i + HALF);
         }
#pragma unroll
         for (int u = 0; u < 8; ++u) {
          const int r = rb + u;
          if (r >= nr) break;                             // uniform over the CTA
          float x1 = xa[u], x2 = xb[u];
          if (use_rope) {
            const float2 a = cs_s[(toff + r) * HALF + i];
            const float y1 = x1 * a.x - x2 * a.y, y2 = x2 * a.x + x1 * a.y;
            x1 = y1; x2 = y2;
          }
          if (phase == 0) {
            s1 += x1; s2 += x2;
          } else {
            // cosine of this row with the chunk mean: sums over the head's d_h dims
            float dot = x1 * m1 + x2 * m2, nn = x1 * x1 + x2 * x2;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
              dot += __shfl_xor_sync(0xffffffffu, dot, o);
              nn += __shfl_xor_sync(0xffffffffu, nn, o);
            }
            if (WPH > 1) {
              __syncthreads();
              if (lane == 0) { red_s[0][warp] = dot; red_s[1][warp] = nn; }
              __syncthreads();
              dot = 0.0f; nn = 0.0f;
#pragma unroll
              for (int w = 0; w < WPH; ++w) { dot += red_s[0][g * WPH + w]; nn += red_s[1][g * WPH + w]; }
            }
            const float den = sqrtf(nn) * sqrtf(mn2);
            best = fminf(best, den > 0.0f ? dot / den : 0.0f);
          }
         }
        }
      }
      if (phase == 0) {
        const float inv = 1.0f / (float)rows;
        m1 = s1 * inv; m2 = s2 * inv;
        __nv_bfloat16* L = landmarks + ((((size_t)b * G + l) * H_kv + g) * n_c + j) * DH;
        L[i] = __float2bfloat16(m1);
        L[i + HALF] = __float2bfloat16(m2);
      }
    }
    if (min_cos && i == 0) min_cos[(((size_t)l * batch + b) * H_kv + g) * n_c + j] = best;
  }
}

}  // namespace

cudaError_t launch_landmarks(const __nv_bfloat16* keys, __nv_bfloat16* landmarks, float* min_cos, int G, int batch, int T,
                             int H_kv, int d_h, int c, float rope_base, cudaStream_t s) {
  const int n_c = (T + c - 1) / c;
  const int threads = H_kv * d_h / 2;
  const int cpc = c >= kLmRows ? 1 : kLmRows / c;
  const dim3 grid((n_c + cpc - 1) / cpc, G, batch);
  const size_t smem = (size_t)kLmRows * (d_h / 2) * sizeof(float2);
  const int use_rope = rope_base > 0.0f ? 1 : 0;
  if (d_h == 128)
    landmark_kernel<128><<<grid, threads, smem, s>>>(keys, landmarks, min_cos, G, batch, T, H_kv, c, n_c, cpc,
                                                     (double)rope_base, use_rope);
  else
    landmark_kernel<64><<<grid, threads, smem, s>>>(keys, landmarks, min_cos, G, batch, T, H_kv, c, n_c, cpc,
                                                    (double)rope_base, use_rope);
  count_launch();
  return cudaGetLastError();
}

}  // namespace xkv
