// One-time preparation at handle creation: transposed head blocks of B and the rotary tables.
#include "xkv_internal.cuh"

namespace xkv {

// B [batch][G][r][H_kv*d_h]  ->  Bt [batch][G][H_kv][kDP][r], Bt[..][g][j][m] = B[..][m][g*d_h+j]
// (rows j >= d_h are zero).  The head block B_{l,g} of Eq. 2 becomes a K-major operand.
__global__ void repack_b_kernel(const __nv_bfloat16* __restrict__ B, __nv_bfloat16* __restrict__ Bt, int r,
                                int H_kv, int d_h) {
  __shared__ __nv_bfloat16 tile[32][33];
  const int d = H_kv * d_h;
  const size_t blk = blockIdx.z;                       // (batch*G) index
  const int g = blockIdx.y / (kDP / 32);
  const int j0 = (blockIdx.y % (kDP / 32)) * 32;       // row block inside the padded head
  const int m0 = blockIdx.x * 32;
  const __nv_bfloat16* src = B + blk * (size_t)r * d;
  __nv_bfloat16* dst = Bt + (blk * H_kv + g) * (size_t)kDP * r;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int m = m0 + i, j = j0 + threadIdx.x;
    tile[i][threadIdx.x] = (m < r && j < d_h) ? src[(size_t)m * d + g * d_h + j] : __float2bfloat16(0.0f);
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    const int j = j0 + i, m = m0 + threadIdx.x;
    if (m < r) dst[(size_t)j * r + m] = tile[threadIdx.x][i];
  }
}

cudaError_t launch_repack_b(const __nv_bfloat16* B, __nv_bfloat16* Bt, int batch, int G, int r, int H_kv,
                            int d_h, cudaStream_t s) {
  dim3 grid((r + 31) / 32, H_kv * (kDP / 32), batch * G);
  repack_b_kernel<<<grid, dim3(32, 8), 0, s>>>(B, Bt, r, H_kv, d_h);
  count_launch(kFamPrep);
  return cudaGetLastError();
}

// theta_i = base^(-2i/d_h); position p = (p_hi << shift) + p_lo.  hi[p_hi][i] = (cos, sin)((p_hi << shift) * theta_i),
// lo[p_lo][i] = (cos, sin)(p_lo * theta_i), evaluated in fp64 so that combining the two by the angle-addition
// formulas carries fp32 rounding only.  Position-major layout: the d_h/2 entries of one position are contiguous.
__global__ void rope_tables_kernel(float2* hi, float2* lo, int n_hi, int shift, int half, double base) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int n_lo = 1 << shift;
  const long long total = (long long)(n_hi + n_lo) * half;
  if (idx >= total) return;
  const int col = (int)(idx / half);
  const int i = (int)(idx % half);
  const double theta = pow(base, -(double)i / (double)half);
  const double p = col < n_hi ? (double)((long long)col << shift) : (double)(col - n_hi);
  double sn, cs;
  sincos(p * theta, &sn, &cs);
  const float2 v = make_float2((float)cs, (float)sn);
  if (col < n_hi) hi[(size_t)col * half + i] = v; else lo[(size_t)(col - n_hi) * half + i] = v;
}

cudaError_t launch_rope_tables(float2* hi, float2* lo, int n_hi, int rope_shift, int d_h, double base,
                               cudaStream_t s) {
  const int half = d_h / 2;
  const long long total = (long long)(n_hi + (1 << rope_shift)) * half;
  rope_tables_kernel<<<(unsigned)((total + 255) / 256), 256, 0, s>>>(hi, lo, n_hi, rope_shift, half, base);
  count_launch(kFamPrep);
  return cudaGetLastError();
}

}  // namespace xkv
