// Cross-layer factorisation on the GPU (Sec. 3.1, Eq. 1; App. "Custom SVD Kernel": a randomised SVD whose power
// iterations are 16-bit tensor-core matrix products and whose orthogonalisation is a shifted Cholesky QR).
//
// X = [X_l0 ... X_l0+G-1] (T x N, N = G d, bf16) is tall, so the iteration runs on the right side.  With l = r + p:
//   Z (N x l) <- the random test matrix
//   repeat q + 1 times:   Y^T = Z^T X^T   (l x T, bf16)          tensor core
//                         U   = X^T Y     (N x l, fp32)          tensor core
//                         Z   = U R^-1,  R^T R = U^T U + shift I (shifted Cholesky QR in fp64: two passes inside the
//                               iteration, five for the last iterate, which has to be orthonormal)
//   Rayleigh-Ritz:        W^T = Z^T X^T,  U' = X^T W,  M = Z^T U' (= Z^T X^T X Z, l x l),  M = P Lambda P^T (Jacobi)
//   V = Z P_r (N x r);    B_l = rows of V^T (bf16);   A = X V_bf16 (T x r, tensor core);   sigma = sqrt(Lambda).
// A = U Sigma and B = V^T of the truncated SVD of X, up to the accuracy of the subspace (checked against the exact
// optimum sum_{i>r} sigma_i^2, never factor by factor: signs and degenerate subspaces are not unique).
//
// One tensor-core kernel serves the three tall products.  It computes C (M x N) = A B^T for A given as [K][M]
// row-major (an MN-major operand: the M index is contiguous) and B as [N][K] row-major (K-major), the two operand
// forms the fused decode kernel already uses, so no matrix is ever transposed in memory:
//   Y^T = Z-as-A (K = N_x)  x  X-as-B;     U = X-as-A (K = T)  x  Y^T-as-B;     A^T = V-as-A  x  X-as-B (stored transposed).
#include <cuda.h>
#include <math.h>

#include "xkv_internal.cuh"
#include "xkv_ptx.cuh"

namespace xkv {

namespace {

using namespace ptx;

constexpr int kGemmThreads = 192;                 // warps 0-3 epilogue, 4 TMA producer, 5 MMA issue
// One stage of the operand ring: A, two slabs of [64 k][64 m] (8 KB each), and B, [BN n][64 k] (BN * 128 bytes).
// Tiles are 128 x BN with BN = 256, 192 or 128: an N = 128 step reads 8 KB of operands per 64 cycles, all the shared-
// memory pipe gives, an N = 256 step 12 KB per 128 cycles.  Four stages for the wide tiles (one CTA per SM), three
// for BN = 128 (two CTAs per SM, so that one's epilogue hides behind the other's products).
template <int BN> constexpr int gemm_stage_bytes() { return 16384 + BN * 128; }
template <int BN> constexpr int gemm_stages() { return BN == 128 ? 3 : 4; }
constexpr int kGemmMaxStages = 4;
constexpr uint32_t kGemmWaitLimit = 1u << 24;

__device__ __forceinline__ bool gemm_wait(uint32_t bar, uint32_t parity) {
  for (uint32_t i = 0; i < kGemmWaitLimit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
  }
  return false;
}

// C[m][n] = sum_k A[k][m] B[n][k].  grid = (ceil(N/BN), ceil(M/128)).  TRANS: store C^T (out[n][m]).
// Out-of-range rows and columns of the operands are zero-filled by the copy engine; stores are guarded.
template <bool TRANS, int BN>
__global__ void __launch_bounds__(kGemmThreads)
clf_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, int M, int N, int K,
                float* __restrict__ Cf, __nv_bfloat16* __restrict__ Cb, long long ldc, unsigned int* __restrict__ flags) {
  extern __shared__ uint8_t gemm_smem[];
  constexpr int kGemmStages = gemm_stages<BN>(), kGemmStageBytes = gemm_stage_bytes<BN>();
  constexpr uint32_t kCols = BN <= 128 ? 128u : 256u;      // tensor-memory columns (a power of two)
  __shared__ __align__(8) uint64_t bars[2 * kGemmMaxStages + 1];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_s;
  const uint32_t base = (smem_u32(gemm_smem) + 1023u) & ~1023u;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n0 = blockIdx.x * BN, m0 = blockIdx.y * 128;
  const int KB = (K + 63) / 64;
  const uint32_t bar0 = smem_u32(bars);
  auto FULL = [&](int s) { return bar0 + 8u * (uint32_t)s; };
  auto EMPTY = [&](int s) { return bar0 + 8u * (uint32_t)(kGemmStages + s); };
  const uint32_t ACC = bar0 + 8u * (uint32_t)(2 * kGemmStages);
  if (tid == 0) {
    for (int s = 0; s < kGemmStages; ++s) { mbar_init(FULL(s), 1); mbar_init(EMPTY(s), 1); }
    mbar_init(ACC, 1);
    abort_s = 0;
    fence_mbar_init();
  }
  if (warp == 5) {
    tmem_alloc(smem_u32(&tmem_slot), kCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_slot;
  bool ok = true;
  if (warp == 4) {
    if (lane == 0) {
      for (int kb = 0; kb < KB; ++kb) {
        const int s = kb % kGemmStages;
        if (kb >= kGemmStages && !gemm_wait(EMPTY(s), (uint32_t)((kb / kGemmStages - 1) & 1))) { ok = false; break; }
        const uint32_t st = base + (uint32_t)s * kGemmStageBytes;
        mbar_expect_tx(FULL(s), kGemmStageBytes);
        tma_load_2d(st, &map_a, m0, kb * 64, FULL(s));                 // A: columns m0..m0+63, rows (k) kb*64..+63
        tma_load_2d(st + 8192, &map_a, m0 + 64, kb * 64, FULL(s));     //    columns m0+64..m0+127
        tma_load_2d(st + 16384, &map_b, kb * 64, n0, FULL(s));         // B: columns (k) kb*64..+63, rows n0..n0+BN-1
      }
    }
  } else if (warp == 5) {
    if (lane == 0) {
      const uint64_t desc_hi = smem_desc_sw128(0, 0) & 0xFFFFFFFF00000000ull;
      constexpr uint32_t idesc = idesc_bf16_f32(128, BN) | (1u << 15);    // A is read along its rows (MN-major)
      for (int kb = 0; kb < KB; ++kb) {
        const int s = kb % kGemmStages;
        if (!gemm_wait(FULL(s), (uint32_t)((kb / kGemmStages) & 1))) { ok = false; break; }
        tc_fence_after();
        const uint32_t st = base + (uint32_t)s * kGemmStageBytes;
        // A: two 64-column slabs 8192 bytes apart, 8-row groups (along k) 1024 bytes apart; 16 k-rows per step
        const uint32_t a_lo = ((uint32_t)((st & 0x3FFFFu) >> 4)) | ((uint32_t)(8192 >> 4) << 16);
        const uint32_t b_lo = (uint32_t)(smem_desc_sw128(st + 16384, 0) & 0xFFFFFFFFull);
#pragma unroll
        for (int kk = 0; kk < 4; ++kk)
          tc_mma_bf16(tmem, desc_hi | (a_lo + (uint32_t)kk * (2048u >> 4)), desc_hi | (b_lo + 2u * (uint32_t)kk), idesc,
                      (kb | kk) ? 1u : 0u);
        tc_commit(EMPTY(s));
      }
      tc_commit(ACC);
    }
  }
  if (warp >= 4) {                  // a producer or issuer that gave up tells the epilogue not to wait for ever
    if (!ok && lane == 0) { abort_s = 1; atomicOr(flags, XKV_FLAG_TIMEOUT); }
  } else {
    // ---- epilogue: thread = accumulator lane = row m0 + tid
    bool done = false;
    for (uint32_t i = 0; i < kGemmWaitLimit && !done; ++i) {
      done = mbar_try_wait(ACC, 0);
      if (!done && (i & 1023u) == 1023u && *(volatile int*)&abort_s) break;
    }
    if (done) {
      tc_fence_after();
      const int m = m0 + tid;
      const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
#pragma unroll 1
      for (int cb = 0; cb < BN / 32; ++cb) {
        float v[32];
        tmem_ld32(tmem + lane_base + (uint32_t)(cb * 32), v);
        tc_wait_ld();
        if (m < M) {
          const int nb = n0 + cb * 32;
          if (!TRANS && nb + 32 <= N && (ldc & 7) == 0) {
            // a whole run of 32 columns of one row: 16-byte stores (the row pitch keeps them aligned)
            const long long at = (long long)m * ldc + nb;
            if (Cf) {
#pragma unroll
              for (int i = 0; i < 32; i += 4) *reinterpret_cast<float4*>(Cf + at + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
            }
            if (Cb) {
#pragma unroll
              for (int i = 0; i < 32; i += 8) {
                __nv_bfloat162 h0 = __floats2bfloat162_rn(v[i], v[i + 1]), h1 = __floats2bfloat162_rn(v[i + 2], v[i + 3]);
                __nv_bfloat162 h2 = __floats2bfloat162_rn(v[i + 4], v[i + 5]), h3 = __floats2bfloat162_rn(v[i + 6], v[i + 7]);
                uint4 u;
                u.x = *reinterpret_cast<uint32_t*>(&h0); u.y = *reinterpret_cast<uint32_t*>(&h1);
                u.z = *reinterpret_cast<uint32_t*>(&h2); u.w = *reinterpret_cast<uint32_t*>(&h3);
                *reinterpret_cast<uint4*>(Cb + at + i) = u;
              }
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const int n = nb + i;
              if (n < N) {
                const long long at = TRANS ? (long long)n * ldc + m : (long long)m * ldc + n;
                if (Cf) Cf[at] = v[i];
                if (Cb) Cb[at] = __float2bfloat16(v[i]);
              }
            }
          }
        }
      }
    } else if (tid == 0) {
      atomicOr(flags, XKV_FLAG_TIMEOUT);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    tmem_dealloc(tmem, kCols);
  }
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// The small matrices (l x l, N x l) in fp32 on the ordinary cores.
namespace {

// C (m x n, ldc) = op(A) B with B (k x n, ldb) row-major and op(A) = A^T for A (k x m, lda) if TA, else A (m x k, lda).
// 64 x 64 tiles, 256 threads, 4 x 4 outputs per thread.
// TO = double accumulates in double.
template <bool TA, typename TO>
__global__ void __launch_bounds__(256)
sgemm_small_kernel(const float* __restrict__ A, const float* __restrict__ B, TO* __restrict__ C, int m, int n, int k,
                   int lda, int ldb, int ldc) {
  __shared__ float As[16][64 + 4], Bs[16][64 + 4];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  TO acc[4][4] = {};
  for (int k0 = 0; k0 < k; k0 += 16) {
    for (int i = tid; i < 16 * 64; i += 256) {
      const int kk = TA ? i / 64 : i % 16, mm = TA ? i % 64 : i / 16;
      const int gk = k0 + kk, gm = m0 + mm;
      As[kk][mm] = (gk < k && gm < m) ? (TA ? A[(size_t)gk * lda + gm] : A[(size_t)gm * lda + gk]) : 0.0f;
      const int bk = i / 64, bn = i % 64;
      Bs[bk][bn] = (k0 + bk < k && n0 + bn < n) ? B[(size_t)(k0 + bk) * ldb + n0 + bn] : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[kk][ty * 4 + i]; b[i] = Bs[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] += (TO)a[i] * (TO)b[j];
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gm = m0 + ty * 4 + i, gn = n0 + tx * 4 + j;
      if (gm < m && gn < n) C[(size_t)gm * ldc + gn] = acc[i][j];
    }
}

// C (m x n, fp64 or rounded to fp32) = A^T B for fp32 A (k x m) and B (k x n) on the fp64 tensor-core path (mma.sync m8n8k4): the Gram
// matrices of the Cholesky QR, accumulated in fp64 because their condition number is the square of the iterate's.
// (A scalar fp64 kernel with 4 x 4 outputs per thread spent 0.79 ms on a 576 x 576 x 4096 product, this one 0.33 ms.)  64 x 64 tiles, 8 warps of 16 x 32, chunks of 32 rows
// widened to fp64 on their way into shared memory; m, n multiples of 64, k a multiple of 32.
constexpr int kDgemmLd = 68;                         // doubles per staged row: 4 mod 16, so fragment loads are conflict free
__device__ __forceinline__ void dmma_8x8x4(double (&d)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
               : "+d"(d[0]), "+d"(d[1]) : "d"(a), "d"(b));
}
template <typename TO>
__global__ void __launch_bounds__(256)
dgemm_tn_mma_kernel(const float* __restrict__ A, const float* __restrict__ B, TO* __restrict__ C, int k, int lda,
                    int ldb, int ldc) {
  __shared__ double As[32][kDgemmLd], Bs[32][kDgemmLd];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wm = (warp & 3) * 16, wn = (warp >> 2) * 32;
  const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
  const int lr = tid >> 4, lc = (tid & 15) * 4;       // this thread's piece of a staged chunk: rows lr, lr + 16; 4 columns
  double acc[2][4][2];
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) { acc[i][j][0] = 0.0; acc[i][j][1] = 0.0; }
  float4 pa[2], pb[2];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      pa[h] = *reinterpret_cast<const float4*>(A + (size_t)(k0 + lr + 16 * h) * lda + m0 + lc);
      pb[h] = *reinterpret_cast<const float4*>(B + (size_t)(k0 + lr + 16 * h) * ldb + n0 + lc);
    }
  };
  fetch(0);
  for (int k0 = 0; k0 < k; k0 += 32) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      double* da = &As[lr + 16 * h][lc];
      double* db = &Bs[lr + 16 * h][lc];
      da[0] = (double)pa[h].x; da[1] = (double)pa[h].y; da[2] = (double)pa[h].z; da[3] = (double)pa[h].w;
      db[0] = (double)pb[h].x; db[1] = (double)pb[h].y; db[2] = (double)pb[h].z; db[3] = (double)pb[h].w;
    }
    __syncthreads();
    if (k0 + 32 < k) fetch(k0 + 32);                  // the next chunk travels while this one is multiplied
#pragma unroll
    for (int kk = 0; kk < 32; kk += 4) {
      double a[2], b[4];
#pragma unroll
      for (int i = 0; i < 2; ++i) a[i] = As[kk + (lane & 3)][wm + 8 * i + (lane >> 2)];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[kk + (lane & 3)][wn + 8 * j + (lane >> 2)];
#pragma unroll
      for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) dmma_8x8x4(acc[i][j], a[i], b[j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      TO* dst = C + (size_t)(m0 + wm + 8 * i + (lane >> 2)) * ldc + n0 + wn + 8 * j + 2 * (lane & 3);
      dst[0] = (TO)acc[i][j][0];
      dst[1] = (TO)acc[i][j][1];
    }
}

// Blocked Cholesky factorisation (fp64) of the symmetric l x l matrix G + shift_rel * max_diag(G) * I, lower factor in
// place, in panels of 32 columns: factor the diagonal block, solve the panel below it, update the trailing matrix.
constexpr int kCholNb = 32;

__global__ void __launch_bounds__(1024)
chol_shift_kernel(double* __restrict__ G, int l, double shift_rel) {
  __shared__ double red[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  double mx = 0.0;
  for (int i = tid; i < l; i += 1024) mx = fmax(mx, G[(size_t)i * l + i]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if (lane == 0) red[warp] = mx;
  __syncthreads();
  mx = red[lane];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  for (int i = tid; i < l; i += 1024) G[(size_t)i * l + i] += shift_rel * mx;
}

// Diagonal block [kb, kb+nb): unblocked factorisation by one warp.  A pivot that is not positive (breakdown) is
// replaced by a tiny one and reported in flags.
__global__ void __launch_bounds__(kCholNb)
chol_diag_kernel(double* __restrict__ G, int l, int kb, int nb, unsigned int* __restrict__ flags) {
  // One warp, lane i holds row i of the block in registers.  Step c: lane c takes the root of its diagonal entry, every
  // lane below scales its entry of column c, the column goes through shared memory, and every lane takes it out of
  // the rest of its row (independent multiply-adds).  Roots and quotients go through rsqrt: a step is a chain of
  // dependent fp64 latencies, and sqrt and division are the longest of them.
  __shared__ double col[kCholNb];
  __shared__ double piv;
  const int i = threadIdx.x;
  double a[kCholNb];
#pragma unroll
  for (int j = 0; j < kCholNb; ++j) a[j] = (i < nb && j < nb && j <= i) ? G[(size_t)(kb + i) * l + kb + j] : (i == j ? 1.0 : 0.0);
#pragma unroll
  for (int c = 0; c < kCholNb; ++c) {
    if (i == c) {
      double d = a[c];
      if (!(d > 0.0)) { atomicOr(flags, XKV_FLAG_CLF_BREAKDOWN); d = 1e-300; }
      const double y = rsqrt(d);
      a[c] = d * y;                                   // sqrt(d)
      piv = y;
    }
    __syncwarp();
    const double y = piv;
    if (i > c) a[c] *= y;
    col[i] = a[c];
    __syncwarp();
#pragma unroll
    for (int j = 0; j < kCholNb; ++j) {
      if (j > c && j <= i) a[j] -= a[c] * col[j];
    }
    __syncwarp();
  }
#pragma unroll
  for (int j = 0; j < kCholNb; ++j) if (i < nb && j < nb && j <= i) G[(size_t)(kb + i) * l + kb + j] = a[j];
}

constexpr int kCholPanelThreads = 128;             // (one warp per CTA, to spread the rows over more SMs: 24 us instead of 16)
// Panel below the diagonal block: row i of L21 solves x L11^T = A21[i] (one thread per row).
__global__ void __launch_bounds__(kCholPanelThreads)
chol_panel_kernel(double* __restrict__ G, int l, int kb, int nb) {
  __shared__ double L11[kCholNb][kCholNb + 1];
  __shared__ double dinv[kCholNb];
  for (int e = threadIdx.x; e < kCholNb * kCholNb; e += kCholPanelThreads) {
    const int r = e / kCholNb, c = e % kCholNb;
    const double v = (r < nb && c <= r) ? G[(size_t)(kb + r) * l + kb + c] : 0.0;
    L11[r][c] = v;
    if (r == c) dinv[r] = r < nb ? 1.0 / v : 0.0;
  }
  __syncthreads();
  const int i = kb + nb + blockIdx.x * kCholPanelThreads + threadIdx.x;
  if (i >= l) return;
  // column sweep: once x_c is known it is taken out of every later entry, so the multiply-adds of a step are
  // independent of one another (a dot product per entry is one long dependent chain on the fp64 pipe)
  double x[kCholNb];
  double* row = G + (size_t)i * l + kb;
#pragma unroll
  for (int c = 0; c < kCholNb; ++c) x[c] = c < nb ? row[c] : 0.0;
#pragma unroll
  for (int c = 0; c < kCholNb; ++c) {
    if (c < nb) {
      x[c] *= dinv[c];
#pragma unroll
      for (int t = 0; t < kCholNb; ++t) if (t > c) x[t] -= x[c] * L11[t][c];
    }
  }
#pragma unroll
  for (int c = 0; c < kCholNb; ++c) if (c < nb) row[c] = x[c];
}

// Trailing update of the lower triangle: G[i][k] -= sum_t L21[i][t] L21[k][t]; one 32 x 32 tile per CTA.
__global__ void __launch_bounds__(1024)
chol_update_kernel(double* __restrict__ G, int l, int kb, int nb) {
  if (blockIdx.x > blockIdx.y) return;                                 // upper triangle: not needed
  __shared__ double Li[kCholNb][kCholNb + 1], Lk[kCholNb][kCholNb + 1];
  const int t0 = kb + nb;
  const int i = t0 + blockIdx.y * kCholNb + threadIdx.y, k = t0 + blockIdx.x * kCholNb + threadIdx.x;
  const int ii = t0 + blockIdx.y * kCholNb + threadIdx.x;              // the row this thread loads for the tiles
  const int kk = t0 + blockIdx.x * kCholNb + threadIdx.x;
  // thread (y, x) loads element (row x of the tile, column y of the panel)
  Li[threadIdx.x][threadIdx.y] = (ii < l && threadIdx.y < nb) ? G[(size_t)ii * l + kb + threadIdx.y] : 0.0;
  Lk[threadIdx.x][threadIdx.y] = (kk < l && threadIdx.y < nb) ? G[(size_t)kk * l + kb + threadIdx.y] : 0.0;
  __syncthreads();
  if (i < l && k <= i) {
    double acc = 0.0;
#pragma unroll
    for (int t = 0; t < kCholNb; ++t) acc += Li[threadIdx.y][t] * Lk[threadIdx.x][t];
    G[(size_t)i * l + k] -= acc;
  }
}

// Z (n x l) = U L^-T for the lower factor L: row by row, z_j = (u_j - sum_{i<j} z_i L[j][i]) / L[j][j] (fp64).  One warp
// per row; the row lives in shared memory.  Also writes the bf16 copy the tensor-core products read.
constexpr int kSolveWarps = 4;
__global__ void __launch_bounds__(kSolveWarps * 32)
trsolve_rows_kernel(const float* __restrict__ U, const double* __restrict__ L, float* __restrict__ Z,
                    __nv_bfloat16* __restrict__ Zb, int n, int l) {
  extern __shared__ double zrow[];                   // [kSolveWarps][l]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int row = blockIdx.x * kSolveWarps + warp;
  if (row >= n) return;
  double* z = zrow + (size_t)warp * l;
  for (int j = lane; j < l; j += 32) z[j] = (double)U[(size_t)row * l + j];
  __syncwarp();
  for (int j = 0; j < l; ++j) {
    const double* Lj = L + (size_t)j * l;
    double s = 0.0;
    for (int i = lane; i < j; i += 32) s += z[i] * Lj[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) z[j] = (z[j] - s) / Lj[j];
    __syncwarp();
  }
  for (int j = lane; j < l; j += 32) {
    Z[(size_t)row * l + j] = (float)z[j];
    if (Zb) Zb[(size_t)row * l + j] = __float2bfloat16((float)z[j]);
  }
}

// ---- the triangular solve Z = U L^-T in 64-column blocks on the fp64 tensor-core path ----
// Z[:, J] = (U[:, J] - sum_{I<J} Z[:, I] L[J, I]^T) inv(L[J, J])^T.  The inverses of the 64 x 64 diagonal blocks come
// from a small kernel (one thread per column of the inverse, forward substitution); the solve keeps 32 rows of Z in
// fp64 in shared memory per CTA and streams the blocks of L through a 64 x 64 staging tile.
constexpr int kTriBlock = 64;
__global__ void __launch_bounds__(kTriBlock)
tri_inv_diag_kernel(const double* __restrict__ L, int l, double* __restrict__ Xinv) {
  __shared__ double Xs[kTriBlock][kTriBlock + 1];
  const int c = threadIdx.x, jb = blockIdx.x * kTriBlock;
  const double* Lb = L + (size_t)jb * l + jb;
  for (int j = 0; j < kTriBlock; ++j) {
    double x = 0.0;
    if (j >= c) {
      double s0 = (j == c) ? 1.0 : 0.0, s1 = 0.0;
      const double* Lj = Lb + (size_t)j * l;
      int i = c;
      for (; i + 1 < j; i += 2) { s0 -= Lj[i] * Xs[i][c]; s1 -= Lj[i + 1] * Xs[i + 1][c]; }
      if (i < j) s0 -= Lj[i] * Xs[i][c];
      x = (s0 + s1) / Lj[j];
    }
    Xs[j][c] = x;                                    // a thread only ever reads its own column
  }
  __syncthreads();
  double* out = Xinv + (size_t)blockIdx.x * kTriBlock * kTriBlock;
  for (int e = c; e < kTriBlock * kTriBlock; e += kTriBlock) out[e] = Xs[e / kTriBlock][e % kTriBlock];
}

constexpr int kTriRows = 32;                         // rows of Z per CTA
__global__ void __launch_bounds__(256)
trsolve_mma_kernel(const float* __restrict__ U, const double* __restrict__ L, const double* __restrict__ Xinv,
                   float* __restrict__ Z, __nv_bfloat16* __restrict__ Zb, int n, int l) {
  extern __shared__ double tri_s[];
  const int ldz = l + 4;                             // 4 mod 16 doubles: fragment loads are conflict free
  double* Zs = tri_s;                                // [kTriRows][ldz]
  double* Ls = tri_s + (size_t)kTriRows * ldz;       // [64][kDgemmLd]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wm = (warp & 1) * 16, wn = (warp >> 1) * 16;
  const int row0 = blockIdx.x * kTriRows;
  const int fr = lane >> 2, fc = lane & 3;
  auto stage = [&](const double* src, int ld) {      // 64 x 64 block, row-major
    for (int e = tid; e < kTriBlock * kTriBlock; e += 256) Ls[(e >> 6) * kDgemmLd + (e & 63)] = src[(size_t)(e >> 6) * ld + (e & 63)];
  };
  const int nb = l / kTriBlock;
  for (int J = 0; J < nb; ++J) {
    double acc[2][2][2];
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int r = row0 + wm + 8 * i + fr;
        const float2 u = r < n ? *reinterpret_cast<const float2*>(U + (size_t)r * l + J * kTriBlock + wn + 8 * j + 2 * fc)
                               : make_float2(0.0f, 0.0f);
        acc[i][j][0] = (double)u.x;
        acc[i][j][1] = (double)u.y;
      }
    for (int I = 0; I < J; ++I) {
      __syncthreads();                               // the staging tile and the last block of Z are free / written
      stage(L + (size_t)J * kTriBlock * l + (size_t)I * kTriBlock, l);
      __syncthreads();
#pragma unroll 4
      for (int kk = 0; kk < kTriBlock; kk += 4) {
        double a[2], b[2];
#pragma unroll
        for (int i = 0; i < 2; ++i) a[i] = -Zs[(size_t)(wm + 8 * i + fr) * ldz + I * kTriBlock + kk + fc];
#pragma unroll
        for (int j = 0; j < 2; ++j) b[j] = Ls[(wn + 8 * j + fr) * kDgemmLd + kk + fc];
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
          for (int j = 0; j < 2; ++j) dmma_8x8x4(acc[i][j], a[i], b[j]);
      }
    }
    __syncthreads();
    // the right-hand side of the diagonal step goes through the block's own columns of Zs
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        double* d = Zs + (size_t)(wm + 8 * i + fr) * ldz + J * kTriBlock + wn + 8 * j + 2 * fc;
        d[0] = acc[i][j][0];
        d[1] = acc[i][j][1];
        acc[i][j][0] = 0.0;
        acc[i][j][1] = 0.0;
      }
    stage(Xinv + (size_t)J * kTriBlock * kTriBlock, kTriBlock);
    __syncthreads();
#pragma unroll 4
    for (int kk = 0; kk < kTriBlock; kk += 4) {
      double a[2], b[2];
#pragma unroll
      for (int i = 0; i < 2; ++i) a[i] = Zs[(size_t)(wm + 8 * i + fr) * ldz + J * kTriBlock + kk + fc];
#pragma unroll
      for (int j = 0; j < 2; ++j) b[j] = Ls[(wn + 8 * j + fr) * kDgemmLd + kk + fc];
#pragma unroll
      for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int j = 0; j < 2; ++j) dmma_8x8x4(acc[i][j], a[i], b[j]);
    }
    __syncthreads();                                 // every warp has read the right-hand side
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int rl = wm + 8 * i + fr, col = J * kTriBlock + wn + 8 * j + 2 * fc;
        double* d = Zs + (size_t)rl * ldz + col;
        d[0] = acc[i][j][0];
        d[1] = acc[i][j][1];
        const int r = row0 + rl;
        if (r < n) {
          const float z0 = (float)acc[i][j][0], z1 = (float)acc[i][j][1];
          *reinterpret_cast<float2*>(Z + (size_t)r * l + col) = make_float2(z0, z1);
          if (Zb) *reinterpret_cast<__nv_bfloat162*>(Zb + (size_t)r * l + col) = __floats2bfloat162_rn(z0, z1);
        }
      }
  }
}

}  // namespace

namespace {

// Eigen-decomposition of the symmetric l x l matrix M by cyclic Jacobi rotations in the round-robin (tournament)
// order: every round rotates l/2 disjoint index pairs at once.  A check per sweep ends the sweeps once the
// off-diagonal weight is below kJacobiTol.  On return the eigenvalues are on the diagonal of M, the
// eigenvectors the columns of P.
constexpr int kJacobiMaxPairs = 1024;
constexpr int kJacobiSweeps = 12;
// The sweeps end when the off-diagonal weight (sum of squares) is below this fraction of the total.  The
// eigenvectors are stored as bf16 (relative rounding 2^-9); an off-diagonal residue of 1e-4 in relative norm is
// twenty times below that, and the convergence is quadratic (measured per sweep on a 576 x 576 Rayleigh-Ritz matrix:
// 9e-4, 2e-5, 1e-6, 7e-9, 9e-12, 2e-14), so the value reached is well under the bound.
constexpr float kJacobiTol = 1e-8f;

// The sweeps are one cooperative kernel.  All CTAs are resident at once, so a round needs no kernel boundary (as
// three launches per round the ~7000 rounds of a 576 x 576 matrix were launch bound: 63 ms against 13 ms): every round reads the
// matrices of the previous round (M, P in buffer `cur`) and writes the other buffer, and one grid-wide barrier
// separates the rounds.  A round: every CTA works out the l/2 rotations of the round from M (cheap, and saves a
// second barrier), then the grid updates M block by block -- the 2 x 2 block (rows p_a, q_a; columns p_b, q_b)
// takes the column rotation of pair b and then the row rotation of pair a --
// and rotates the column pairs of P.  Reads bypass L1 (other SMs wrote the data), the barrier is an arrival
// counter that only grows plus a generation word; its wait is bounded like every wait of the library: a CTA that
// gives up raises XKV_FLAG_TIMEOUT and the abort word, and every other CTA leaves at its next wait.
constexpr int kJacobiCoopThreads = 512;
constexpr unsigned kJacobiSpinLimit = 1u << 18;   // polls of a barrier that normally opens within microseconds

struct JacobiSync {          // words of the workspace's flag block
  unsigned int* flags;       // status word
  unsigned int* count;       // arrivals so far (monotonic)
  unsigned int* gen;         // barriers completed
  unsigned int* abort;       // a CTA gave up
  unsigned int spin_limit;   // polls of one barrier wait
  unsigned int skip_first;   // fault injection (tests of the give-up path): CTA 0 passes the first barrier without arriving
};

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned int* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_u32(unsigned int* p, unsigned v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Returns false when the barrier was abandoned (by this CTA or another one).  `my_gen` counts this CTA's barriers.
__device__ __forceinline__ bool jacobi_grid_barrier(const JacobiSync& sy, unsigned& my_gen, int* ok_s) {
  __syncthreads();
  if (threadIdx.x == 0) {
    ++my_gen;
    __threadfence();
    bool ok = true;
    if (sy.skip_first && blockIdx.x == 0 && my_gen == 1u) {
      // injected fault: the others never see this arrival, run into their limit and raise the abort word
    } else if (atomicAdd(sy.count, 1u) == gridDim.x * my_gen - 1u) {
      st_release_u32(sy.gen, my_gen);                      // last to arrive: open the barrier
    } else {
      unsigned i = 0;
      while (ld_acquire_u32(sy.gen) < my_gen) {
        if (++i >= sy.spin_limit || ld_acquire_u32(sy.abort) != 0u) { ok = false; break; }
      }
    }
    if (!ok) { atomicOr(sy.flags, XKV_FLAG_TIMEOUT); atomicExch(sy.abort, 1u); }
    __threadfence();
    *ok_s = ok ? 1 : 0;
  }
  __syncthreads();
  return *ok_s != 0;
}

__global__ void __launch_bounds__(kJacobiCoopThreads, 1)
jacobi_coop_kernel(float* __restrict__ M0, float* __restrict__ M1, float* __restrict__ P0, float* __restrict__ P1, int l,
                   float2* __restrict__ partial, JacobiSync sy) {
  __shared__ float2 cs_s[kJacobiMaxPairs];
  __shared__ int2 pq_s[kJacobiMaxPairs];
  __shared__ int ok_s;
  __shared__ float2 red_s[kJacobiCoopThreads / 32];
  __shared__ int done_s;
  const int tid = threadIdx.x, nb = gridDim.x;
  const int np = l / 2;                                   // l is even (a multiple of 64)
  const long long gtid = (long long)blockIdx.x * kJacobiCoopThreads + tid, gstride = (long long)nb * kJacobiCoopThreads;
  unsigned my_gen = 0;
  for (long long e = gtid; e < (long long)l * l; e += gstride) P0[e] = (e / l == e % l) ? 1.0f : 0.0f;
  int cur = 0;
  bool alive = jacobi_grid_barrier(sy, my_gen, &ok_s);
  int sweeps_done = 0;
  for (int sweep = 0; alive && sweep < kJacobiSweeps; ++sweep) {
    // ---- off-diagonal weight of M: per-CTA partial sums, then every CTA adds them up in the same order
    {
      const float* M = cur ? M1 : M0;
      float off = 0.0f, all = 0.0f;
      for (long long e = gtid; e < (long long)l * l; e += gstride) {
        const float v = __ldcg(M + e);
        all += v * v;
        if (e / l != e % l) off += v * v;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) { off += __shfl_xor_sync(0xffffffffu, off, o); all += __shfl_xor_sync(0xffffffffu, all, o); }
      if ((tid & 31) == 0) red_s[tid >> 5] = make_float2(off, all);
      __syncthreads();
      if (tid == 0) {
        float o2 = 0.0f, a2 = 0.0f;
        for (int w = 0; w < kJacobiCoopThreads / 32; ++w) { o2 += red_s[w].x; a2 += red_s[w].y; }
        partial[(sweep & 1) * nb + blockIdx.x] = make_float2(o2, a2);
      }
      alive = jacobi_grid_barrier(sy, my_gen, &ok_s);
      if (!alive) break;
      if (tid == 0) {
        float o2 = 0.0f, a2 = 0.0f;
        for (int b = 0; b < nb; ++b) { const float2 v = __ldcg(partial + (sweep & 1) * nb + b); o2 += v.x; a2 += v.y; }
        done_s = (o2 <= kJacobiTol * a2) ? 1 : 0;
      }
      __syncthreads();
      if (done_s) break;                                  // the same decision in every CTA
    }
    ++sweeps_done;
    for (int t = 0; alive && t < l - 1; ++t) {
      const float* M = cur ? M1 : M0;
      const float* P = cur ? P1 : P0;
      float* Mn = cur ? M0 : M1;
      float* Pn = cur ? P0 : P1;
      // pair k of round t (round-robin order), smaller index first
      auto pair_of = [&](int k) -> int2 {
        int p, q;
        if (k == 0) { p = l - 1; q = t; }
        else { p = (t + k) % (l - 1); q = (t - k + l - 1) % (l - 1); }
        return p < q ? make_int2(p, q) : make_int2(q, p);
      };
      // M: 2 x 2 blocks (pair a of rows, pair b of columns); P: column pairs, every row; kBatch items of each per
      // pass.  The loads of the first pass are issued before the rotations are worked out -- their addresses
      // depend on the round only -- so that a round of a 576 x 576 matrix is one trip to L2, not three.
      constexpr int kBatch = 4;
      const long long nM = (long long)np * np, nP = (long long)l * np;
      float x0[kBatch], y0[kBatch], x1[kBatch], y1[kBatch], pu[kBatch], pv[kBatch];
      int ka[kBatch], kb[kBatch], pi[kBatch], pk[kBatch];
      auto load_m = [&](long long base) {
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
          const long long it = base + u * gstride;
          ka[u] = -1;
          if (it < nM) {
            ka[u] = (int)(it / np); kb[u] = (int)(it - (long long)ka[u] * np);
            const int2 ra = pair_of(ka[u]), cb = pair_of(kb[u]);
            const float* r0 = M + (size_t)ra.x * l;
            const float* r1 = M + (size_t)ra.y * l;
            x0[u] = __ldcg(r0 + cb.x); y0[u] = __ldcg(r0 + cb.y); x1[u] = __ldcg(r1 + cb.x); y1[u] = __ldcg(r1 + cb.y);
          }
        }
      };
      auto load_p = [&](long long base) {
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
          const long long it = base + u * gstride;
          pi[u] = -1;
          if (it < nP) {
            pi[u] = (int)(it / np); pk[u] = (int)(it - (long long)pi[u] * np);
            const int2 ix = pair_of(pk[u]);
            pu[u] = __ldcg(P + (size_t)pi[u] * l + ix.x); pv[u] = __ldcg(P + (size_t)pi[u] * l + ix.y);
          }
        }
      };
      auto finish_m = [&]() {
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
          if (ka[u] < 0) continue;
          const int2 ra = pq_s[ka[u]], cb = pq_s[kb[u]];
          const float2 ja = cs_s[ka[u]], jb = cs_s[kb[u]];
          float a0 = x0[u], b0 = y0[u], a1 = x1[u], b1 = y1[u];
          if (jb.y != 0.0f) {                             // columns p_b, q_b
            const float u0 = jb.x * a0 - jb.y * b0, v0 = jb.y * a0 + jb.x * b0;
            const float u1 = jb.x * a1 - jb.y * b1, v1 = jb.y * a1 + jb.x * b1;
            a0 = u0; b0 = v0; a1 = u1; b1 = v1;
          }
          if (ja.y != 0.0f) {                             // rows p_a, q_a
            const float u0 = ja.x * a0 - ja.y * a1, u1 = ja.y * a0 + ja.x * a1;
            const float v0 = ja.x * b0 - ja.y * b1, v1 = ja.y * b0 + ja.x * b1;
            a0 = u0; a1 = u1; b0 = v0; b1 = v1;
          }
          float* w0 = Mn + (size_t)ra.x * l;
          float* w1 = Mn + (size_t)ra.y * l;
          w0[cb.x] = a0; w0[cb.y] = b0; w1[cb.x] = a1; w1[cb.y] = b1;
        }
      };
      auto finish_p = [&]() {
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
          if (pi[u] < 0) continue;
          const int2 ix = pq_s[pk[u]];
          const float2 j = cs_s[pk[u]];
          float nu = pu[u], nv = pv[u];
          if (j.y != 0.0f) { nu = j.x * pu[u] - j.y * pv[u]; nv = j.y * pu[u] + j.x * pv[u]; }
          Pn[(size_t)pi[u] * l + ix.x] = nu;
          Pn[(size_t)pi[u] * l + ix.y] = nv;
        }
      };
      load_m(gtid);
      load_p(gtid);
      for (int k = tid; k < np; k += kJacobiCoopThreads) {
        const int2 ix = pair_of(k);
        const int p = ix.x, q = ix.y;
        float c = 1.0f, sn = 0.0f;
        const float app = __ldcg(M + (size_t)p * l + p), aqq = __ldcg(M + (size_t)q * l + q), apq = __ldcg(M + (size_t)p * l + q);
        if (fabsf(apq) > 1e-30f && fabsf(apq) > 1e-9f * sqrtf(fabsf(app * aqq))) {
          const float tau = (aqq - app) / (2.0f * apq);
          const float tt = (tau >= 0.0f ? 1.0f : -1.0f) / (fabsf(tau) + sqrtf(1.0f + tau * tau));
          c = rsqrtf(1.0f + tt * tt);
          sn = tt * c;
        }
        cs_s[k] = make_float2(c, sn);
        pq_s[k] = ix;
      }
      __syncthreads();
      finish_m();
      finish_p();
      for (long long base = gtid + kBatch * gstride; base < nM; base += kBatch * gstride) { load_m(base); finish_m(); }
      for (long long base = gtid + kBatch * gstride; base < nP; base += kBatch * gstride) { load_p(base); finish_p(); }
      alive = jacobi_grid_barrier(sy, my_gen, &ok_s);
      cur ^= 1;
    }
  }
  if (blockIdx.x == 0 && tid == 0) sy.abort[1] = (unsigned)sweeps_done;   // diagnostic: sweeps that ran
  if (alive && cur == 1) {                                // the callers read buffer 0
    for (long long e = gtid; e < (long long)l * l; e += gstride) { M0[e] = __ldcg(M1 + e); P0[e] = __ldcg(P1 + e); }
  }
}

// The r largest eigenvalues (ties to the lower index) and their eigenvectors as the columns of Psel (l x r);
// sigma = sqrt(lambda).
__global__ void __launch_bounds__(1024)
eig_select_kernel(const float* __restrict__ M, const float* __restrict__ P, int l, int r, float* __restrict__ Psel,
                  float* __restrict__ sigma) {
  extern __shared__ int rank_s[];                      // [l]
  const int tid = threadIdx.x;
  for (int i = tid; i < l; i += 1024) {
    const float li = M[(size_t)i * l + i];
    int rk = 0;
    for (int j = 0; j < l; ++j) {
      const float lj = M[(size_t)j * l + j];
      rk += (lj > li || (lj == li && j < i)) ? 1 : 0;
    }
    rank_s[i] = rk;
    if (rk < r && sigma) sigma[rk] = sqrtf(fmaxf(li, 0.0f));
  }
  __syncthreads();
  for (int e = tid; e < l * l; e += 1024) {
    const int row = e / l, i = e % l;
    const int rk = rank_s[i];
    if (rk < r) Psel[(size_t)row * r + rk] = P[e];
  }
}

// V (N x r, fp32) -> its bf16 copy and the per-layer matrices B [G][r][d], B[g][m][j] = V[g d + j][m].
__global__ void clf_finish_kernel(const float* __restrict__ V, int G, int d, int r, __nv_bfloat16* __restrict__ Vb,
                                  __nv_bfloat16* __restrict__ B) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long total = (long long)G * d * r;
  if (idx >= total) return;
  const int m = (int)(idx % r);
  const long long row = idx / r;                       // g d + j
  const int g = (int)(row / d), j = (int)(row % d);
  const __nv_bfloat16 v = __float2bfloat16(V[idx]);
  Vb[idx] = v;
  B[((size_t)g * r + m) * d + j] = v;
}

}  // namespace

namespace {

__global__ void symmetrize_kernel(float* __restrict__ M, int l) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= l * l) return;
  const int i = e / l, j = e % l;
  if (i < j) {
    const float v = 0.5f * (M[(size_t)i * l + j] + M[(size_t)j * l + i]);
    M[(size_t)i * l + j] = v;
    M[(size_t)j * l + i] = v;
  }
}

struct ClfPlan {
  int T, Tp, N, r, l, q;
  size_t off_flags, off_zb, off_yt, off_u, off_z, off_g, off_m, off_p, off_ps, off_v, off_vb, off_cs, off_m2, off_p2, off_xinv, total;
};

size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }

bool make_plan(const xkv_clf_config* c, ClfPlan* p) {
  p->T = c->T; p->Tp = (c->T + 7) & ~7; p->N = c->G * c->d; p->r = c->r; p->q = c->power_iters;
  const int over = c->oversample > 0 ? c->oversample : 32;
  p->l = (c->r + over + 63) & ~63;
  if (p->l > p->N) p->l = p->N & ~63;
  if (p->l < c->r || p->l < 64 || p->l / 2 > kJacobiMaxPairs) return false;
  size_t o = 0;
  p->off_flags = o; o = align_up(o + 256);
  p->off_zb = o; o = align_up(o + (size_t)p->N * p->l * 2);
  p->off_yt = o; o = align_up(o + (size_t)p->l * p->Tp * 2);
  p->off_u = o; o = align_up(o + (size_t)p->N * p->l * 4);
  p->off_z = o; o = align_up(o + (size_t)p->N * p->l * 4);
  p->off_g = o; o = align_up(o + (size_t)p->l * p->l * 8);      // the Gram matrix / Cholesky factor, fp64
  p->off_m = o; o = align_up(o + (size_t)p->l * p->l * 4);
  p->off_p = o; o = align_up(o + (size_t)p->l * p->l * 4);
  p->off_ps = o; o = align_up(o + (size_t)p->l * p->r * 4);
  p->off_v = o; o = align_up(o + (size_t)p->N * p->r * 4);
  p->off_vb = o; o = align_up(o + (size_t)p->N * p->r * 2);
  p->off_cs = o; o = align_up(o + (size_t)2 * 1024 * 8);            // per-CTA partial sums of the Jacobi convergence check
  p->off_m2 = o; o = align_up(o + (size_t)p->l * p->l * 4);      // second buffers of the one-kernel Jacobi sweeps
  p->off_p2 = o; o = align_up(o + (size_t)p->l * p->l * 4);
  p->off_xinv = o; o = align_up(o + (size_t)p->l * kTriBlock * 8);   // inverses of the diagonal blocks of a Cholesky factor
  p->total = o;
  return true;
}

int check_clf_config(const xkv_clf_config* c) {
  if (!c || c->struct_size != sizeof(xkv_clf_config)) return XKV_ERR_INVALID_ARG;
  if (c->T < 1 || c->T >= (1 << 24) || c->G < 1 || c->d < 8 || c->r < 8 || c->power_iters < 0 || c->power_iters > 8 ||
      c->oversample < 0)
    return XKV_ERR_INVALID_ARG;
  if (c->r % 8 || (c->G * (long long)c->d) % 64 || c->G * (long long)c->d > (1 << 20)) return XKV_ERR_INVALID_ARG;
  if (c->r > c->G * c->d) return XKV_ERR_INVALID_ARG;
  return XKV_OK;
}

template <bool TRANS, int BN>
cudaError_t launch_gemm_bn(const void* a, int a_rows_k, int a_cols_m, int a_pitch, const void* b, int b_rows_n, int b_cols_k,
                           int b_pitch, float* Cf, __nv_bfloat16* Cb, long long ldc, unsigned int* flags, int device,
                           cudaStream_t s) {
  CUtensorMap ma, mb;
  if (!encode_bf16_map(&ma, a, (uint64_t)a_rows_k, (uint64_t)a_cols_m, (uint64_t)a_pitch, 64) ||
      !encode_bf16_map(&mb, b, (uint64_t)b_rows_n, (uint64_t)b_cols_k, (uint64_t)b_pitch, BN))
    return cudaErrorInvalidValue;
  const size_t smem = 1024 + (size_t)gemm_stages<BN>() * gemm_stage_bytes<BN>();
  cudaError_t e = ensure_dyn_smem<clf_gemm_kernel<TRANS, BN>>(smem, device);
  if (e != cudaSuccess) return e;
  const dim3 grid((b_rows_n + BN - 1) / BN, (a_cols_m + 127) / 128);
  clf_gemm_kernel<TRANS, BN><<<grid, kGemmThreads, smem, s>>>(ma, mb, a_cols_m, b_rows_n, a_rows_k, Cf, Cb, ldc, flags);
  count_launch(kFamClf);
  return cudaGetLastError();
}

// The tile width that pads N least (the widest on a tie): 576 columns are three tiles of 192, a tall N is tiles of 256.
template <bool TRANS>
cudaError_t launch_gemm(const void* a, int a_rows_k, int a_cols_m, int a_pitch, const void* b, int b_rows_n, int b_cols_k,
                        int b_pitch, float* Cf, __nv_bfloat16* Cb, long long ldc, unsigned int* flags, int device,
                        cudaStream_t s) {
  const int N = b_rows_n;
  auto padded = [&](int bn) { return (long long)((N + bn - 1) / bn) * bn; };
  int bn = 256;
  if (padded(192) < padded(bn)) bn = 192;
  if (padded(128) < padded(bn)) bn = 128;
  if (bn == 256) return launch_gemm_bn<TRANS, 256>(a, a_rows_k, a_cols_m, a_pitch, b, b_rows_n, b_cols_k, b_pitch, Cf, Cb, ldc, flags, device, s);
  if (bn == 192) return launch_gemm_bn<TRANS, 192>(a, a_rows_k, a_cols_m, a_pitch, b, b_rows_n, b_cols_k, b_pitch, Cf, Cb, ldc, flags, device, s);
  return launch_gemm_bn<TRANS, 128>(a, a_rows_k, a_cols_m, a_pitch, b, b_rows_n, b_cols_k, b_pitch, Cf, Cb, ldc, flags, device, s);
}

}  // namespace

int clf_rank_l(const xkv_clf_config* c, int* l) {
  int st = check_clf_config(c);
  if (st != XKV_OK) return st;
  ClfPlan p;
  if (!make_plan(c, &p)) return XKV_ERR_UNSUPPORTED;
  *l = p.l;
  return XKV_OK;
}

int clf_workspace_bytes(const xkv_clf_config* c, uint64_t* bytes) {
  int st = check_clf_config(c);
  if (st != XKV_OK) return st;
  ClfPlan p;
  if (!make_plan(c, &p)) return XKV_ERR_UNSUPPORTED;
  *bytes = p.total;
  return XKV_OK;
}

// Debug/test entry of the tensor-core product alone: C (M x N, fp32) = A B^T, A bf16 [K][M], B bf16 [N][K].
cudaError_t clf_gemm(const void* a, const void* b, int M, int N, int K, float* C, unsigned int* flags, int device, cudaStream_t s) {
  return launch_gemm<false>(a, K, M, M, b, N, K, K, C, nullptr, N, flags, device, s);
}

static std::atomic<unsigned> g_clf_inject{0};
void clf_set_fault_injection(unsigned mask) { g_clf_inject.store(mask, std::memory_order_relaxed); }

int clf_factorize(const xkv_clf_config* c, const void* X, const void* omega, void* workspace, uint64_t workspace_bytes,
                  void* A_out, void* B_out, float* sigma, int device, cudaStream_t s) {
  int st = check_clf_config(c);
  if (st != XKV_OK) return st;
  ClfPlan p;
  if (!make_plan(c, &p)) return XKV_ERR_UNSUPPORTED;
  if (workspace_bytes < p.total) return XKV_ERR_INVALID_ARG;
  uint8_t* w = (uint8_t*)workspace;
  unsigned int* flags = (unsigned int*)(w + p.off_flags);
  __nv_bfloat16* Zb = (__nv_bfloat16*)(w + p.off_zb);
  __nv_bfloat16* Yt = (__nv_bfloat16*)(w + p.off_yt);
  float* U = (float*)(w + p.off_u);
  float* Z = (float*)(w + p.off_z);
  double* Gm = (double*)(w + p.off_g);
  float* Mm = (float*)(w + p.off_m);
  float* Pm = (float*)(w + p.off_p);
  float* Ps = (float*)(w + p.off_ps);
  float* V = (float*)(w + p.off_v);
  __nv_bfloat16* Vb = (__nv_bfloat16*)(w + p.off_vb);
  const int N = p.N, l = p.l, r = p.r, T = p.T;
  cudaError_t e = cudaMemsetAsync(flags, 0, 256, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(Zb, omega, (size_t)N * l * 2, cudaMemcpyDeviceToDevice, s);
  const dim3 g_ll((l + 63) / 64, (l + 63) / 64);
  // Y^T = Z^T X^T  then  U = X^T Y
  auto two_products = [&]() -> cudaError_t {
    cudaError_t e2 = launch_gemm<false>(Zb, N, l, l, X, T, N, N, nullptr, Yt, p.Tp, flags, device, s);
    if (e2 != cudaSuccess) return e2;
    return launch_gemm<false>(X, T, N, N, Yt, l, T, p.Tp, U, nullptr, l, flags, device, s);
  };
  // Z = orth(src) by three passes of shifted Cholesky QR.  The Gram matrix is accumulated, factorised and solved
  // in fp64: its condition number is the square of the iterate's, which after a multiplication by X^T X spans the
  // whole range between the largest singular value and the noise floor.
  const size_t solve_smem = (size_t)kSolveWarps * l * sizeof(double);
  e = e == cudaSuccess ? ensure_dyn_smem<trsolve_rows_kernel>(solve_smem, device) : e;
  const size_t tri_smem = ((size_t)kTriRows * (l + 4) + (size_t)kTriBlock * kDgemmLd) * sizeof(double);
  // the blocked solve keeps 32 rows of Z in shared memory: sketches wider than about 700 columns take the row-wise kernel
  const bool mma_solve = tri_smem <= 227u * 1024u;
  if (mma_solve) e = e == cudaSuccess ? ensure_dyn_smem<trsolve_mma_kernel>(tri_smem, device) : e;
  double* Xinv = (double*)(w + p.off_xinv);
  // Every pass divides the condition number by about shift^-1/2; the iterate of a power iteration only has to stay
  // well conditioned (two passes), the last one has to be orthonormal (five passes with decreasing shifts: the
  // columns of U that lie in the noise floor are 10^8 times smaller than the leading ones).
  static const double kShifts[5] = {1e-4, 1e-5, 1e-6, 1e-8, 1e-10};
  auto cholqr = [&](const float* src, int passes) -> cudaError_t {
    for (int pass = 0; pass < passes; ++pass) {
      const float* in = pass == 0 ? src : Z;
      dgemm_tn_mma_kernel<double><<<g_ll, 256, 0, s>>>(in, in, Gm, N, l, l, l);
      const double shift_rel = kShifts[pass];
      chol_shift_kernel<<<1, 1024, 0, s>>>(Gm, l, shift_rel);
      int launches = 2;
      for (int kb = 0; kb < l; kb += kCholNb) {
        const int nb = l - kb < kCholNb ? l - kb : kCholNb;
        chol_diag_kernel<<<1, kCholNb, 0, s>>>(Gm, l, kb, nb, flags);
        const int rem = l - kb - nb;
        ++launches;
        if (rem > 0) {
          chol_panel_kernel<<<(rem + kCholPanelThreads - 1) / kCholPanelThreads, kCholPanelThreads, 0, s>>>(Gm, l, kb, nb);
          const int tiles = (rem + kCholNb - 1) / kCholNb;
          chol_update_kernel<<<dim3(tiles, tiles), dim3(kCholNb, kCholNb), 0, s>>>(Gm, l, kb, nb);
          launches += 2;
        }
      }
      if (!mma_solve) {
        trsolve_rows_kernel<<<(N + kSolveWarps - 1) / kSolveWarps, kSolveWarps * 32, solve_smem, s>>>(in, Gm, Z, Zb, N, l);
      } else {
        tri_inv_diag_kernel<<<l / kTriBlock, kTriBlock, 0, s>>>(Gm, l, Xinv);
        trsolve_mma_kernel<<<(N + kTriRows - 1) / kTriRows, 256, tri_smem, s>>>(in, Gm, Xinv, Z, Zb, N, l);
        ++launches;
      }
      count_launch(kFamClf, launches + 1);
    }
    return cudaGetLastError();
  };
  for (int it = 0; it <= p.q && e == cudaSuccess; ++it) {
    e = two_products();
    if (e == cudaSuccess) e = cholqr(U, it == p.q ? 5 : 2);
  }
  if (e == cudaSuccess) e = two_products();              // W = X Z and U' = X^T W for the Rayleigh-Ritz step
  if (e == cudaSuccess) {
    dgemm_tn_mma_kernel<float><<<g_ll, 256, 0, s>>>(Z, U, Mm, N, l, l, l);     // M = Z^T U', accumulated in fp64
    symmetrize_kernel<<<(l * l + 255) / 256, 256, 0, s>>>(Mm, l);
    {
      int per_sm = 0, sms = 0;
      e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, jacobi_coop_kernel, kJacobiCoopThreads, 0);
      if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
      if (e == cudaSuccess && per_sm < 1) e = cudaErrorLaunchOutOfResources;
      if (e == cudaSuccess) {
        float* M2 = (float*)(w + p.off_m2);
        float* P2 = (float*)(w + p.off_p2);
        float2* partial = (float2*)(w + p.off_cs);
        const bool inject = (g_clf_inject.load(std::memory_order_relaxed) & XKV_INJECT_CLF_BARRIER) != 0u;
        JacobiSync sy{flags, flags + 8, flags + 9, flags + 10,            // zeroed with the flag block above
                      inject ? 1024u : kJacobiSpinLimit, inject ? 1u : 0u};
        int l_arg = l;
        void* args[] = {&Mm, &M2, &Pm, &P2, &l_arg, &partial, &sy};
        e = cudaLaunchCooperativeKernel((const void*)jacobi_coop_kernel, dim3(sms), dim3(kJacobiCoopThreads), args, 0, s);
        count_launch(kFamClf, 1);
      }
    }
    if (e == cudaSuccess) {
      eig_select_kernel<<<1, 1024, (size_t)l * sizeof(int), s>>>(Mm, Pm, l, r, Ps, sigma);
      sgemm_small_kernel<false, float><<<dim3((r + 63) / 64, (N + 63) / 64), 256, 0, s>>>(Z, Ps, V, N, r, l, l, r, r);
      const long long tot = (long long)N * r;
      clf_finish_kernel<<<(unsigned)((tot + 255) / 256), 256, 0, s>>>(V, c->G, c->d, r, Vb, (__nv_bfloat16*)B_out);
      count_launch(kFamClf, 5);
      e = cudaGetLastError();
    }
  }
  // A = X V_bf16, stored [T][r]
  if (e == cudaSuccess) e = launch_gemm<true>(Vb, N, r, r, X, T, N, N, nullptr, (__nv_bfloat16*)A_out, r, flags, device, s);
  if (e != cudaSuccess) { set_cuda_error(e); (void)cudaGetLastError(); return XKV_ERR_CUDA; }
  return XKV_OK;
}

}  // namespace xkv
