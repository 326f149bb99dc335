// Selective reconstruction (Sec. 3.2, Eq. 3) fused with decode attention over the rebuilt rows.
//
// recon_attend_tile_kernel   one CTA per (problem, tile of 64 selected rows): gathers the rows of
//                            A_k / A_v, multiplies by the head's reconstruction block, rotates the key
//                            rows, and reduces the tile to an un-normalised partial (m, l, o).
// merge_kernel               combines the partials of a problem by log-sum-exp.
#include "xkv_internal.cuh"

namespace xkv {

namespace {

constexpr int kTileRows = 64;
constexpr int kSlab = 32;            // columns of r per staged slab
constexpr int kThreads = 256;

// K-hat / V-hat tile = A[S_tile] (64 x r) * Bt^T (r x DH), fp32 accumulate, result to smem [64][DH+1].
template <int DH>
__device__ __forceinline__ void recon_tile(const __nv_bfloat16* __restrict__ A, int r, const int* rows_s,
                                           const __nv_bfloat16* __restrict__ Bt, float* As_t, float* Bs,
                                           float* Xs) {
  constexpr int CPT = DH / 16;       // output columns per thread
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  float acc[4][CPT];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < CPT; ++j) acc[i][j] = 0.0f;

  for (int m0 = 0; m0 < r; m0 += kSlab) {
    {  // gathered A slab: 64 rows x 32 columns, one 16-byte piece per thread
      const int row = tid >> 2, piece = tid & 3, m = m0 + piece * 8;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (m < r) v = *reinterpret_cast<const uint4*>(A + (size_t)rows_s[row] * r + m);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        As_t[(piece * 8 + 2 * e) * (kTileRows + 4) + row] = __uint_as_float(w[e] << 16);
        As_t[(piece * 8 + 2 * e + 1) * (kTileRows + 4) + row] = __uint_as_float(w[e] & 0xffff0000u);
      }
    }
    for (int t = tid; t < DH * 4; t += kThreads) {  // Bt slab: DH rows x 32 columns
      const int j = t >> 2, piece = t & 3, m = m0 + piece * 8;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (m < r) v = *reinterpret_cast<const uint4*>(Bt + (size_t)j * r + m);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        Bs[(piece * 8 + 2 * e) * (DH + 4) + j] = __uint_as_float(w[e] << 16);
        Bs[(piece * 8 + 2 * e + 1) * (DH + 4) + j] = __uint_as_float(w[e] & 0xffff0000u);
      }
    }
    __syncthreads();
#pragma unroll 8
    for (int kk = 0; kk < kSlab; ++kk) {
      const float4 a = *reinterpret_cast<const float4*>(As_t + kk * (kTileRows + 4) + ty * 4);
      const float av[4] = {a.x, a.y, a.z, a.w};
      float bv[CPT];
#pragma unroll
      for (int j = 0; j < CPT; j += 4) {
        const float4 b4 = *reinterpret_cast<const float4*>(Bs + kk * (DH + 4) + tx * CPT + j);
        bv[j] = b4.x; bv[j + 1] = b4.y; bv[j + 2] = b4.z; bv[j + 3] = b4.w;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < CPT; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < CPT; ++j) Xs[(ty * 4 + i) * (DH + 1) + tx * CPT + j] = acc[i][j];
  __syncthreads();
}

// grid.x = tiles (ceil(k_cap/64)), grid.y = problems of the call
template <int DH>
__global__ void __launch_bounds__(kThreads)
recon_attend_tile_kernel(GroupDev dev, int l0, const __nv_bfloat16* __restrict__ q,
                         const int32_t* __restrict__ sel_idx, const int32_t* __restrict__ sel_cnt, int k_cap,
                         int n_tiles) {
  extern __shared__ float sm[];
  float* As_t = sm;                                    // [32][64+4]
  float* Bs = As_t + kSlab * (kTileRows + 4);          // [32][DH+4]
  float* Xs = Bs + kSlab * (DH + 4);                   // [64][DH+1]
  float* qs = Xs + kTileRows * (DH + 1);               // [n_rep][DH]
  float* ps = qs + kMaxRep * DH;                       // [n_rep][64] logits, then weights
  float* ms = ps + kMaxRep * kTileRows;                // [n_rep] tile max
  float* ls = ms + kMaxRep;                            // [n_rep] tile sum
  int* rows_s = reinterpret_cast<int*>(ls + kMaxRep);  // [64] gathered row (clamped)
  int* pos_s = rows_s + kTileRows;                     // [64] token position, -1 if masked

  const int tid = threadIdx.x;
  const int per_layer = dev.batch * dev.H_kv;
  const int g = blockIdx.y % dev.H_kv;
  const int b = (blockIdx.y / dev.H_kv) % dev.batch;
  const int l = l0 + blockIdx.y / per_layer;
  const long long prob = ((long long)l * dev.batch + b) * dev.H_kv + g;
  const int cnt = min(sel_cnt[prob], k_cap);
  const int t0 = blockIdx.x * kTileRows;
  if (t0 >= cnt) return;
  const int n_rep = dev.n_rep;

  if (tid < kTileRows) {
    int p = -1;
    if (t0 + tid < cnt) {
      p = sel_idx[prob * k_cap + t0 + tid];
      if (p < 0 || p >= dev.T) { atomicOr(dev.flags, XKV_FLAG_INDEX_RANGE); p = -1; }
    }
    pos_s[tid] = p;
    rows_s[tid] = p < 0 ? 0 : p;
  }
  const __nv_bfloat16* qg = q + (((long long)l * dev.batch + b) * dev.H_q + (long long)g * n_rep) * DH;
  for (int i = tid; i < n_rep * DH; i += kThreads) qs[i] = __bfloat162float(qg[i]);
  __syncthreads();

  const size_t head = ((size_t)b * dev.G + l) * dev.H_kv + g;
  // ---- keys: reconstruct, rotate, logits
  recon_tile<DH>(dev.A_k + (size_t)b * dev.T * dev.r_k, dev.r_k, rows_s, dev.Bt_k + head * kDP * dev.r_k,
                 As_t, Bs, Xs);
  constexpr int HALF = DH / 2;
  if (dev.use_rope) {
    // thread (j, part) rotates a quarter of row j in place
    const int j = tid >> 2, part = tid & 3;
    const int p = rows_s[j];
    const float2* hi = dev.rope_hi + (size_t)(p >> dev.rope_shift) * HALF;
    const float2* lo = dev.rope_lo + (size_t)(p & ((1 << dev.rope_shift) - 1)) * HALF;
    for (int i = part; i < HALF; i += 4) {
      const float2 a = hi[i], c2 = lo[i];
      const float cs = a.x * c2.x - a.y * c2.y, sn = a.y * c2.x + a.x * c2.y;
      const float x1 = Xs[j * (DH + 1) + i], x2 = Xs[j * (DH + 1) + i + HALF];
      Xs[j * (DH + 1) + i] = x1 * cs - x2 * sn;
      Xs[j * (DH + 1) + i + HALF] = x2 * cs + x1 * sn;
    }
    __syncthreads();
  }
  for (int t = tid; t < n_rep * kTileRows; t += kThreads) {
    const int h = t / kTileRows, j = t % kTileRows;
    float z = 0.0f;
#pragma unroll 8
    for (int i = 0; i < DH; ++i) z = fmaf(qs[h * DH + i], Xs[j * (DH + 1) + i], z);
    ps[h * kTileRows + j] = pos_s[j] < 0 ? -INFINITY : z * dev.att_scale;
  }
  __syncthreads();
  {  // per head: tile max, weights, sum (one warp per head, 8 warps round-robin)
    const int warp = tid >> 5, lane = tid & 31;
    for (int h = warp; h < n_rep; h += kThreads / 32) {
      const float z0 = ps[h * kTileRows + lane], z1 = ps[h * kTileRows + lane + 32];
      float m = fmaxf(z0, z1);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      const float w0 = (m == -INFINITY) ? 0.0f : __expf(z0 - m), w1 = (m == -INFINITY) ? 0.0f : __expf(z1 - m);
      float sum = w0 + w1;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      ps[h * kTileRows + lane] = w0;
      ps[h * kTileRows + lane + 32] = w1;
      if (lane == 0) { ms[h] = m; ls[h] = sum; }
    }
  }
  __syncthreads();
  // ---- values: reconstruct, weighted sum
  recon_tile<DH>(dev.A_v + (size_t)b * dev.T * dev.r_v, dev.r_v, rows_s, dev.Bt_v + head * kDP * dev.r_v,
                 As_t, Bs, Xs);
  float* part = dev.part + ((size_t)prob * n_tiles + blockIdx.x) * n_rep * (DH + 2);
  for (int t = tid; t < n_rep * DH; t += kThreads) {
    const int h = t / DH, dcol = t % DH;
    float o = 0.0f;
#pragma unroll 8
    for (int j = 0; j < kTileRows; ++j) o = fmaf(ps[h * kTileRows + j], Xs[j * (DH + 1) + dcol], o);
    part[h * (DH + 2) + dcol] = o;
  }
  if (tid < n_rep) {
    part[tid * (DH + 2) + DH] = ms[tid];
    part[tid * (DH + 2) + DH + 1] = ls[tid];
  }
}

// grid.x = problems of the call * n_rep; blockDim = DH.  Partials are merged in tile order.
template <int DH>
__global__ void __launch_bounds__(DH)
merge_kernel(GroupDev dev, int l0, const int32_t* __restrict__ sel_cnt, int k_cap, int n_tiles, int rows_per_part,
             __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
  const int n_rep = dev.n_rep;
  const int h = blockIdx.x % n_rep;
  const int py = blockIdx.x / n_rep;
  const int per_layer = dev.batch * dev.H_kv;
  const int g = py % dev.H_kv;
  const int b = (py / dev.H_kv) % dev.batch;
  const int l = l0 + py / per_layer;
  const long long prob = ((long long)l * dev.batch + b) * dev.H_kv + g;
  const int cnt = min(sel_cnt[prob], k_cap);
  const int used = (cnt + rows_per_part - 1) / rows_per_part;
  const float* part = dev.part + ((size_t)prob * n_tiles) * n_rep * (DH + 2) + (size_t)h * (DH + 2);
  const size_t stride = (size_t)n_rep * (DH + 2);
  float M = -INFINITY;
  for (int t = 0; t < used; ++t) M = fmaxf(M, part[t * stride + DH]);
  float L = 0.0f, o = 0.0f;
  if (M != -INFINITY) {
    for (int t = 0; t < used; ++t) {
      const float mt = part[t * stride + DH];
      const float w = (mt == -INFINITY) ? 0.0f : __expf(mt - M);
      L += w * part[t * stride + DH + 1];
      o += w * part[t * stride + threadIdx.x];
    }
  }
  const long long qh = ((long long)l * dev.batch + b) * dev.H_q + (long long)g * n_rep + h;
  out[qh * DH + threadIdx.x] = __float2bfloat16(L > 0.0f ? o / L : 0.0f);
  if (lse && threadIdx.x == 0) lse[qh] = L > 0.0f ? M + logf(L) : -INFINITY;
}

template <int DH>
cudaError_t launch_t(const xkv_group* grp, int l0, int l1, const __nv_bfloat16* q, const int32_t* sel_idx,
                     const int32_t* sel_cnt, int k_cap, __nv_bfloat16* out, float* lse, cudaStream_t s) {
  const GroupDev& dev = grp->dev;
  const int problems = (l1 - l0) * dev.batch * dev.H_kv;
  const int n_tiles = (grp->k_cap_max + kTileRows - 1) / kTileRows;   // slot stride of the partials
  const int tiles = (k_cap + kTileRows - 1) / kTileRows;
  const size_t smem = sizeof(float) * (kSlab * (kTileRows + 4) + kSlab * (DH + 4) + kTileRows * (DH + 1) +
                                       kMaxRep * DH + kMaxRep * kTileRows + 2 * kMaxRep) +
                      sizeof(int) * 2 * kTileRows;
  cudaError_t e = ensure_dyn_smem<recon_attend_tile_kernel<DH>>(smem, grp->device);
  if (e != cudaSuccess) return e;
  recon_attend_tile_kernel<DH><<<dim3(tiles, problems), kThreads, smem, s>>>(dev, l0, q, sel_idx, sel_cnt, k_cap,
                                                                            n_tiles);
  count_launch(kFamTile);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  merge_kernel<DH><<<problems * dev.n_rep, DH, 0, s>>>(dev, l0, sel_cnt, k_cap, n_tiles, kTileRows, out, lse);
  count_launch(kFamTile);
  return cudaGetLastError();
}

}  // namespace

size_t attend_part_floats(const xkv_group* grp) {
  const xkv_group_config& c = grp->cfg;
  const size_t problems = (size_t)c.G * c.batch * c.H_kv;
  const size_t n_tiles = ((size_t)grp->k_cap_max + kTileRows - 1) / kTileRows;
  return problems * n_tiles * (size_t)(c.H_q / c.H_kv) * (c.d_h + 2);
}

cudaError_t launch_reconstruct_attend(const xkv_group* grp, int l0, int l1, const __nv_bfloat16* q,
                                      const int32_t* sel_idx, const int32_t* sel_cnt, int k_cap,
                                      __nv_bfloat16* out, float* lse, cudaStream_t s) {
  if (grp->dev.d_h == 128) return launch_t<128>(grp, l0, l1, q, sel_idx, sel_cnt, k_cap, out, lse, s);
  return launch_t<64>(grp, l0, l1, q, sel_idx, sel_cnt, k_cap, out, lse, s);
}

}  // namespace xkv
