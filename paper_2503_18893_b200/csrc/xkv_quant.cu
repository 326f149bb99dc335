// Round-to-nearest quantisation of the factorised cache (App. "Integrate with Quantization": "a simple
// round-to-nearest (RTN) quantization method to the compressed cache"; 4 bits give 8.03x -> 25.7x, i.e. 5 stored
// bits per scalar).  Groups of 32 consecutive scalars of a row share a bf16 scale and a bf16 offset:
//   zero = bf16(min), scale = bf16((max - min) / 15), code = clip(rint((x - zero) / scale), 0, 15)   (fp32, IEEE)
//   x_hat = bf16(code * scale + zero)                                   (one rounding of the exact value)
// (4 bits; the 3-bit variant divides by 7, clips at 7 and stores 16-byte records, see dequant_group3.)
// Storage: codes, 4 bits each, [rows][cols/2] bytes; inside every 32-bit word (8 consecutive scalars e0..e7) the
// low half holds e0, e2, e4, e6 and the high half e1, e3, e5, e7 (nibble k of each half), so that
// (word >> 4k) & 0x000F000F is the pair (e_2k, e_2k+1) in the two halves of a register -- the form the packed
// bf16 arithmetic of the gather wants.  meta, [rows][cols/32] 32-bit words: scale in the low half, offset in the high.
#include "xkv_internal.cuh"
#include "xkv_ptx.cuh"

namespace xkv {

namespace {

constexpr int kQuantThreads = 256;

// One thread per group of 32 scalars.
__global__ void __launch_bounds__(kQuantThreads)
quantize_rtn4_kernel(const __nv_bfloat16* __restrict__ x, long long n_groups, uint4* __restrict__ codes,
                     uint32_t* __restrict__ meta) {
  const long long gidx = (long long)blockIdx.x * kQuantThreads + threadIdx.x;
  if (gidx >= n_groups) return;
  const uint4* src = reinterpret_cast<const uint4*>(x + gidx * 32);
  float v[32];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint4 u = src[i];
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) { v[8 * i + 2 * e] = __uint_as_float(w[e] << 16); v[8 * i + 2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u); }
  }
  float lo = v[0], hi = v[0];
#pragma unroll
  for (int i = 1; i < 32; ++i) { lo = fminf(lo, v[i]); hi = fmaxf(hi, v[i]); }
  const __nv_bfloat16 zb = __float2bfloat16_rn(lo);
  const __nv_bfloat16 sb = __float2bfloat16_rn(__fdiv_rn(__fsub_rn(hi, lo), 15.0f));
  const float zero = __bfloat162float(zb), scale = __bfloat162float(sb);
  uint32_t word[4];
#pragma unroll
  for (int wi = 0; wi < 4; ++wi) {
    uint32_t w = 0;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      float q = 0.0f;
      if (scale > 0.0f) q = rintf(__fdiv_rn(__fsub_rn(v[8 * wi + e], zero), scale));     // ties to even
      q = fminf(fmaxf(q, 0.0f), 15.0f);
      const uint32_t c = (uint32_t)q;
      w |= c << (4 * (e >> 1) + 16 * (e & 1));
    }
    word[wi] = w;
  }
  codes[gidx] = make_uint4(word[0], word[1], word[2], word[3]);
  meta[gidx] = (uint32_t)__bfloat16_as_ushort(sb) | ((uint32_t)__bfloat16_as_ushort(zb) << 16);
}

// x_hat of one group per thread: bf16(code * scale + zero) with a single rounding (the packed bf16 fused
// multiply-add rounds the exact value once; small integers are exact in bf16).
__global__ void __launch_bounds__(kQuantThreads)
dequantize_rtn4_kernel(const uint4* __restrict__ codes, const uint32_t* __restrict__ meta, long long n_groups,
                       uint4* __restrict__ x) {
  const long long gidx = (long long)blockIdx.x * kQuantThreads + threadIdx.x;
  if (gidx >= n_groups) return;
  const uint4 cw = codes[gidx];
  const uint32_t m = meta[gidx];
  const uint32_t w[4] = {cw.x, cw.y, cw.z, cw.w};
  uint32_t o[16];
#pragma unroll
  for (int wi = 0; wi < 4; ++wi) ptx::dequant_word(w[wi], m, &o[4 * wi]);
  uint4* dst = x + gidx * 4;
#pragma unroll
  for (int i = 0; i < 4; ++i) dst[i] = make_uint4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
}

// The 3-bit variant: 16-byte records {meta, w0, w1, w2} per group (layout beside dequant_group3).
__global__ void __launch_bounds__(kQuantThreads)
quantize_rtn3_kernel(const __nv_bfloat16* __restrict__ x, long long n_groups, uint4* __restrict__ rec) {
  const long long gidx = (long long)blockIdx.x * kQuantThreads + threadIdx.x;
  if (gidx >= n_groups) return;
  const uint4* src = reinterpret_cast<const uint4*>(x + gidx * 32);
  float v[32];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const uint4 u = src[i];
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) { v[8 * i + 2 * e] = __uint_as_float(w[e] << 16); v[8 * i + 2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u); }
  }
  float lo = v[0], hi = v[0];
#pragma unroll
  for (int i = 1; i < 32; ++i) { lo = fminf(lo, v[i]); hi = fmaxf(hi, v[i]); }
  const __nv_bfloat16 zb = __float2bfloat16_rn(lo);
  const __nv_bfloat16 sb = __float2bfloat16_rn(__fdiv_rn(__fsub_rn(hi, lo), 7.0f));
  const float zero = __bfloat162float(zb), scale = __bfloat162float(sb);
  uint32_t word[3] = {0u, 0u, 0u};
#pragma unroll
  for (int e = 0; e < 32; ++e) {
    float q = 0.0f;
    if (scale > 0.0f) q = rintf(__fdiv_rn(__fsub_rn(v[e], zero), scale));       // ties to even
    q = fminf(fmaxf(q, 0.0f), 7.0f);
    const uint32_t c = (uint32_t)q;
    if (e < 30) {
      const int j = e / 10, k = (e % 10) >> 1;
      word[j] |= c << (3 * k + 16 * (e & 1));
    } else {
      const int sh = e == 30 ? 15 : 31;
      word[0] |= (c & 1u) << sh; word[1] |= ((c >> 1) & 1u) << sh; word[2] |= ((c >> 2) & 1u) << sh;
    }
  }
  rec[gidx] = make_uint4((uint32_t)__bfloat16_as_ushort(sb) | ((uint32_t)__bfloat16_as_ushort(zb) << 16), word[0], word[1], word[2]);
}

__global__ void __launch_bounds__(kQuantThreads)
dequantize_rtn3_kernel(const uint4* __restrict__ rec, long long n_groups, uint4* __restrict__ x) {
  const long long gidx = (long long)blockIdx.x * kQuantThreads + threadIdx.x;
  if (gidx >= n_groups) return;
  const uint4 r = rec[gidx];
  uint32_t o[16];
  ptx::dequant_group3(r.x, r.y, r.z, r.w, o);
  uint4* dst = x + gidx * 4;
#pragma unroll
  for (int i = 0; i < 4; ++i) dst[i] = make_uint4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
}

}  // namespace

cudaError_t launch_quantize_rtn3(const __nv_bfloat16* x, long long rows, int cols, void* rec, cudaStream_t s) {
  const long long n_groups = rows * (cols / 32);
  if (n_groups == 0) return cudaSuccess;
  const long long blocks = (n_groups + kQuantThreads - 1) / kQuantThreads;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
  quantize_rtn3_kernel<<<(unsigned)blocks, kQuantThreads, 0, s>>>(x, n_groups, (uint4*)rec);
  count_launch(kFamPrep);
  return cudaGetLastError();
}

cudaError_t launch_dequantize_rtn3(const void* rec, long long rows, int cols, __nv_bfloat16* x, cudaStream_t s) {
  const long long n_groups = rows * (cols / 32);
  if (n_groups == 0) return cudaSuccess;
  const long long blocks = (n_groups + kQuantThreads - 1) / kQuantThreads;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
  dequantize_rtn3_kernel<<<(unsigned)blocks, kQuantThreads, 0, s>>>((const uint4*)rec, n_groups, (uint4*)x);
  count_launch(kFamPrep);
  return cudaGetLastError();
}

cudaError_t launch_quantize_rtn4(const __nv_bfloat16* x, long long rows, int cols, void* codes, void* meta, cudaStream_t s) {
  const long long n_groups = rows * (cols / 32);
  if (n_groups == 0) return cudaSuccess;
  const long long blocks = (n_groups + kQuantThreads - 1) / kQuantThreads;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
  quantize_rtn4_kernel<<<(unsigned)blocks, kQuantThreads, 0, s>>>(x, n_groups, (uint4*)codes, (uint32_t*)meta);
  count_launch(kFamPrep);
  return cudaGetLastError();
}

cudaError_t launch_dequantize_rtn4(const void* codes, const void* meta, long long rows, int cols, __nv_bfloat16* x,
                                   cudaStream_t s) {
  const long long n_groups = rows * (cols / 32);
  if (n_groups == 0) return cudaSuccess;
  const long long blocks = (n_groups + kQuantThreads - 1) / kQuantThreads;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
  dequantize_rtn4_kernel<<<(unsigned)blocks, kQuantThreads, 0, s>>>((const uint4*)codes, (const uint32_t*)meta, n_groups,
                                                                     (uint4*)x);
  count_launch(kFamPrep);
  return cudaGetLastError();
}

}  // namespace xkv
