// Landmark-guided top-k chunk selection (App. B.1, Algorithm 2) in two kernels:
//   score_pool_kernel  lines 2-3: streams every landmark once (HBM bound), fp32 scores in the canonical
//                      order, max-pool over the query heads of each KV head;
//   topk_kernel        lines 1,4: exact k_ch-th largest pooled score by radix select, then an ordered
//                      compaction (ties to the lowest chunk index, output ascending) and expansion of
//                      chunk ids to token rows.
#include <cuda.h>
#include <math.h>

#include <mutex>

#include "xkv_internal.cuh"
#include "xkv_ptx.cuh"

namespace xkv {

namespace {

constexpr int kScoreRows = kLandmarkBoxRows;   // landmark rows (chunks) per CTA
constexpr int kScoreThreads = 32;    // two rows per thread
constexpr uint32_t kWaitLimit = 1u << 22;

using namespace ptx;

// Bounded wait: returns false if the phase did not complete within `limit` polls.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, uint32_t limit = kWaitLimit) {
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
  }
  return false;
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}

// Order-preserving map float -> uint32 (larger float = larger key), with -0 folded onto +0.
__device__ __forceinline__ uint32_t score_key(float f) {
  uint32_t u = __float_as_uint(f);
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// One pass over the staged tile for HB query heads; returns per-row max of the scaled scores.
template <int DH, int HB>
__device__ __forceinline__ void score_pass(uint32_t tile, const float* __restrict__ qs, int row0, float s,
                                           float& best0, float& best1) {
  float acc0[HB], acc1[HB];
#pragma unroll
  for (int h = 0; h < HB; ++h) { acc0[h] = 0.0f; acc1[h] = 0.0f; }
  const uint32_t sw = (uint32_t)(row0 & 7);
  const uint32_t a0 = tile + (uint32_t)row0 * 128u;
  const uint32_t a1 = a0 + (uint32_t)kScoreThreads * 128u;
#pragma unroll 4
  for (int cc = 0; cc < DH / 8; ++cc) {
    const uint32_t off = (uint32_t)(cc >> 3) * (kScoreRows * 128u) + ((((uint32_t)cc & 7u) ^ sw) << 4);
    const uint4 va = lds128(a0 + off);
    const uint4 vb = lds128(a1 + off);
    const uint32_t wa[4] = {va.x, va.y, va.z, va.w};
    const uint32_t wb[4] = {vb.x, vb.y, vb.z, vb.w};
    float qv[HB][8];
#pragma unroll
    for (int h = 0; h < HB; ++h) {
      const float4 q0 = *reinterpret_cast<const float4*>(qs + h * DH + cc * 8);
      const float4 q1 = *reinterpret_cast<const float4*>(qs + h * DH + cc * 8 + 4);
      qv[h][0] = q0.x; qv[h][1] = q0.y; qv[h][2] = q0.z; qv[h][3] = q0.w;
      qv[h][4] = q1.x; qv[h][5] = q1.y; qv[h][6] = q1.z; qv[h][7] = q1.w;
    }
    // element by element (ascending i, the canonical order of every sum), all heads and both rows per element: the
    // 2 * HB multiply-adds of an element are independent of one another
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float xa0 = __uint_as_float(wa[w] << 16), xb0 = __uint_as_float(wb[w] << 16);
      const float xa1 = __uint_as_float(wa[w] & 0xffff0000u), xb1 = __uint_as_float(wb[w] & 0xffff0000u);
#pragma unroll
      for (int h = 0; h < HB; ++h) {
        acc0[h] = fmaf(qv[h][2 * w], xa0, acc0[h]);
        acc1[h] = fmaf(qv[h][2 * w], xb0, acc1[h]);
      }
#pragma unroll
      for (int h = 0; h < HB; ++h) {
        acc0[h] = fmaf(qv[h][2 * w + 1], xa1, acc0[h]);
        acc1[h] = fmaf(qv[h][2 * w + 1], xb1, acc1[h]);
      }
    }
  }
#pragma unroll
  for (int h = 0; h < HB; ++h) {
    best0 = fmaxf(best0, acc0[h] * s);
    best1 = fmaxf(best1, acc1[h] * s);
  }
}

// grid.x = ceil(n_c / kScoreRows) tiles, grid.y = (layers in call) * batch * H_kv problems.
template <int DH, int HMAX>
__global__ void __launch_bounds__(kScoreThreads)
score_pool_kernel(const __grid_constant__ CUtensorMap tmap, GroupDev dev, const __nv_bfloat16* __restrict__ q,
                  int l0) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_storage;
  const uint32_t tile = (smem_u32(smem_raw) + 1023u) & ~1023u;
  float* qs = reinterpret_cast<float*>(smem_raw + (tile - smem_u32(smem_raw)) + (DH / 64) * kScoreRows * 128);
  const uint32_t bar = smem_u32(&bar_storage);

  const int g = blockIdx.y % dev.H_kv;
  const int b = (blockIdx.y / dev.H_kv) % dev.batch;
  const int l = l0 + blockIdx.y / (dev.H_kv * dev.batch);
  const int j0 = blockIdx.x * kScoreRows;
  const long long prob_lm = ((long long)b * dev.G + l) * dev.H_kv + g;       // landmark order
  const long long prob_out = ((long long)l * dev.batch + b) * dev.H_kv + g;  // [G][batch][H_kv] order

  // fault injection (tests of the give-up path): no load is issued, so the wait below must run into its limit
  const bool no_load = (dev.inject & XKV_INJECT_SCAN_NO_LOAD) != 0u;
  // A handle's landmarks are constant while the handle is used (the caller's contract), so their loads may start
  // before the kernel launched before this one has finished; the queries may come from that kernel and are
  // read after the dependency wait.  Without a handle (the allocation-free entry point) nothing is known about
  // the landmarks, and the loads wait too.
  const bool early = dev.lm_const != 0;
  if (!early) grid_dependency_wait();
  if (threadIdx.x == 0) {          // the thread that initialises the barrier also issues the loads: nothing to wait for
    mbar_init(bar, 1);
    fence_mbar_init();
    if (!no_load) {
      mbar_expect_tx(bar, (uint32_t)((DH / 64) * kScoreRows * 128));
      const int y = (int)(prob_lm * dev.n_c + j0);
      // every landmark is read once per call: first in line for eviction, so that the stream does not push the
      // pooled scores (written below, read by the top-k) and the gathered basis rows out of L2
      const uint64_t pol = l2_policy_evict_first();
#pragma unroll
      for (int bx = 0; bx < DH / 64; ++bx) tma_load_2d_hint(tile + bx * kScoreRows * 128, &tmap, bx * 64, y, bar, pol);
    }
  }
  if (early) grid_dependency_wait();
  grid_dependency_launch();
  // queries of this KV head, widened to fp32 while the landmarks are in flight
  const __nv_bfloat16* qg = q + (((long long)l * dev.batch + b) * dev.H_q + (long long)g * dev.n_rep) * DH;
  // (all the 16-byte loads of a lane are issued before the first is used: one trip to L2, not one per element)
  {
    const uint4* qv = reinterpret_cast<const uint4*>(qg);
    const int n_pieces = dev.n_rep * (DH / 8);
    constexpr int kMaxPieces = kMaxRep * (DH / 8) / kScoreThreads;   // at most kMaxRep query heads per KV head
    uint4 u[kMaxPieces];
#pragma unroll
    for (int i = 0; i < kMaxPieces; ++i) {
      const int pc = threadIdx.x + i * kScoreThreads;
      u[i] = pc < n_pieces ? qv[pc] : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int i = 0; i < kMaxPieces; ++i) {
      const int pc = threadIdx.x + i * kScoreThreads;
      if (pc < n_pieces) {
        float4 a, b;
        a.x = __uint_as_float(u[i].x << 16); a.y = __uint_as_float(u[i].x & 0xffff0000u);
        a.z = __uint_as_float(u[i].y << 16); a.w = __uint_as_float(u[i].y & 0xffff0000u);
        b.x = __uint_as_float(u[i].z << 16); b.y = __uint_as_float(u[i].z & 0xffff0000u);
        b.z = __uint_as_float(u[i].w << 16); b.w = __uint_as_float(u[i].w & 0xffff0000u);
        *reinterpret_cast<float4*>(qs + pc * 8) = a;
        *reinterpret_cast<float4*>(qs + pc * 8 + 4) = b;
      }
    }
  }
  __syncthreads();

  if (!mbar_wait_bounded(bar, 0, no_load ? 1024u : kWaitLimit)) {
    if (threadIdx.x == 0) atomicOr(dev.flags, XKV_FLAG_TIMEOUT);
    // The boxes may still be on their way into this CTA's shared memory, which the next CTA on the SM would
    // inherit: stay for a second (again bounded) wait before giving the memory up.
    if (!no_load) (void)mbar_wait_bounded(bar, 0);
    return;
  }
  float best0 = -INFINITY, best1 = -INFINITY;
  const int row0 = threadIdx.x;
  // heads in passes of HMAX: a pass reads the tile once for all its heads.  The kernel for up to four heads per
  // KV head is kept apart from the wider one: its code is smaller, and the scan is sensitive to that.
  for (int h0 = 0; h0 < dev.n_rep; h0 += HMAX) {
    const int hb = min(HMAX, dev.n_rep - h0);
    const float* qh = qs + h0 * DH;
    if constexpr (HMAX == 8) {
      if (hb == 8) { score_pass<DH, 8>(tile, qh, row0, dev.sel_scale, best0, best1); continue; }
      if (hb == 7) { score_pass<DH, 7>(tile, qh, row0, dev.sel_scale, best0, best1); continue; }
      if (hb == 6) { score_pass<DH, 6>(tile, qh, row0, dev.sel_scale, best0, best1); continue; }
      if (hb == 5) { score_pass<DH, 5>(tile, qh, row0, dev.sel_scale, best0, best1); continue; }
    }
    if (hb == 4) score_pass<DH, 4>(tile, qh, row0, dev.sel_scale, best0, best1);
    else if (hb == 3) score_pass<DH, 3>(tile, qh, row0, dev.sel_scale, best0, best1);
    else if (hb == 2) score_pass<DH, 2>(tile, qh, row0, dev.sel_scale, best0, best1);
    else score_pass<DH, 1>(tile, qh, row0, dev.sel_scale, best0, best1);
  }
  // the pooled scores are handed on as order-preserving integer keys (what the top-k compares)
  uint32_t* dst = reinterpret_cast<uint32_t*>(dev.pooled) + prob_out * dev.n_c;
  if (j0 + row0 < dev.n_c) dst[j0 + row0] = score_key(best0);
  if (j0 + row0 + kScoreThreads < dev.n_c) dst[j0 + row0 + kScoreThreads] = score_key(best1);
}

// ---------------------------------------------------------------------------------------------

constexpr int kTopkThreads = 1024;
constexpr int kTopkItems = 16;    // consecutive chunks per thread and super-block
constexpr int kTopkBins = 2048;   // histogram bins per radix pass
constexpr int kTopkCand = 256;    // at most this many keys are ranked against one another directly

// Keys of this thread's 16 consecutive chunks of one super-block (0 beyond n_c; callers mask by index).
// sign == 0: the array already holds keys (the landmark scan writes them); else it holds floats and the key is
// that of sign * value.
template <int ITEMS>
__device__ __forceinline__ void load_keys(const float* __restrict__ S, int j0, int n_c, float sign, uint32_t (&key)[ITEMS]) {
  const bool keyed = sign == 0.0f;
  if (j0 + ITEMS <= n_c && ((n_c & 3) == 0)) {
    const float4* p = reinterpret_cast<const float4*>(S + j0);
#pragma unroll
    for (int i = 0; i < ITEMS / 4; ++i) {
      const float4 v = p[i];
      const float f[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) key[4 * i + e] = keyed ? __float_as_uint(f[e]) : score_key(f[e] * sign);
    }
  } else {
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
      const float f = (j0 + i < n_c) ? S[j0 + i] : 0.0f;
      key[i] = (j0 + i < n_c) ? (keyed ? __float_as_uint(f) : score_key(f * sign)) : 0u;
    }
  }
}

// One CTA per (layer, sequence, KV head).  grid.x = problems of the call.
// Exact k_ch-th largest key by a radix select whose bins subdivide the range that still contains it
// (first the [min, max] range of all keys, then the chosen bin, ...: at most three 11-bit passes), followed
// by an ordered compaction.  CACHED: n_c fits one super-block and the keys stay in registers.
template <bool CACHED>
__global__ void __launch_bounds__(kTopkThreads)
topk_kernel(GroupDev dev, int l0, int k_ch, int k_cap, const int32_t* __restrict__ outliers, int n_out, float sign,
            int32_t* __restrict__ sel_idx, int32_t* __restrict__ sel_cnt) {
  __shared__ __align__(16) uint32_t hist[kTopkBins];
  __shared__ uint32_t warp_tot[kTopkThreads / 32];
  __shared__ uint32_t warp_min[kTopkThreads / 32], warp_max[kTopkThreads / 32];
  __shared__ uint32_t sh_a, sh_b, sh_c;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per_layer = dev.batch * dev.H_kv;
  const long long prob = (long long)l0 * per_layer + blockIdx.x;     // [G][batch][H_kv] order
  const float* __restrict__ S = dev.pooled + prob * dev.n_c;
  int32_t* __restrict__ out = sel_idx + prob * k_cap;
  const int n_c = dev.n_c, c = dev.c, T = dev.T;
  const int super = kTopkThreads * kTopkItems;
  const bool out_vec = (reinterpret_cast<uintptr_t>(out) & 15u) == 0;   // 16-byte stores of the row ids

  grid_dependency_wait();                      // the pooled scores come from the kernel launched before
  grid_dependency_launch();
  uint32_t creg[kTopkItems];
  if (CACHED) load_keys(S, tid * kTopkItems, n_c, sign, creg);

  uint32_t thr = 0, need_eq = 0;
  const bool all = (k_ch >= n_c);
  if (!all) {
    // ---- range of the keys
    uint32_t kmin = 0xffffffffu, kmax = 0u;
    for (int base = 0; base < n_c; base += super) {
      uint32_t key[kTopkItems];
      const int j0 = base + tid * kTopkItems;
      if (CACHED) {
#pragma unroll
        for (int i = 0; i < kTopkItems; ++i) key[i] = creg[i];
      } else {
        load_keys(S, j0, n_c, sign, key);
      }
#pragma unroll
      for (int i = 0; i < kTopkItems; ++i) {
        if (j0 + i < n_c) { kmin = min(kmin, key[i]); kmax = max(kmax, key[i]); }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
      kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
    }
    if (lane == 0) { warp_min[warp] = kmin; warp_max[warp] = kmax; }
    __syncthreads();
    kmin = warp_min[lane]; kmax = warp_max[lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
      kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
    }
    // ---- radix passes over the window [lo, lo + span]
    uint32_t lo = kmin, span = kmax - kmin, need = (uint32_t)k_ch;
    for (;;) {
      const int bits = 32 - __clz(span);                      // span < 2^bits
      const int sh = bits > 11 ? bits - 11 : 0;
      for (int i = tid; i < kTopkBins; i += kTopkThreads) hist[i] = 0;
      __syncthreads();
      for (int base = 0; base < n_c; base += super) {
        uint32_t key[kTopkItems];
        const int j0 = base + tid * kTopkItems;
        if (CACHED) {
#pragma unroll
          for (int i = 0; i < kTopkItems; ++i) key[i] = creg[i];
        } else {
          load_keys(S, j0, n_c, sign, key);
        }
#pragma unroll
        for (int i = 0; i < kTopkItems; ++i) {
          const uint32_t rel = key[i] - lo;
          if (j0 + i < n_c && key[i] >= lo && rel <= span) atomicAdd(&hist[rel >> sh], 1u);
        }
      }
      __syncthreads();
      // suffix counts from the top bin down: thread t owns bins 2t, 2t+1
      const uint32_t h0 = hist[2 * tid], h1 = hist[2 * tid + 1];
      const uint32_t mine = h0 + h1;
      uint32_t suf = mine;                                     // inclusive over higher lanes of the warp
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_down_sync(0xffffffffu, suf, o);
        if (lane + o < 32) suf += v;
      }
      if (lane == 0) warp_tot[warp] = suf;
      __syncthreads();
      if (warp == 0) {
        const uint32_t t = warp_tot[lane];
        uint32_t ws = t;                                       // inclusive over higher warps
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t v = __shfl_down_sync(0xffffffffu, ws, o);
          if (lane + o < 32) ws += v;
        }
        warp_tot[lane] = ws - t;                               // keys in bins of higher warps
      }
      __syncthreads();
      const uint32_t above = warp_tot[warp] + (suf - mine);    // keys in bins above 2t+1
      if (above < need && above + mine >= need) {              // exactly one thread
        if (above + h1 >= need) { sh_a = 2 * tid + 1; sh_b = need - above; sh_c = h1; }
        else { sh_a = 2 * tid; sh_b = need - above - h1; sh_c = h0; }
      }
      __syncthreads();
      const uint32_t bsel = sh_a, in_bin = sh_c;
      need = sh_b;
      lo += bsel << sh;
      span = min(span - (bsel << sh), (sh ? (1u << sh) : 1u) - 1u);
      __syncthreads();
      if (sh == 0) { thr = lo; need_eq = need; break; }
      if (in_bin <= (uint32_t)kTopkCand) {
        // Few keys are left in the window: collect them (in any order) and rank them against one another.
        // The `need`-th largest of them is the threshold; need_eq = how many keys equal to it are still wanted.
        uint32_t* cand = hist;
        if (tid == 0) sh_a = 0;
        __syncthreads();
        for (int base = 0; base < n_c; base += super) {
          uint32_t key[kTopkItems];
          const int j0 = base + tid * kTopkItems;
          if (CACHED) {
#pragma unroll
            for (int i = 0; i < kTopkItems; ++i) key[i] = creg[i];
          } else {
            load_keys(S, j0, n_c, sign, key);
          }
          // this thread's candidates as a bit mask; the warp reserves room for all of its candidates with one atomic
          uint32_t cm = 0;
#pragma unroll
          for (int i = 0; i < kTopkItems; ++i) {
            if (j0 + i < n_c && key[i] >= lo && key[i] - lo <= span) cm |= 1u << i;
          }
          const uint32_t mine_c = (uint32_t)__popc(cm);
          if (__any_sync(0xffffffffu, cm != 0u)) {
            uint32_t inc = mine_c;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
              const uint32_t v = __shfl_up_sync(0xffffffffu, inc, o);
              if (lane >= o) inc += v;
            }
            uint32_t wbase = 0;
            if (lane == 31) wbase = atomicAdd(&sh_a, inc);
            wbase = __shfl_sync(0xffffffffu, wbase, 31);
            uint32_t at = wbase + inc - mine_c;
#pragma unroll
            for (int i = 0; i < kTopkItems; ++i) {
              if ((cm >> i) & 1u) cand[at++] = key[i];
            }
          }
        }
        __syncthreads();
        const uint32_t n_cand = sh_a;                          // == in_bin
        __syncthreads();
        if ((uint32_t)tid < n_cand) {
          const uint32_t mykey = cand[tid];
          uint32_t gt = 0, eq = 0;
          const uint32_t n4 = n_cand & ~3u;
          const uint4* c4 = reinterpret_cast<const uint4*>(cand);
#pragma unroll 4
          for (uint32_t i = 0; i < n4; i += 4) {
            const uint4 v = c4[i >> 2];
            gt += (v.x > mykey ? 1u : 0u) + (v.y > mykey ? 1u : 0u) + (v.z > mykey ? 1u : 0u) + (v.w > mykey ? 1u : 0u);
            eq += (v.x == mykey ? 1u : 0u) + (v.y == mykey ? 1u : 0u) + (v.z == mykey ? 1u : 0u) + (v.w == mykey ? 1u : 0u);
          }
          for (uint32_t i = n4; i < n_cand; ++i) {
            const uint32_t c2 = cand[i];
            gt += c2 > mykey ? 1u : 0u;
            eq += c2 == mykey ? 1u : 0u;
          }
          if (gt < need && need <= gt + eq) { sh_a = mykey; sh_b = need - gt; }   // equal keys write the same pair
        }
        __syncthreads();
        thr = sh_a;
        need_eq = sh_b;
        __syncthreads();
        break;
      }
    }
  }

  // Ordered compaction: chunk j is taken if key > thr, or key == thr and fewer than need_eq equal
  // keys precede it, or (Algorithm 2 line 5) it is one of the head's static outlier chunks.  Positions follow
  // ascending j.
  __shared__ uint32_t obits[kTopkThreads * kTopkItems / 32];   // outlier chunks of the current super-block
  __shared__ uint32_t sh_last_taken;
  // packed (low 16 bits, high 16 bits) exclusive prefix over the CTA in thread order; the total goes to sh_a
  auto block_scan = [&](uint32_t mine) -> uint32_t {
    uint32_t inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t v = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += v;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    if (warp == 0) {
      const uint32_t t = warp_tot[lane];
      uint32_t ti = t;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_up_sync(0xffffffffu, ti, o);
        if (lane >= o) ti += v;
      }
      warp_tot[lane] = ti - t;                      // exclusive prefix of warp totals
      if (lane == 31) sh_a = ti;                    // super-block total
    }
    __syncthreads();
    return inc - mine + warp_tot[warp];
  };
  auto write_chunk = [&](uint32_t pos, int j) {
    const int rows = min(c, T - j * c);
    if (c == 8 && rows == 8 && out_vec) {
      int4* o4 = reinterpret_cast<int4*>(out + (size_t)pos * 8);
      o4[0] = make_int4(j * 8, j * 8 + 1, j * 8 + 2, j * 8 + 3);
      o4[1] = make_int4(j * 8 + 4, j * 8 + 5, j * 8 + 6, j * 8 + 7);
    } else {
      for (int t = 0; t < rows; ++t) out[(size_t)pos * c + t] = j * c + t;
    }
  };
  const int32_t* outl = nullptr;                    // this problem's outlier chunk ids
  if (n_out > 0) {
    outl = outliers + (size_t)prob * (size_t)n_out;          // [G][batch][H_kv][n_out], like sel_idx
    if (tid == 0) sh_last_taken = 0;
  }
  uint32_t run_gt = 0, run_eq = 0;                  // totals of the super-blocks already done
  uint32_t run_taken = 0;                           // chunks written so far (outlier path)
  uint32_t last_key = 0;
  for (int base = 0; base < n_c; base += super) {
    const int j0 = base + tid * kTopkItems;
    uint32_t gtm = 0, eqm = 0;                      // bit i set: item i is > / == thr
    if (all) {
#pragma unroll
      for (int i = 0; i < kTopkItems; ++i) if (j0 + i < n_c) gtm |= 1u << i;
    } else {
      uint32_t key[kTopkItems];
      if (CACHED) {
#pragma unroll
        for (int i = 0; i < kTopkItems; ++i) key[i] = creg[i];
      } else {
        load_keys(S, j0, n_c, sign, key);
      }
#pragma unroll
      for (int i = 0; i < kTopkItems; ++i) {
        if (j0 + i < n_c) {
          gtm |= (key[i] > thr ? 1u : 0u) << i;
          eqm |= (key[i] == thr ? 1u : 0u) << i;
          if (j0 + i == n_c - 1) last_key = key[i];
        }
      }
    }
    const uint32_t mine = (uint32_t)__popc(gtm) | ((uint32_t)__popc(eqm) << 16);
    const uint32_t excl = block_scan(mine);
    const uint32_t tot1 = sh_a;
    uint32_t gt_before = run_gt + (excl & 0xffffu);
    uint32_t eq_before = run_eq + (excl >> 16);
    if (n_out == 0) {
      // Only a few percent of the chunks are taken.  Output position of a taken chunk = taken chunks before it.
      // If the super-block's taken chunks fit the list (the histogram's memory, free by now), their ids go there
      // first and the whole CTA then writes the rows, consecutive threads to consecutive words; else every thread
      // writes the rows of its own chunks.
      const uint32_t blk_gt = tot1 & 0xffffu, blk_eq = tot1 >> 16;
      const uint32_t eq_room = need_eq > run_eq ? need_eq - run_eq : 0u;        // equal keys this super-block may still take
      const uint32_t blk_taken = blk_gt + min(blk_eq, eq_room);
      const uint32_t pos0 = run_gt + min(run_eq, need_eq);                       // chunks written by earlier super-blocks
      const bool listed = blk_taken <= (uint32_t)kTopkBins;
      uint32_t m = gtm | eqm;
      while (m) {
        const int i = __ffs(m) - 1;
        m &= m - 1;
        const uint32_t below = (1u << i) - 1u;
        const uint32_t g_b = gt_before + (uint32_t)__popc(gtm & below), e_b = eq_before + (uint32_t)__popc(eqm & below);
        const bool is_gt = (gtm >> i) & 1u;
        if (is_gt || e_b < need_eq) {
          const uint32_t pos = g_b + min(e_b, need_eq);
          if (listed) hist[pos - pos0] = (uint32_t)(j0 + i); else write_chunk(pos, j0 + i);
        }
      }
      if (listed) {
        __syncthreads();
        if (c == 8) {
          for (uint32_t w = (uint32_t)tid; w < blk_taken * 8u; w += kTopkThreads) {
            const int row = (int)hist[w >> 3] * 8 + (int)(w & 7u);
            if (row < T) out[(size_t)pos0 * 8 + w] = row;
          }
        } else {
          for (uint32_t w = (uint32_t)tid; w < blk_taken * (uint32_t)c; w += kTopkThreads) {
            const uint32_t e = w / (uint32_t)c, t = w - e * (uint32_t)c;
            const int row = (int)hist[e] * c + (int)t;
            if (row < T) out[(size_t)pos0 * c + w] = row;
          }
        }
      }
    } else {
      // membership in the top-k first, then the union with the outlier chunks, then positions over the union
      uint32_t takem = 0;
#pragma unroll
      for (int i = 0; i < kTopkItems; ++i) {
        const bool is_gt = (gtm >> i) & 1u, is_eq = (eqm >> i) & 1u;
        if (is_gt || (is_eq && eq_before < need_eq)) takem |= 1u << i;
        gt_before += is_gt ? 1u : 0u;
        eq_before += is_eq ? 1u : 0u;
      }
      for (int w = tid; w < super / 32; w += kTopkThreads) obits[w] = 0u;
      __syncthreads();                                // also: everybody has read sh_a and warp_tot of the first scan
      const int hi = min(base + super, n_c);
      for (int o = tid; o < n_out; o += kTopkThreads) {
        const int jo = outl[o];
        if (jo >= base && jo < hi) atomicOr(&obits[(jo - base) >> 5], 1u << ((jo - base) & 31));
      }
      __syncthreads();
      static_assert(kTopkItems == 16, "two threads share one word of the outlier bitmap");
      takem |= (obits[tid >> 1] >> ((tid & 1) * 16)) & 0xffffu;
      const uint32_t excl2 = block_scan((uint32_t)__popc(takem));
      uint32_t pos = run_taken + excl2;
#pragma unroll
      for (int i = 0; i < kTopkItems; ++i) {
        if ((takem >> i) & 1u) {
          write_chunk(pos++, j0 + i);
          if (j0 + i == n_c - 1) sh_last_taken = 1u;
        }
      }
      run_taken += sh_a;
    }
    run_gt += tot1 & 0xffffu;
    run_eq += tot1 >> 16;
    __syncthreads();
  }
  // Row count: whole chunks unless the ragged last chunk was taken (it is then the last one).
  // Without outliers: k_ch chunks; the last chunk has the highest index, so it wins a tie only if every equal key fits.
  __shared__ uint32_t sh_last;                    // key of chunk n_c-1, published by the thread that owns it
  {
    const int owner = ((n_c - 1) % super) / kTopkItems;
    if (tid == owner) sh_last = last_key;
    __syncthreads();
  }
  int cnt;
  if (n_out == 0) {
    cnt = (all ? n_c : k_ch) * c;
    bool last_in = all;
    if (!all) last_in = sh_last > thr || (sh_last == thr && run_eq <= need_eq);
    if (last_in) cnt -= (n_c * c - T);
  } else {
    cnt = (int)run_taken * c;
    if (sh_last_taken) cnt -= (n_c * c - T);
  }
  for (int i = cnt + tid; i < k_cap; i += kTopkThreads) out[i] = -1;
  if (tid == 0 && sel_cnt) sel_cnt[prob] = cnt;
}


// ---------------------------------------------------------------------------------------------
// The same selection for n_c <= 16384 chunks (one super-block), organised so that almost all of the work is done
// on a short list instead of on every key.  Each thread holds 16 consecutive keys, split into GPT groups; the
// k_ch-th largest of the group maxima is a lower bound P of the k_ch-th largest key (at least k_ch keys -- those
// maxima -- are >= it), and with k_ch a few percent of n_c only a few percent of the keys pass it.  The keys >= P
// go to a list in shared memory (key, chunk index); the exact k_ch-th largest key is then found on the list by
// the radix select of topk_kernel; membership goes to a bitmap over the chunks (united with the head's outlier
// chunks), whose prefix popcounts give the ascending output positions.  GPT = 0 disables the filter (P = the
// smallest key): chosen by the host when there are fewer groups than k_ch.  ITEMS = 16 keys per thread serve
// n_c <= 16384 chunks, ITEMS = 32 (keys read twice instead of held in registers) n_c <= 32768.  The result is
// identical to topk_kernel's for every input; only the amount of work differs.
// Bin (counted from the top) that holds the `need`-th largest of the keys counted in hist[0..kTopkBins), by a
// suffix sum over the bins; thread t of the TH owns the kTopkBins / TH bins from t * (kTopkBins / TH).  Results in
// sh[0] = bin, sh[1] = rank wanted inside the bin, sh[2] = keys in the bin.  Contains barriers: call it from all threads.
template <int TH>
__device__ __forceinline__ void find_bin(const uint32_t* hist, uint32_t need, uint32_t* warp_tot, uint32_t* sh, int tid) {
  constexpr int BPT = kTopkBins / TH, NWARP = TH / 32;
  static_assert(BPT >= 1 && BPT * TH == kTopkBins, "bins per thread");
  const int lane = tid & 31, warp = tid >> 5;
  uint32_t h[BPT];
  uint32_t mine = 0;
#pragma unroll
  for (int i = 0; i < BPT; ++i) { h[i] = hist[BPT * tid + i]; mine += h[i]; }
  uint32_t suf = mine;                                     // inclusive over higher lanes of the warp
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t v = __shfl_down_sync(0xffffffffu, suf, o);
    if (lane + o < 32) suf += v;
  }
  if (lane == 0) warp_tot[warp] = suf;
  __syncthreads();
  if (warp == 0) {
    const uint32_t t = lane < NWARP ? warp_tot[lane] : 0u;
    uint32_t ws = t;                                       // inclusive over higher warps
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t v = __shfl_down_sync(0xffffffffu, ws, o);
      if (lane + o < 32) ws += v;
    }
    if (lane < NWARP) warp_tot[lane] = ws - t;             // keys in bins of higher warps
  }
  __syncthreads();
  const uint32_t above = warp_tot[warp] + (suf - mine);    // keys in bins above this thread's
  if (above < need && above + mine >= need) {              // exactly one thread
    uint32_t acc = above;
#pragma unroll
    for (int i = BPT - 1; i >= 0; --i) {
      if (acc < need && acc + h[i] >= need) { sh[0] = (uint32_t)(BPT * tid + i); sh[1] = need - acc; sh[2] = h[i]; }
      acc += h[i];
    }
  }
  __syncthreads();
}

template <int GPT, int ITEMS, int TH>
__global__ void __launch_bounds__(TH, 1)
topk_pivot_kernel(GroupDev dev, int l0, int k_ch, int k_cap, const int32_t* __restrict__ outliers, int n_out, float sign,
                  int32_t* __restrict__ sel_idx, int32_t* __restrict__ sel_cnt) {
  extern __shared__ __align__(16) uint8_t pivot_smem[];
  constexpr int kPivotListMax = TH * ITEMS;                              // every key may pass (all keys equal)
  static_assert(kPivotListMax <= 65536 && kPivotListMax / 32 <= TH, "16-bit chunk index, one bitmap word per thread");
  uint32_t* list_key = reinterpret_cast<uint32_t*>(pivot_smem);                    // [kPivotListMax]; later the chunk list
  uint16_t* list_idx = reinterpret_cast<uint16_t*>(list_key + kPivotListMax);      // [kPivotListMax]
  __shared__ __align__(16) uint32_t hist[kTopkBins];
  __shared__ uint32_t take_w[kPivotListMax / 32], eq_w[kPivotListMax / 32];        // bitmaps over the chunks
  __shared__ uint32_t warp_tot[TH / 32];
  __shared__ uint32_t warp_min[TH / 32], warp_max[TH / 32];
  __shared__ uint32_t sh[4];
  __shared__ uint32_t sh_n;

  constexpr int NWARP = TH / 32;
  constexpr int kCand = kTopkCand < TH ? kTopkCand : TH;      // every candidate is ranked by a thread of its own
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int per_layer = dev.batch * dev.H_kv;
  const long long prob = (long long)l0 * per_layer + blockIdx.x;     // [G][batch][H_kv] order
  const float* __restrict__ S = dev.pooled + prob * dev.n_c;
  int32_t* __restrict__ out = sel_idx + prob * k_cap;
  const int n_c = dev.n_c, c = dev.c, T = dev.T;
  constexpr int NW = kPivotListMax / 32;                               // words of a bitmap
  constexpr int NG = GPT == 0 ? 1 : GPT;                               // group maxima kept per thread
  constexpr int GS = ITEMS / NG;                                       // keys per group

  grid_dependency_wait();                      // the pooled scores come from the kernel launched before
  grid_dependency_launch();
  const int j0 = tid * ITEMS;
  const bool all = (k_ch >= n_c);
  uint32_t thr = 0, need_eq = 0;
  for (int w = tid; w < NW; w += TH) { take_w[w] = 0u; eq_w[w] = 0u; }
  if (tid == 0) sh_n = 0;
  if (!all) {
    uint32_t key[ITEMS];
    load_keys(S, j0, n_c, sign, key);
    // ---- extrema of this thread's keys and of its groups
    uint32_t kmin = 0xffffffffu, kmax = 0u;
    uint32_t gmax[NG];
#pragma unroll
    for (int g = 0; g < NG; ++g) gmax[g] = 0u;
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
      if (j0 + i < n_c) {
        kmin = min(kmin, key[i]); kmax = max(kmax, key[i]);
        if (GPT != 0) gmax[i / GS] = max(gmax[i / GS], key[i]);
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
      kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
    }
    if (lane == 0) { warp_min[warp] = kmin; warp_max[warp] = kmax; }
    for (int i = tid; i < kTopkBins; i += TH) hist[i] = 0;
    __syncthreads();
    kmin = lane < NWARP ? warp_min[lane] : 0xffffffffu; kmax = lane < NWARP ? warp_max[lane] : 0u;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
      kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
    }
    // ---- pivot: lower edge of the bin that holds the k_ch-th largest group maximum
    uint32_t P = kmin;
    if (GPT != 0) {
      const uint32_t span1 = kmax - kmin;
      const int bits1 = 32 - __clz(span1);
      const int sh1 = bits1 > 11 ? bits1 - 11 : 0;
#pragma unroll
      for (int g = 0; g < NG; ++g) {
        if (j0 + g * GS < n_c) atomicAdd(&hist[(gmax[g] - kmin) >> sh1], 1u);    // the group has at least one key
      }
      __syncthreads();
      find_bin<TH>(hist, (uint32_t)k_ch, warp_tot, sh, tid);
      P = kmin + (sh[0] << sh1);
      __syncthreads();
    }
    // ---- the keys >= P, with their chunk index, to the list (one shared-memory atomic per warp)
    {
      if (ITEMS > 16) load_keys(S, j0, n_c, sign, key);   // 32 keys are not held across the barriers above: read them again
      uint32_t cm = 0;
#pragma unroll
      for (int i = 0; i < ITEMS; ++i) {
        if (j0 + i < n_c && key[i] >= P) cm |= 1u << i;
      }
      const uint32_t mine_c = (uint32_t)__popc(cm);
      if (__any_sync(0xffffffffu, cm != 0u)) {
        uint32_t inc = mine_c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t v = __shfl_up_sync(0xffffffffu, inc, o);
          if (lane >= o) inc += v;
        }
        uint32_t wbase = 0;
        if (lane == 31) wbase = atomicAdd(&sh_n, inc);
        wbase = __shfl_sync(0xffffffffu, wbase, 31);
        uint32_t at = wbase + inc - mine_c;
#pragma unroll
        for (int i = 0; i < ITEMS; ++i) {
          if ((cm >> i) & 1u) { list_key[at] = key[i]; list_idx[at] = (uint16_t)(j0 + i); ++at; }
        }
      }
    }
    __syncthreads();
    const int n_list = (int)sh_n;                                      // >= k_ch
    // ---- radix select of the k_ch-th largest key on the list: bins subdivide the window [lo, lo + span]
    uint32_t lo = P, span = kmax - P, need = (uint32_t)k_ch;
    for (;;) {
      const int bits = 32 - __clz(span);                               // span < 2^bits
      const int shb = bits > 11 ? bits - 11 : 0;
      for (int i = tid; i < kTopkBins; i += TH) hist[i] = 0;
      __syncthreads();
      for (int e = tid; e < n_list; e += TH) {
        const uint32_t rel = list_key[e] - lo;                         // keys below lo wrap to huge values
        if (rel <= span) atomicAdd(&hist[rel >> shb], 1u);
      }
      __syncthreads();
      find_bin<TH>(hist, need, warp_tot, sh, tid);
      const uint32_t bsel = sh[0], in_bin = sh[2];
      need = sh[1];
      lo += bsel << shb;
      span = min(span - (bsel << shb), (shb ? (1u << shb) : 1u) - 1u);
      __syncthreads();
      if (shb == 0) { thr = lo; need_eq = need; break; }
      if (in_bin <= (uint32_t)kCand) {
        // few keys are left in the window: collect them and rank them against one another
        uint32_t* cand = hist;
        if (tid == 0) sh[3] = 0;
        __syncthreads();
        for (int e = tid; e < n_list; e += TH) {
          const uint32_t kk = list_key[e];
          if (kk - lo <= span) cand[atomicAdd(&sh[3], 1u)] = kk;
        }
        __syncthreads();
        const uint32_t n_cand = sh[3];                                 // == in_bin
        __syncthreads();
        if ((uint32_t)tid < n_cand) {
          const uint32_t mykey = cand[tid];
          uint32_t gt = 0, eq = 0;
          const uint32_t n4 = n_cand & ~3u;
          const uint4* c4 = reinterpret_cast<const uint4*>(cand);
#pragma unroll 4
          for (uint32_t i = 0; i < n4; i += 4) {
            const uint4 v = c4[i >> 2];
            gt += (v.x > mykey ? 1u : 0u) + (v.y > mykey ? 1u : 0u) + (v.z > mykey ? 1u : 0u) + (v.w > mykey ? 1u : 0u);
            eq += (v.x == mykey ? 1u : 0u) + (v.y == mykey ? 1u : 0u) + (v.z == mykey ? 1u : 0u) + (v.w == mykey ? 1u : 0u);
          }
          for (uint32_t i = n4; i < n_cand; ++i) {
            const uint32_t c2 = cand[i];
            gt += c2 > mykey ? 1u : 0u;
            eq += c2 == mykey ? 1u : 0u;
          }
          if (gt < need && need <= gt + eq) { sh[0] = mykey; sh[1] = need - gt; }   // equal keys write the same pair
        }
        __syncthreads();
        thr = sh[0];
        need_eq = sh[1];
        __syncthreads();
        break;
      }
    }
    // ---- membership: keys above the threshold, and (separately) keys equal to it
    for (int e = tid; e < n_list; e += TH) {
      const uint32_t kk = list_key[e];
      const uint32_t j = list_idx[e];
      if (kk > thr) atomicOr(&take_w[j >> 5], 1u << (j & 31u));
      else if (kk == thr) atomicOr(&eq_w[j >> 5], 1u << (j & 31u));
    }
  } else {
    __syncthreads();                                                   // the bitmaps are zeroed
    for (int w = tid; w < NW; w += TH) {
      const int first = w * 32;
      take_w[w] = first + 32 <= n_c ? 0xffffffffu : (first < n_c ? ((1u << (n_c - first)) - 1u) : 0u);
    }
  }
  // Algorithm 2 line 5: the head's static outlier chunks join the set
  if (n_out > 0) {
    __syncthreads();
    const int32_t* outl = outliers + (size_t)prob * (size_t)n_out;     // [G][batch][H_kv][n_out], like sel_idx
    for (int o = tid; o < n_out; o += TH) {
      const int jo = outl[o];
      if (jo >= 0 && jo < n_c) atomicOr(&take_w[jo >> 5], 1u << (jo & 31));
    }
  }
  __syncthreads();
  // ---- exclusive prefix over the CTA in thread order; the total goes to sh[3]
  auto block_scan = [&](uint32_t mine) -> uint32_t {
    uint32_t inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t v = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += v;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    if (warp == 0) {
      const uint32_t t = lane < NWARP ? warp_tot[lane] : 0u;
      uint32_t ti = t;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_up_sync(0xffffffffu, ti, o);
        if (lane >= o) ti += v;
      }
      if (lane < NWARP) warp_tot[lane] = ti - t;
      if (lane == 31) sh[3] = ti;
    }
    __syncthreads();
    return inc - mine + warp_tot[warp];
  };
  // keys equal to the threshold: the need_eq with the lowest chunk index are taken (thread w owns word w)
  static_assert(NW <= TH, "one bitmap word per thread");
  uint32_t fw = tid < NW ? take_w[tid] : 0u;
  {
    const uint32_t ew = tid < NW ? eq_w[tid] : 0u;
    const uint32_t eq_before = block_scan((uint32_t)__popc(ew));
    uint32_t room = need_eq > eq_before ? need_eq - eq_before : 0u;
    uint32_t rest = ew;
    while (rest && room) { fw |= rest & (0u - rest); rest &= rest - 1u; --room; }   // lowest set bits first
    __syncthreads();                                                   // sh[3] and warp_tot are reused below
  }
  // ---- positions over the union, chunk ids to the chunk list (ascending), rows written by the whole CTA
  const uint32_t before = block_scan((uint32_t)__popc(fw));
  const uint32_t taken = sh[3];
  {
    uint32_t pos = before, rest = fw;
    while (rest) {
      list_key[pos++] = (uint32_t)(tid * 32 + __ffs(rest) - 1);
      rest &= rest - 1u;
    }
  }
  __syncthreads();
  if (c == 8) {
    for (uint32_t w = (uint32_t)tid; w < taken * 8u; w += TH) {
      const int row = (int)list_key[w >> 3] * 8 + (int)(w & 7u);
      if (row < T) out[w] = row;
    }
  } else {
    for (uint32_t w = (uint32_t)tid; w < taken * (uint32_t)c; w += TH) {
      const uint32_t e = w / (uint32_t)c, t = w - e * (uint32_t)c;
      const int row = (int)list_key[e] * c + (int)t;
      if (row < T) out[w] = row;
    }
  }
  // whole chunks unless the ragged last chunk was taken (it is then the last one)
  int cnt = (int)taken * c;
  if (taken > 0 && list_key[taken - 1] == (uint32_t)(n_c - 1)) cnt -= (n_c * c - T);
  for (int i = cnt + tid; i < k_cap; i += TH) out[i] = -1;
  if (tid == 0 && sel_cnt) sel_cnt[prob] = cnt;
}

}  // namespace

// Top-k of `problems` rows of dev.pooled (sign == 0: keys; else floats compared as sign * value).
static cudaError_t launch_topk(const GroupDev& dev, int device, int problems, int l0, int k_ch, int k_cap,
                               const int32_t* outliers, int n_out, float sign, int32_t* sel_idx, int32_t* sel_cnt,
                               cudaStream_t s) {
  if (dev.n_c > kTopkThreads * 32)
    return launch_pdl(topk_kernel<false>, dim3(problems), dim3(kTopkThreads), 0, s, dev, l0, k_ch, k_cap, outliers, n_out,
                      sign, sel_idx, sel_cnt);
  // keys per thread: 16 up to 16384 chunks, 32 beyond; threads: the fewest of 128, 256, 512, 1024 that cover the
  // chunks (a short context needs fewer barriers' worth of warps, and several of its CTAs share an SM); groups per
  // thread: the fewest with at least k_ch groups in all (0 = no filter)
  const int items = dev.n_c <= kTopkThreads * 16 ? 16 : 32;
  const int th = items == 32 ? 1024 : (dev.n_c <= 128 * 16 ? 128 : dev.n_c <= 256 * 16 ? 256 : dev.n_c <= 512 * 16 ? 512 : 1024);
  const size_t smem = (size_t)th * items * (sizeof(uint32_t) + sizeof(uint16_t));
  cudaError_t e;
#define XKV_PIVOT(GPT, ITEMS, TH)                                                                                     \
  do {                                                                                                                \
    e = ensure_dyn_smem<topk_pivot_kernel<GPT, ITEMS, TH>>(smem, device);                                             \
    if (e == cudaSuccess)                                                                                             \
      e = launch_pdl(topk_pivot_kernel<GPT, ITEMS, TH>, dim3(problems), dim3(TH), smem, s, dev, l0, k_ch, k_cap,      \
                     outliers, n_out, sign, sel_idx, sel_cnt);                                                        \
  } while (0)
#define XKV_PIVOT_G(ITEMS, TH)                                                                                        \
  do {                                                                                                                \
    if (groups(1) >= k_ch) XKV_PIVOT(1, ITEMS, TH);                                                                   \
    else if (groups(2) >= k_ch) XKV_PIVOT(2, ITEMS, TH);                                                              \
    else if (groups(4) >= k_ch) XKV_PIVOT(4, ITEMS, TH);                                                              \
    else XKV_PIVOT(0, ITEMS, TH);                                                                                     \
  } while (0)
  auto groups = [&](int gpt) { return (dev.n_c + items / gpt - 1) / (items / gpt); };
  if (items == 32) XKV_PIVOT_G(32, 1024);
  else if (th == 128) XKV_PIVOT_G(16, 128);
  else if (th == 256) XKV_PIVOT_G(16, 256);
  else if (th == 512) XKV_PIVOT_G(16, 512);
  else XKV_PIVOT_G(16, 1024);
#undef XKV_PIVOT_G
#undef XKV_PIVOT
  return e;
}

// Both kernels of the selection for the problems of layers [l0, l1); `tmap` describes dev.landmarks.
// The caller has checked that the row stride (ceil(k/c) + n_out) * c fits 32 bits (select_stride_ok).
static cudaError_t launch_select_dev(const GroupDev& dev, const CUtensorMap& tmap, int device, int l0, int l1,
                                     const __nv_bfloat16* q, int k, int32_t* sel_idx, int32_t* sel_cnt, cudaStream_t s) {
  const int problems = (l1 - l0) * dev.batch * dev.H_kv;
  const int tiles = (dev.n_c + kScoreRows - 1) / kScoreRows;
  const int c = dev.c;
  const int k_ch_raw = (int)(((int64_t)k + c - 1) / c);
  const int k_ch = k_ch_raw < dev.n_c ? k_ch_raw : dev.n_c;
  const int k_cap = (k_ch_raw + dev.n_out) * c;      // room for the union with the outlier chunks
  const size_t smem = 1024 + (size_t)(dev.d_h / 64) * kScoreRows * 128 + (size_t)dev.n_rep * dev.d_h * 4;
  dim3 grid(tiles, problems);
  cudaError_t e;
#define XKV_SCAN(DH, HMAX)                                                                              \
  do {                                                                                                  \
    e = ensure_dyn_smem<score_pool_kernel<DH, HMAX>>(smem, device);                                     \
    if (e != cudaSuccess) return e;                                                                     \
    e = launch_pdl(score_pool_kernel<DH, HMAX>, grid, dim3(kScoreThreads), smem, s, tmap, dev, q, l0); \
  } while (0)
  if (dev.d_h == 128) {
    if (dev.n_rep <= 4) XKV_SCAN(128, 4); else XKV_SCAN(128, 8);
  } else {
    if (dev.n_rep <= 4) XKV_SCAN(64, 4); else XKV_SCAN(64, 8);
  }
#undef XKV_SCAN
  count_launch(kFamScan);
  if (e != cudaSuccess) return e;
  e = launch_topk(dev, device, problems, l0, k_ch, k_cap, dev.outliers, dev.n_out, 0.0f, sel_idx, sel_cnt, s);
  count_launch(kFamTopk);
  return e;
}

// (ceil(k/c) + n_out) * c, the row stride of sel_idx, must fit the 32-bit arithmetic of the kernels.
bool select_stride_ok(int64_t k, int c, int n_out) {
  return k >= 1 && ((k + c - 1) / c + n_out) * (int64_t)c < ((int64_t)1 << 30);
}

// The k entries with the largest sign * scores[p][j] of each of `problems` score rows of length n, ids ascending
// (ties to the lowest id), padded with -1: out [problems][k].  Used for the static outlier chunks (Algorithm 1 line 5).
cudaError_t launch_topk_rows(const float* scores, int problems, int n, int k, float sign, int32_t* out, int device,
                             cudaStream_t s) {
  GroupDev dev{};
  dev.G = 1; dev.batch = problems; dev.H_kv = 1; dev.T = n; dev.c = 1; dev.n_c = n;
  dev.pooled = const_cast<float*>(scores);
  const int k_ch = k < n ? k : n;
  cudaError_t e = launch_topk(dev, device, problems, 0, k_ch, k, nullptr, 0, sign, out, nullptr, s);
  count_launch(kFamTopk);
  return e;
}

cudaError_t launch_select(const xkv_group* grp, int l0, int l1, const __nv_bfloat16* q, int k,
                          int32_t* sel_idx, int32_t* sel_cnt, cudaStream_t s) {
  CUtensorMap tmap;
  memcpy(&tmap, grp->lm_tmap, sizeof(tmap));
  return launch_select_dev(grp->dev, tmap, grp->device, l0, l1, q, k, sel_idx, sel_cnt, s);
}

// ---------------------------------------------------------------------------------------------
// Selection without a handle and without any allocation: the pooled scores live in a file-scope device array.

// 64 flag words followed by the pooled scores of every problem of the call.
static __device__ __align__(256) float g_static_scratch[64 + XKV_STATIC_SELECT_MAX_SCORES];

// The array's name is only a host-side stand-in; its device address is looked up once per device.
static float* static_scratch_ptr(int device, cudaError_t* err) {
  static std::mutex mu;
  static float* ptrs[64] = {};
  std::lock_guard<std::mutex> lock(mu);
  *err = cudaSuccess;
  if (device < 0 || device >= 64) { *err = cudaErrorInvalidDevice; return nullptr; }
  if (!ptrs[device]) {
    float* p = nullptr;
    *err = cudaGetSymbolAddress((void**)&p, g_static_scratch);   // the current device is `device`
    if (*err != cudaSuccess) return nullptr;
    ptrs[device] = p;
  }
  return ptrs[device];
}

int select_static(const xkv_select_static_config* c, int l0, int l1, const void* q, int32_t k, int32_t* sel_idx,
                  int32_t* sel_cnt, cudaStream_t s) {
  if (!c || !q || !sel_idx || !sel_cnt || c->struct_size != sizeof(xkv_select_static_config)) return XKV_ERR_INVALID_ARG;
  if (c->G < 1 || c->batch < 1 || c->T < 1 || c->T >= (1 << 24) || c->H_kv < 1 || c->H_q < 1 ||
      c->H_q % c->H_kv != 0 || c->H_q / c->H_kv > kMaxRep || (c->d_h != 64 && c->d_h != 128) || c->chunk < 0 ||
      c->chunk > 4096 || !c->landmarks || ((uintptr_t)c->landmarks & 15u) || ((uintptr_t)q & 15u) ||
      ((uintptr_t)sel_idx & 3u) || ((uintptr_t)sel_cnt & 3u))
    return XKV_ERR_INVALID_ARG;
  if (l0 < 0 || l1 > c->G || l0 >= l1 || k < 1) return XKV_ERR_INVALID_ARG;
  // a budget beyond the context means "every row"; the row stride the caller allocated follows from k, so a k whose
  // stride leaves 32-bit range is rejected here, before anything is launched
  if (!select_stride_ok(k, c->chunk ? c->chunk : 8, 0)) return XKV_ERR_INVALID_ARG;
  GroupDev dev{};
  dev.G = c->G; dev.batch = c->batch; dev.T = c->T; dev.H_kv = c->H_kv; dev.H_q = c->H_q; dev.d_h = c->d_h;
  dev.c = c->chunk ? c->chunk : 8;
  dev.n_c = (c->T + dev.c - 1) / dev.c;
  dev.n_rep = c->H_q / c->H_kv;
  dev.sel_scale = 1.0f / sqrtf((float)c->d_h);
  dev.landmarks = (const __nv_bfloat16*)c->landmarks;
  const size_t scores = (size_t)c->G * c->batch * c->H_kv * dev.n_c;   // indexed by absolute layer, like the handle's
  if (scores > (size_t)XKV_STATIC_SELECT_MAX_SCORES) return XKV_ERR_TOO_LARGE;
  if ((size_t)c->G * c->batch * c->H_kv > 65535) return XKV_ERR_TOO_LARGE;   // problems of a call are a grid dimension
  int device = 0;
  cudaError_t e = cudaGetDevice(&device);
  if (e != cudaSuccess) { set_cuda_error(e); return XKV_ERR_CUDA; }
  static std::atomic<int> cc_major[kMaxDevices];          // 0: not looked up yet
  if (device < 0 || device >= kMaxDevices) return XKV_ERR_ARCH;
  int major = cc_major[device].load(std::memory_order_relaxed);
  if (major == 0) {
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device);
    if (e != cudaSuccess) { set_cuda_error(e); return XKV_ERR_CUDA; }
    cc_major[device].store(major, std::memory_order_relaxed);
  }
  if (major != 10) return XKV_ERR_ARCH;
  float* scratch = static_scratch_ptr(device, &e);
  if (!scratch) { set_cuda_error(e); (void)cudaGetLastError(); return XKV_ERR_CUDA; }
  dev.flags = reinterpret_cast<unsigned int*>(scratch);
  dev.pooled = scratch + 64;
  CUtensorMap tmap;
  if (!encode_landmark_map(&tmap, c->landmarks, (uint64_t)c->batch * c->G * c->H_kv * dev.n_c, (uint64_t)c->d_h))
    return XKV_ERR_CUDA;
  e = cudaMemsetAsync(scratch, 0, 64 * sizeof(float), s);              // the flag words start at zero
  if (e == cudaSuccess) e = launch_select_dev(dev, tmap, device, l0, l1, (const __nv_bfloat16*)q, k, sel_idx, sel_cnt, s);
  if (e != cudaSuccess) { set_cuda_error(e); (void)cudaGetLastError(); return XKV_ERR_CUDA; }
  return XKV_OK;
}

}  // namespace xkv
