// Selective reconstruction (Sec. 3.2, Eq. 3) fused with decode attention over the rebuilt rows: the
// tensor-core path.  One persistent CTA per SM walks a contiguous range of 128-row tiles of the selected
// sets; a problem is one (layer, sequence, KV head).
//
// Per tile (128 selected rows S_t of one problem, j indexes the tile's rows, m the rank dimension):
//   keys    K_hat[j][d] = sum_m A_k[S_t[j]][m] B_k[m][d]       tcgen05.mma, M = rows, N = d_h, fp32 in TMEM
//           z[h][j]     = scale * <q_h, rope(K_hat[j])>          thread j owns TMEM lane j (one rebuilt key row)
//           p[h][j]     = exp(z - running max)                   online softmax; p is handed on as bf16
//   values  W[m][h]    += sum_j A_v[S_t[j]][m] p[h][j]           tcgen05.mma, M = 128 rank columns, N = heads
// and once per problem, after the segments have been merged,  out_h = (W[:, h] / l_h)^T B_v.
// This is Eq. 3 for the values with the product re-associated: sum_j p_j (A_v[S_j] B_v) = (sum_j p_j A_v[S_j]) B_v,
// so the rebuilt value rows are consumed in factored form and never materialised.  Rebuilt key rows live in
// TMEM only.  Every gathered byte is written to shared memory once and read by the tensor core once.
//
// Warp roles: 0-3 key epilogue, 4-7 value epilogue, 8-9 gather producers of the key stream, 10-11 of the value
// stream (cp.async of the selected rows of A_k / A_v into two rings of 16 KB slabs, one per stream), 12 MMA issue
// for the key phases, 13 TMA loader of the B_k slabs (a short ring: they come from L2), 14 MMA issue for the value
// phases.  The two streams are coupled only through the data: a value phase needs the weights that the key
// epilogue derives from the same tile's key phase.  Slots are released in pairs by tcgen05.commit; every barrier
// has one producer side and waiters that see each of its phases in order, so that one parity bit per waiter is
// enough.  Every wait is bounded; a wait that runs out raises XKV_FLAG_TIMEOUT and the CTA winds down.
// The kernel starts under programmatic dependent launch: set-up overlaps the tail of the selection kernels.
//
// Diagnostic counters (cycles, per CTA, 64 words; see xkv_debug_read_profile): 0 key-stream producer total, 1-3 its
// waits (rotary/position buffers, positions, ring), 4 tiles; 48 value-stream producer total, 50-51 its waits
// (positions, ring); key-phase MMA warp: 8 total, 9 accumulator wait, 10 B ring, 11 row ring, 12 issue;
// value-phase MMA warp: 40 total, 41 accumulator wait, 43 row ring, 44 issue, 45 weights; 17/18 loader waits;
// 24 key epilogue total, 25 positions, 26 accumulator, 27 group barrier, 28 weights buffer; 32 value epilogue
// total, 33 accumulator.
#include <cuda.h>

#include "xkv_internal.cuh"
#include "xkv_ptx.cuh"

namespace xkv {

namespace {

using namespace ptx;

constexpr int kTile = 128;                       // selected rows per tile
constexpr int kSlabBytes = kTile * 128;          // 128 rows x 64 bf16 (one 128-byte swizzle row each)
constexpr int kNB = 4;                           // slots of the B-slab ring
constexpr int kThreads = 15 * 32;
constexpr int kSmemLimit = 227 * 1024;
constexpr int kRopeStride = 66;                  // float2 per staged rotary row (64 + pad against bank conflicts)
constexpr int kPBytes = 2 * 16 * 128;            // softmax weights of a tile as a bf16 MMA operand: [2][16 heads][64 rows]
constexpr int kMaxBlocks = 8;                    // 128-column blocks of r_v that fit the TMEM accumulators
constexpr unsigned long long kWaitLimitNs = 250000000ull;    // a wait that lasts a quarter of a second has failed
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct Sched {
  int l0;            // first layer of the call
  int tpp;           // tiles per problem = ceil(k_cap / 128)
  int n_tiles;       // problems * tpp
  int n_ctas;
  int n_slots;       // partial slots per problem
  int k_cap;
  unsigned long long* prof;   // diagnostic counters [n_ctas][64] or nullptr
};

struct Bars {        // offsets (in 8-byte words) into the barrier array
  int full, fullv, emptyk, emptyv, bfull, kfull, kempty, wfull, wempty, pfull, rfree, posfull, vfree, grp, drain, total;
};
__host__ __device__ constexpr Bars bar_layout(int na) {
  Bars b{};
  // one release barrier per slot pair and kind of occupant (key-phase or value-phase slabs): a waiter that knows
  // the kind it waits for is never confused by the other kind's completions
  b.full = 0; b.fullv = na; b.emptyk = 2 * na; b.emptyv = 2 * na + na / 2; b.bfull = 3 * na; b.kfull = b.bfull + kNB;
  b.kempty = b.kfull + 2; b.wfull = b.kempty + 2; b.wempty = b.wfull + 2; b.pfull = b.wempty + 2;
  b.rfree = b.pfull + 2; b.posfull = b.rfree + 2; b.vfree = b.posfull + 4; b.grp = b.vfree + 4; b.drain = b.grp + 1; b.total = b.drain + 2;
  return b;
}

// cta that owns global tile t when cta i owns tiles [i*N/C, (i+1)*N/C)
__host__ __device__ __forceinline__ int cta_of_tile(long long t, int C, int N) { return (int)(((t + 1) * C - 1) / N); }

// PROF = false: `prof` is a compile-time null pointer and every diagnostic branch of the kernel folds away (the
// loops of the kernel have to stay small: the warps of a scheduler share its instruction cache).
template <bool PROF>
struct CtxT {
  volatile int* abort;
  unsigned int* flags;
  unsigned long long* prof;   // per-CTA diagnostic counters (cycles)
};
template <>
struct CtxT<false> {
  volatile int* abort;
  unsigned int* flags;
  static constexpr unsigned long long* prof = nullptr;
};
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait on an mbarrier phase.  Returns false if another thread of the CTA has given up, or if the
// phase does not complete within kWaitLimitNs (then this thread raises the flag and makes the others give up).
// The polling loop is one out-of-line function: the kernel's loops wait in dozens of places and have to stay
// small (the warps of a scheduler share its instruction cache).
__device__ __noinline__ bool wait_bar_slow(volatile int* abort_flag, unsigned int* flags, uint32_t bar, uint32_t parity) {
  const unsigned long long t0 = global_ns();
  // abort_flag[1] holds the limit in units of 2^16 ns (0: the default)
  const unsigned long long limit = abort_flag[1] ? ((unsigned long long)abort_flag[1] << 16) : kWaitLimitNs;
  for (uint32_t i = 1;; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 63u) == 0u) {
      if (*abort_flag) return false;
      if (global_ns() - t0 > limit) break;
    }
  }
  *abort_flag = 1;
  atomicOr(flags, XKV_FLAG_TIMEOUT);
  return false;
}
template <class Ctx>
__device__ __forceinline__ bool wait_bar_raw(const Ctx& c, uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  return wait_bar_slow(c.abort, c.flags, bar, parity);
}
// `slot` >= 0 (passed warp-uniformly by one warp per role when diagnostics are on) adds the cycles waited.
template <class Ctx>
__device__ __forceinline__ bool wait_bar(const Ctx& c, uint32_t bar, uint32_t parity, int slot = -1) {
  if (c.prof == nullptr || slot < 0) return wait_bar_raw(c, bar, parity);
  const long long c0 = clock64();
  const bool r = wait_bar_raw(c, bar, parity);
  if ((threadIdx.x & 31) == 0) atomicAdd(c.prof + slot, (unsigned long long)(clock64() - c0));
  return r;
}

// Logits of one rebuilt key row against NR query heads: rotate the (i, i+HALF) pairs, accumulate q . k.
// hi/lo point at this row's coarse/fine rotary entries (cos, sin), in shared (SMEM) or global memory.
template <int DH, int NR, bool ROPE, bool SMEM>
__device__ __forceinline__ void key_logits(uint32_t acc, const float2* __restrict__ hi, const float2* __restrict__ lo,
                                           const float* __restrict__ q_s, float (&z)[NR]) {
  constexpr int HALF = DH / 2;
  // 4 rotary pairs per pass: the loop body has to stay small, the four warps of a scheduler run four different
  // loops and share its instruction cache (32 pairs per pass: 77 us per call, 8: 73 us, 4: 71 us)
#pragma unroll 1
  for (int pass = 0; pass < HALF / 4; ++pass) {
    uint32_t xa[4], xb[4];
    tmem_ld4_nb(acc + (uint32_t)(pass * 4), xa);
    tmem_ld4_nb(acc + (uint32_t)(HALF + pass * 4), xb);
    tc_wait_ld_nb(xa, xb);            // the table and query loads below do not depend on it and may be issued above it
    float x1[4], x2[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) { x1[e] = __uint_as_float(xa[e]); x2[e] = __uint_as_float(xb[e]); }
#pragma unroll
    for (int i4 = 0; i4 < 1; ++i4) {
      float r1[4], r2[4];
      const int ii = pass * 4 + i4 * 4;
      if (ROPE) {
        float2 a[4], c2[4];
        if (SMEM) {
          const float4 a01 = *reinterpret_cast<const float4*>(hi + ii), a23 = *reinterpret_cast<const float4*>(hi + ii + 2);
          const float4 c01 = *reinterpret_cast<const float4*>(lo + ii), c23 = *reinterpret_cast<const float4*>(lo + ii + 2);
          a[0] = make_float2(a01.x, a01.y); a[1] = make_float2(a01.z, a01.w);
          a[2] = make_float2(a23.x, a23.y); a[3] = make_float2(a23.z, a23.w);
          c2[0] = make_float2(c01.x, c01.y); c2[1] = make_float2(c01.z, c01.w);
          c2[2] = make_float2(c23.x, c23.y); c2[3] = make_float2(c23.z, c23.w);
        } else {
#pragma unroll
          for (int e = 0; e < 4; ++e) { a[e] = __ldg(hi + ii + e); c2[e] = __ldg(lo + ii + e); }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float cs = a[e].x * c2[e].x - a[e].y * c2[e].y;      // cos(x + y)
          const float sn = a[e].y * c2[e].x + a[e].x * c2[e].y;      // sin(x + y)
          const float u = x1[i4 * 4 + e], v = x2[i4 * 4 + e];
          r1[e] = u * cs - v * sn;
          r2[e] = v * cs + u * sn;
        }
      } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) { r1[e] = x1[i4 * 4 + e]; r2[e] = x2[i4 * 4 + e]; }
      }
      // heads in groups of four, element by element inside a group: the four multiply-adds of an element are
      // independent (one head after the other is a chain of eight dependent ones)
#pragma unroll
      for (int h0 = 0; h0 < NR; h0 += 4) {
        float4 qa[4], qb[4];
#pragma unroll
        for (int h = 0; h < 4; ++h) {
          qa[h] = *reinterpret_cast<const float4*>(q_s + (h0 + h) * DH + ii);
          qb[h] = *reinterpret_cast<const float4*>(q_s + (h0 + h) * DH + HALF + ii);
        }
#pragma unroll
        for (int h = 0; h < 4; ++h) z[h0 + h] = fmaf(qa[h].x, r1[0], z[h0 + h]);
#pragma unroll
        for (int h = 0; h < 4; ++h) z[h0 + h] = fmaf(qb[h].x, r2[0], z[h0 + h]);
#pragma unroll
        for (int h = 0; h < 4; ++h) z[h0 + h] = fmaf(qa[h].y, r1[1], z[h0 + h]);
#pragma unroll
        for (int h = 0; h < 4; ++h) z[h0 + h] = fmaf(qb[h].y, r2[1], z[h0 + h]);
#pragma unroll
        for (int h = 0; h < 4; ++h) z[h0 + h] = fmaf(qa[h].z, r1[2], z[h0 + h]);
#pragma unroll
        for (int h = 0; h < 4; ++h) z[h0 + h] = fmaf(qb[h].z, r2[2], z[h0 + h]);
#pragma unroll
        for (int h = 0; h < 4; ++h) z[h0 + h] = fmaf(qa[h].w, r1[3], z[h0 + h]);
#pragma unroll
        for (int h = 0; h < 4; ++h) z[h0 + h] = fmaf(qb[h].w, r2[3], z[h0 + h]);
      }
    }
  }
}

// The variants that ordinary tiles do not take (no RoPE; a tile whose 8-row groups are not whole landmark chunks, or
// a rotary table that is not staged) are kept out of line: the key epilogue's loop has to stay small.
template <int NR>
struct LogitsOut { float z[NR]; };
template <int DH, int NR, bool ROPE>
__device__ __noinline__ LogitsOut<NR> key_logits_rare(uint32_t acc, const float2* __restrict__ hi, const float2* __restrict__ lo,
                                                      const float* __restrict__ q_s) {
  LogitsOut<NR> o;
#pragma unroll
  for (int h = 0; h < NR; ++h) o.z[h] = 0.0f;
  key_logits<DH, NR, ROPE, false>(acc, hi, lo, q_s, o.z);
  return o;
}

// Shared memory besides the two rings: weights, rotary rows, queries, positions, barriers.
template <int DH, int NR>
__host__ __device__ constexpr int misc_smem_bytes() {
  return (int)(2 * kPBytes + sizeof(float2) * (2 * 16 + 8) * kRopeStride + sizeof(float) * (NR * DH + 2 * NR + 8 * NR) +
               sizeof(int) * (4 * kTile + 8) + 8 * (3 * 16 + kNB + 24) + 16);
}
// Slots of the gathered-row ring: whatever fits beside the B ring.
template <int DH, int NR>
__host__ __device__ constexpr int ring_slots() {
  return ((kSmemLimit - 1024 - misc_smem_bytes<DH, NR>() - kNB * kSlabBytes) / kSlabBytes) & ~1;   // even: released in pairs
}

// NR: query heads per KV head rounded up to 4, 8 or 16.  WB: most 128-column blocks of r_v (registers of the
// value epilogue): NR * WB <= 64.
// QUANT = 4 or 3: the token bases are gathered from 4-bit or 3-bit codes (xkv_group_set_quantized_bases) and
// dequantised by the producer warps on their way into the rings; 0: bf16 bases.
template <int DH, int NR, int WB, bool PROF, int QUANT>
__global__ void __launch_bounds__(kThreads, 1)
sr_fused_kernel(const __grid_constant__ CUtensorMap bk_map, GroupDev dev, Sched sc, const __nv_bfloat16* __restrict__ q,
                const int32_t* __restrict__ sel_idx, const int32_t* __restrict__ sel_cnt) {
  extern __shared__ uint8_t smem_raw[];
  constexpr int HALF = DH / 2;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  constexpr int S = ring_slots<DH, NR>();          // gathered-row slots, all of which may be in flight
  static_assert(S >= 4 && S <= 16, "ring size");   // slot pairs are tracked in 3 bits by the loader
  static_assert(kNB <= 8, "loader fifo");
  // the row slabs are two rings: SK for the key stream, SV for the value stream (both even)
  constexpr int SK = (S % 4 == 0) ? S / 2 : S / 2 + 1, SV = S - SK;
  static_assert(SK >= 2 && SV >= 2 && SK % 2 == 0 && SV % 2 == 0, "ring split");
  const uint32_t bring = base + (uint32_t)S * kSlabBytes;                         // B-slab ring
  // carve-up after the two rings
  uint8_t* P_gen = gen + (size_t)(S + kNB) * kSlabBytes;                         // [2][kPBytes] bf16 weights (MMA operand)
  const uint32_t P_addr = base + (uint32_t)(S + kNB) * kSlabBytes;
  float2* hi_s = reinterpret_cast<float2*>(P_gen + 2 * kPBytes);                 // [2][16][kRopeStride] coarse rotary rows
  float2* lo_s = hi_s + 2 * 16 * kRopeStride;                                    // [8][kRopeStride]     fine rotary rows
  float* q_s = reinterpret_cast<float*>(lo_s + 8 * kRopeStride);                 // [NR][DH]
  float* alpha_s = q_s + NR * DH;                                                // [2][NR]
  float* red_s = alpha_s + 2 * NR;                                               // [2][4][NR]
  int* pos_s = reinterpret_cast<int*>(red_s + 2 * 4 * NR);                       // [4][128]
  int* algn_s = pos_s + 4 * kTile;                                               // [2][4]
  uint64_t* bars = reinterpret_cast<uint64_t*>(algn_s + 8);
  constexpr Bars bl = bar_layout(S);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + bl.total);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const uint32_t bar0 = smem_u32(bars);
  auto BAR = [&](int word) { return bar0 + 8u * (uint32_t)word; };
  CtxT<PROF> ctx;
  ctx.abort = abort_flag;
  ctx.flags = dev.flags;
  if constexpr (PROF) ctx.prof = sc.prof ? sc.prof + (size_t)blockIdx.x * 64 : nullptr;
  // the staged rotary path needs the fine table to cover exactly 8 positions
  const bool rope_smem = dev.use_rope && dev.rope_shift == 3;
  // both phases are padded to an even number of 64-column slabs so that slabs pair up inside ring-slot pairs
  const int nks_k = (dev.r_k + 63) >> 6, nks_v = (dev.r_v + 63) >> 6;
  const int nst_k = (nks_k + 1) & ~1, nst_v = (nks_v + 1) & ~1;

  if (tid == 0) {
    for (int s = 0; s < S; ++s) { mbar_init(BAR(bl.full + s), 64); mbar_init(BAR(bl.fullv + s), 64); }   // 64 threads per stream
    for (int s = 0; s < S / 2; ++s) { mbar_init(BAR(bl.emptyk + s), 1); mbar_init(BAR(bl.emptyv + s), 1); }
    for (int s = 0; s < kNB; ++s) mbar_init(BAR(bl.bfull + s), 1);
    for (int b = 0; b < 2; ++b) {
      mbar_init(BAR(bl.kfull + b), 1); mbar_init(BAR(bl.kempty + b), 128);
      mbar_init(BAR(bl.wfull + b), 1); mbar_init(BAR(bl.wempty + b), 128);
      mbar_init(BAR(bl.pfull + b), 128);
      mbar_init(BAR(bl.rfree + b), 128);
    }
    for (int b = 0; b < 4; ++b) { mbar_init(BAR(bl.posfull + b), 64); mbar_init(BAR(bl.vfree + b), 64); }
    mbar_init(BAR(bl.grp), 128);
    mbar_init(BAR(bl.drain), 1); mbar_init(BAR(bl.drain + 1), 1);
    abort_flag[0] = 0;
    abort_flag[1] = (dev.inject & XKV_INJECT_FUSED_NO_B) ? 16 : 0;   // injected fault: give up after about a millisecond
    fence_mbar_init();
  }
  if (rope_smem) {
    for (int i = tid; i < 8 * HALF; i += kThreads) lo_s[(i / HALF) * kRopeStride + (i % HALF)] = dev.rope_lo[i];
  }
  // weights of heads that do not exist stay zero for the whole kernel
  for (int i = tid; i < 2 * kPBytes / 4; i += kThreads) reinterpret_cast<uint32_t*>(P_gen)[i] = 0u;
  fence_proxy_async();
  if (warp == 12) {
    tmem_alloc(smem_u32(tmem_slot), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // everything above is independent of the inputs; the selection (or whatever wrote q and the index sets) comes
  // from earlier kernels of the stream
  grid_dependency_wait();
  grid_dependency_launch();

  const int C = sc.n_ctas, N = sc.n_tiles;
  const long long t_begin = ((long long)blockIdx.x * N) / C, t_end = ((long long)(blockIdx.x + 1) * N) / C;
  const int per_layer = dev.batch * dev.H_kv;
  const int n_rep = dev.n_rep;

  // Walks this CTA's tiles, skipping tiles that start at or beyond the problem's row count.
  struct TileIter {
    int t, py, ti, cnt, l, b, g, pyn; long long prob;   // t: tile ordinal of the call; pyn/ti: problem and tile in it
  };
  // The problem and tile-in-problem of the first tile, the (layer, sequence, head) of that problem and this CTA's
  // segment number in it, once (divisions); the walk then only counts.  Later problems of the CTA start inside
  // its tile range, so the CTA holds their first segment.
  const int py_first = (int)(t_begin / sc.tpp), ti_first = (int)(t_begin % sc.tpp);
  const int g_first = py_first % dev.H_kv, b_first = (py_first / dev.H_kv) % dev.batch, l_first = sc.l0 + py_first / per_layer;
  const int seg_first = (int)blockIdx.x - cta_of_tile((long long)py_first * sc.tpp, C, N);
  auto iter_begin = [&](TileIter& it_) {
    it_.t = (int)t_begin - 1; it_.py = -1; it_.cnt = 0; it_.prob = 0; it_.pyn = py_first; it_.ti = ti_first - 1;
  };
  // advance to the next non-empty tile; returns false at the end of the range.  Whenever the walk moves to a new
  // problem (also one whose tiles are all empty), `on_leave()` runs with the old problem still in `it_` (not before
  // the first one) and `on_enter()` with the new one, before its tiles.
  auto iter_next = [&](TileIter& it_, auto&& on_leave, auto&& on_enter) -> bool {
    for (;;) {
      ++it_.t;
      if (it_.t >= (int)t_end) return false;
      if (++it_.ti == sc.tpp) { it_.ti = 0; ++it_.pyn; }
      const int py = it_.pyn;
      if (py != it_.py) {
        if (it_.py < 0) {
          it_.l = l_first; it_.b = b_first; it_.g = g_first;
        } else {
          on_leave();
          if (++it_.g == dev.H_kv) { it_.g = 0; if (++it_.b == dev.batch) { it_.b = 0; ++it_.l; } }
        }
        it_.py = py;
        it_.prob = ((long long)it_.l * dev.batch + it_.b) * dev.H_kv + it_.g;
        it_.cnt = min(sel_cnt[it_.prob], sc.k_cap);
        on_enter();
      }
      if (it_.ti * kTile < it_.cnt) return true;
    }
  };
  auto no_op = []() {};
  // partial slot of the segment (this CTA's share) of problem ordinal py
  auto part_of = [&](int py, long long prob) {
    const int seg = py == py_first ? seg_first : 0;
    return dev.part + ((size_t)prob * sc.n_slots + seg) * (size_t)n_rep * (dev.r_v + 2);
  };

  if (warp >= 8 && warp < 12) {
    // =============================== producers: gather rows of A ===============================
    // Two independent streams with a ring of their own each: warps 8-9 gather the rows of A_k of every tile into
    // the key ring, warps 10-11 the same rows of A_v into the value ring.  A stream waits only for releases of its
    // own ring, so the key MMAs of consecutive tiles follow one another without waiting for the value phase that
    // sits between them in time (with one shared ring the key slabs of tile i+2 could not be requested before the
    // last value slab of tile i, which itself waited for the last key MMA of tile i+1).
    // Eight consecutive lanes copy the eight 16-byte pieces of one 128-byte row slab, so that every request of a
    // warp covers whole 128-byte lines; thread t of a stream serves rows (t>>3) + 8*i, i = 0..15.
    const bool kstream = warp < 10;
    const int t64 = (tid - 256) & 63, pw = (warp - 8) & 1;
    const uint32_t c8 = (uint32_t)(t64 & 7), r8 = (uint32_t)(t64 >> 3);
    // rows r8 + 8*i share the swizzle phase r8; slab-relative destination of the i = 0 piece
    const uint32_t dst0 = r8 * 128u + ((c8 ^ r8) << 4);
    const int ps = (warp == 8) ? 0 : (warp == 10 ? 48 : -1000);
    const long long role_t0 = clock64();
    int slot = 0;                     // position in this stream's ring
    uint32_t used = 0, rel_par = 0;   // per slot pair: filled before; parity of the release to wait for next
    int it = 0, pb = 0;               // tiles done; position buffer of the tile (four in rotation)
    bool ok = true;
    const int RS = kstream ? SK : SV;                           // slabs in this stream's ring
    const uint32_t ring0 = base + (kstream ? 0u : (uint32_t)SK * kSlabBytes) + dst0;
    const int bar_full = kstream ? bl.full : bl.fullv, bar_empty = kstream ? bl.emptyk : bl.emptyv;
    const int r = kstream ? dev.r_k : dev.r_v;
    const uint32_t row_bytes = (uint32_t)r * 2u;
    const int nst = kstream ? nst_k : nst_v;
    const __nv_bfloat16* Abase = kstream ? dev.A_k : dev.A_v;
    // one phase of one tile: the 64-column slabs of its gathered rows, two at a time (slots are released in
    // pairs, one tcgen05.commit per two slabs); ro: the tile rows of this thread
    auto issue_phase = [&](const uint32_t (&ro)[16], int b) {
      const char* Ab = reinterpret_cast<const char*>(Abase + (long long)b * dev.T * r) + c8 * 16u;
#pragma unroll 1
      for (int ks = 0; ks < nst; ks += 2) {
        const int pr = slot >> 1;
        const uint32_t bit = 1u << pr;
        if (used & bit) {             // wait for the release of the pair's previous occupant
          if (!wait_bar(ctx, BAR(bar_empty + pr), (rel_par >> pr) & 1u, ps + 3)) { ok = false; return; }
          rel_par ^= bit;
        }
        used |= bit;
        const uint32_t st = ring0 + (uint32_t)slot * kSlabBytes;
        // false in a ragged last slab or a padding slab: zero-fill (the source stays inside the row)
        const bool in0 = ks * 64 + (int)c8 * 8 < r, in1 = (ks + 1) * 64 + (int)c8 * 8 < r;
        const uint32_t n0 = in0 ? 16u : 0u, n1 = in1 ? 16u : 0u;
        const char* s0 = Ab + (in0 ? ks * 128 : 0);
        const char* s1 = Ab + (in1 ? ks * 128 + 128 : 0);
        const uint32_t bar = BAR(bar_full + slot);
#pragma unroll
        for (int i = 0; i < 16; ++i) cp_async16(st + (uint32_t)i * 1024u, s0 + (size_t)ro[i] * row_bytes, n0);
        cp_async_arrive_noinc(bar);                        // arrives when this thread's copies have landed
#pragma unroll
        for (int i = 0; i < 16; ++i) cp_async16(st + kSlabBytes + (uint32_t)i * 1024u, s1 + (size_t)ro[i] * row_bytes, n1);
        cp_async_arrive_noinc(bar + 8u);
        slot += 2;
        if (slot == RS) slot = 0;
      }
    };
    // The same phase from 4-bit codes.  Four consecutive lanes share a tile row: lane q4 fetches the 16 bytes of
    // codes and the scale/offset word of one 32-column group of the slot pair (64 contiguous bytes per row and
    // request), turns them into 32 bf16 values (packed arithmetic, one rounding) and stores them as four 16-byte
    // units of the swizzled slab; a stream's 64 threads cover 16 rows per pass, 8 passes per pair.  The loads of a
    // pair are issued before the wait for the pair's release, so their latency overlaps it.
    const uint32_t q4 = (uint32_t)(t64 & 3), rq = (uint32_t)(t64 >> 2);
    auto issue_phase_q = [&](const uint32_t (&rw)[8], int b) {
      const uint8_t* Cb = (kstream ? dev.Aq_k : dev.Aq_v) + (size_t)b * dev.T * (size_t)(r >> 1);
      const uint32_t* Mb = (kstream ? dev.Am_k : dev.Am_v) + (size_t)b * dev.T * (size_t)(r >> 5);
      const uint32_t ring_q = base + (kstream ? 0u : (uint32_t)SK * kSlabBytes);
      auto fetch = [&](int ks, uint4 (&cw)[8], uint32_t (&mw)[8]) {
        const int col0 = ks * 64 + (int)q4 * 32;           // first column of this lane's group
        const bool in = col0 < r;                          // false in a padding slab: zeros are stored
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          // 4 bits: 16 bytes of codes and a separate scale/offset word; 3 bits: one 16-byte record {meta, w0, w1, w2}
          cw[i] = in ? __ldg(reinterpret_cast<const uint4*>(Cb + (size_t)rw[i] * (size_t)(r >> 1) + (col0 >> 1))) : make_uint4(0, 0, 0, 0);
          if (QUANT == 4) mw[i] = in ? __ldg(Mb + (size_t)rw[i] * (size_t)(r >> 5) + (col0 >> 5)) : 0u;
        }
      };
      auto store = [&](const uint4 (&cw)[8], const uint32_t (&mw)[8]) -> bool {
        const int pr = slot >> 1;
        const uint32_t bit = 1u << pr;
        if (used & bit) {             // wait for the release of the pair's previous occupant
          if (!wait_bar(ctx, BAR(bar_empty + pr), (rel_par >> pr) & 1u, ps + 3)) { ok = false; return false; }
          rel_par ^= bit;
        }
        used |= bit;
        // this lane's group lies in slab (q4 >> 1) of the pair, 16-byte units 4*(q4 & 1) .. +3 of the 128-byte row
        const uint32_t st = ring_q + (uint32_t)(slot + (int)(q4 >> 1)) * kSlabBytes;
        const uint32_t u0 = (q4 & 1u) * 4u;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const uint32_t j = rq + 16u * (uint32_t)i;       // tile row
          const uint32_t w[4] = {cw[i].x, cw[i].y, cw[i].z, cw[i].w};
          uint32_t o[16];
          if (QUANT == 4) {
#pragma unroll
            for (int u = 0; u < 4; ++u) dequant_word(w[u], mw[i], &o[4 * u]);
          } else {
            dequant_group3(w[0], w[1], w[2], w[3], o);
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const uint32_t a = st + j * 128u + (((u0 + (uint32_t)u) ^ (j & 7u)) << 4);
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(o[4 * u]), "r"(o[4 * u + 1]), "r"(o[4 * u + 2]), "r"(o[4 * u + 3]) : "memory");
          }
        }
        asm volatile("cp.async.wait_all;" ::: "memory");   // the staged rotary rows of this tile (key stream) have landed too
        fence_proxy_async();                               // the tensor core reads these stores
        mbar_arrive(BAR(bar_full + slot));                 // both slabs of the pair are complete when all 64 threads are done
        mbar_arrive(BAR(bar_full + slot + 1));
        slot += 2;
        if (slot == RS) slot = 0;
        return true;
      };
      // (a second register set, so that the next pair's loads are in flight while this pair is converted, was
      // measured and lost: 103 us against 85 us per call at the headline size)
      uint4 ca[8];
      uint32_t ma[8];
#pragma unroll 1
      for (int ks = 0; ks < nst; ks += 2) {
        fetch(ks, ca, ma);
        if (!store(ca, ma)) return;
      }
    };
    auto load_rows_q = [&](uint32_t (&rw)[8]) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int p = pos_s[pb * kTile + (int)rq + 16 * i];
        rw[i] = p < 0 ? 0u : (uint32_t)p;
      }
    };
    auto load_rows = [&](uint32_t (&ro)[16]) {             // rows without a selected token read row 0 (weight 0)
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int p = pos_s[pb * kTile + (int)r8 + 8 * i];
        ro[i] = p < 0 ? 0u : (uint32_t)p;
      }
    };
    // One loop for both streams (one copy of the issue code).  The key stream also publishes the row positions and
    // the coarse rotary rows of every tile: thread t loads the positions of tile rows t and t + 64, one tile ahead;
    // the range check is made when the value is used, so that nobody waits for the load here.
    TileIter cur, nxt;
    iter_begin(nxt);
    bool have = iter_next(nxt, no_op, no_op);
    auto load_pos = [&](const TileIter& x, int row) {
      return (x.ti * kTile + row < x.cnt) ? sel_idx[x.prob * sc.k_cap + x.ti * kTile + row] : -1;
    };
    auto checked = [&](const TileIter& x, int row, int p) {
      if (x.ti * kTile + row < x.cnt && (p < 0 || p >= dev.T)) { atomicOr(dev.flags, XKV_FLAG_INDEX_RANGE); p = -1; }
      return p;
    };
    int pn0 = -1, pn1 = -1;
    if (kstream && have) { pn0 = load_pos(nxt, t64); pn1 = load_pos(nxt, t64 + 64); }
    while (ok && have) {
      cur = nxt;
      int pq[2] = {-1, -1};
      if (kstream) { pq[0] = checked(cur, t64, pn0); pq[1] = checked(cur, t64 + 64, pn1); }
      have = iter_next(nxt, no_op, no_op);
      if (kstream) {
        if (have) { pn0 = load_pos(nxt, t64); pn1 = load_pos(nxt, t64 + 64); }
        const int buf = it & 1;
        // the key epilogue must be done with this buffer's rotary rows (tile it-2), and the value stream with
        // the positions of tile it-4
        if (!wait_bar(ctx, BAR(bl.rfree + buf), (uint32_t)(((it >> 1) & 1) ^ 1), ps + 1)) { ok = false; break; }
        if (it >= 4 && !wait_bar(ctx, BAR(bl.vfree + pb), (uint32_t)(((it >> 2) & 1) ^ 1), ps + 1)) { ok = false; break; }
        pos_s[pb * kTile + t64] = pq[0];
        pos_s[pb * kTile + t64 + 64] = pq[1];
        if (rope_smem) {
          // rows 8a..8a+7 of the tile usually share one coarse rotary row (a landmark chunk): stage it once.
          // Warp pw handles the 32-row blocks pw and pw + 2 (lane = row inside the block).
#pragma unroll
          for (int hb = 0; hb < 2; ++hb) {
            const int blk = pw + 2 * hb, p = pq[hb];
            const int hidx = p < 0 ? -1 : (p >> 3);
            int gmax = hidx;
            gmax = max(gmax, __shfl_xor_sync(0xffffffffu, gmax, 1));
            gmax = max(gmax, __shfl_xor_sync(0xffffffffu, gmax, 2));
            gmax = max(gmax, __shfl_xor_sync(0xffffffffu, gmax, 4));
            const bool aligned = __all_sync(0xffffffffu, p < 0 || hidx == gmax);
            if (lane == 0) algn_s[buf * 4 + blk] = aligned ? 1 : 0;
            if (aligned) {
#pragma unroll
              for (int a = 0; a < 4; ++a) {
                const int gm = __shfl_sync(0xffffffffu, gmax, a * 8);
                if (lane * 2 < HALF) {
                  cp_async16(smem_u32(hi_s + (size_t)(buf * 16 + blk * 4 + a) * kRopeStride + lane * 2),
                             dev.rope_hi + (size_t)(gm < 0 ? 0 : gm) * HALF + lane * 2, 16u);
                }
              }
            }
          }
        }
        // publish the row positions of the tile (to both streams and to the key epilogue)
        mbar_arrive(BAR(bl.posfull + pb));
      }
      if (!wait_bar(ctx, BAR(bl.posfull + pb), (uint32_t)((it >> 2) & 1), ps + 2)) { ok = false; break; }
      if constexpr (QUANT != 0) {
        uint32_t rw[8];
        load_rows_q(rw);
        if (!kstream) mbar_arrive(BAR(bl.vfree + pb));     // this thread is done with the position buffer
        issue_phase_q(rw, cur.b);
      } else {
        uint32_t ro[16];
        load_rows(ro);
        if (!kstream) mbar_arrive(BAR(bl.vfree + pb));     // this thread is done with the position buffer
        issue_phase(ro, cur.b);
      }
      ++it;
      if (++pb == 4) pb = 0;
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    if (ctx.prof && (warp == 8 || warp == 10) && lane == 0) {
      ctx.prof[ps] = (unsigned long long)(clock64() - role_t0);
      if (warp == 8) ctx.prof[4] = (unsigned long long)it;
    }
  } else if (warp == 12 || warp == 14) {
    // =============================== MMA issue: warp 12 the key phases, warp 14 the value phases ===============
    // Two issuing threads, each walking its own ring (one thread spends 70-130 cycles per tcgen05.mma and about
    // 235 per tcgen05.commit).
    const bool kside = warp == 12;
    // the whole warp walks the loop (all values are warp-uniform); one lane issues the tensor-core instructions
    constexpr uint32_t idesc_k = idesc_bf16_f32(128, 128);                     // keys: both operands K-major
    constexpr uint32_t idesc_v = idesc_bf16_f32(128, 16) | (1u << 15);         // values: A is read along its rows (MN-major)
    const int ps = kside ? 8 : 40;
    const long long role_t0 = clock64();
    int slot = 0, bslot = 0;                          // positions in the row ring and the B ring
    uint32_t bring_par = 0;
    // This warp is the only consumer of its ring's `full` barriers and sees every phase of them in order, so one
    // parity bit per slot is enough.
    uint32_t seen = 0;
    // descriptors differ between slots only in the start-address field (units of 16 bytes)
    const uint64_t desc_hi = smem_desc_sw128(0, 0) & 0xFFFFFFFF00000000ull;
    const uint32_t rows_lo0 = (uint32_t)(smem_desc_sw128(base, 0) & 0xFFFFFFFFull);
    const uint32_t b_lo0 = (uint32_t)(smem_desc_sw128(bring, 0) & 0xFFFFFFFFull);
    // value phase: A = two adjacent row slabs of the value ring read transposed (64 rank columns each, 16384
    // bytes apart), rows advance in 8-row groups of 1024 bytes; B = the weights of 16 heads x 16 rows
    const uint32_t rows_t_lo0 = (((rows_lo0 & 0xFFFFu) + (uint32_t)SK * (kSlabBytes >> 4)) & 0xFFFFu) | ((uint32_t)(kSlabBytes >> 4) << 16);
    const uint32_t p_lo0 = (uint32_t)(smem_desc_sw128(P_addr, 0) & 0xFFFFFFFFull);
    int it = 0;
    bool ok = true;
    TileIter cur;
    iter_begin(cur);
    while (ok && iter_next(cur, no_op, no_op)) {
      const int buf = it & 1;
      const uint32_t par = (uint32_t)((it >> 1) & 1);
      if (kside) {
        // ---- keys: K_hat = A_k[S] B_k
        const int last_kk = (((dev.r_k - 1) & 63) >> 4) + 1;    // 16-column steps in the last real slab
        const uint32_t acc = tmem + (uint32_t)(buf * 128);
        if (!wait_bar(ctx, BAR(bl.kempty + buf), par ^ 1u, ps + 1)) { ok = false; break; }
        tc_fence_after();
#pragma unroll 1
        for (int ks = 0; ks < nst_k && ok; ks += 2) {
          // one ring-slot pair per iteration: wait for both slabs and their B slabs, then issue all steps at once
          const bool real1 = ks + 1 < nks_k;             // the second slab of the last pair may be padding
          const int bslot1 = (bslot + 1 == kNB) ? 0 : bslot + 1;
          const uint32_t bpar1 = (bslot + 1 == kNB) ? (bring_par ^ 1u) : bring_par;
          if (!wait_bar(ctx, BAR(bl.bfull + bslot), bring_par, ps + 2)) { ok = false; break; }
          if (real1 && !wait_bar(ctx, BAR(bl.bfull + bslot1), bpar1, ps + 2)) { ok = false; break; }
          if (!wait_bar(ctx, BAR(bl.full + slot), (seen >> slot) & 1u, ps + 3)) { ok = false; break; }
          if (!wait_bar(ctx, BAR(bl.full + slot + 1), (seen >> (slot + 1)) & 1u, ps + 3)) { ok = false; break; }
          seen ^= 3u << slot;
          tc_fence_after();
          const long long i0 = ctx.prof ? clock64() : 0;
          if (lane == 0) {
            const uint64_t a_desc = desc_hi | (rows_lo0 + (uint32_t)slot * (kSlabBytes >> 4));
            const uint64_t b_desc = desc_hi | (b_lo0 + (uint32_t)bslot * (kSlabBytes >> 4));
            const uint64_t b_desc1 = desc_hi | (b_lo0 + (uint32_t)bslot1 * (kSlabBytes >> 4));
            const int nkk0 = (ks == nks_k - 1) ? last_kk : 4;
            const int nkk1 = !real1 ? 0 : ((ks + 1 == nks_k - 1) ? last_kk : 4);
            tc_mma_bf16(acc, a_desc, b_desc, idesc_k, ks ? 1u : 0u);
#pragma unroll
            for (int kk = 1; kk < 4; ++kk) {
              if (kk < nkk0) tc_mma_bf16(acc, a_desc + 2u * kk, b_desc + 2u * kk, idesc_k, 1u);   // +32 bytes per step
            }
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
              if (kk < nkk1) tc_mma_bf16(acc, a_desc + (uint32_t)(kSlabBytes >> 4) + 2u * kk, b_desc1 + 2u * kk, idesc_k, 1u);
            }
            tc_commit(BAR(bl.emptyk + (slot >> 1)));   // releases both slabs of the pair (and their B slabs)
            if (ks + 2 >= nst_k) tc_commit(BAR(bl.kfull + buf));
          }
          __syncwarp();
          if (ctx.prof && lane == 0) atomicAdd(ctx.prof + ps + 4, (unsigned long long)(clock64() - i0));
          slot += 2;
          if (slot == SK) slot = 0;
          bslot = bslot1; bring_par = bpar1;
          if (real1 && ++bslot == kNB) { bslot = 0; bring_par ^= 1u; }
        }
      } else {
        // ---- values: W += A_v[S]^T P^T, one accumulator of 16 columns per 128 rank columns
        if (!wait_bar(ctx, BAR(bl.wempty + buf), par ^ 1u, ps + 1)) { ok = false; break; }
        if (!wait_bar(ctx, BAR(bl.pfull + buf), par, ps + 5)) { ok = false; break; }
        tc_fence_after();
        const uint32_t accw = tmem + 256u + (uint32_t)(buf * 128);
        const uint32_t p_lo = p_lo0 + (uint32_t)buf * (kPBytes >> 4);
#pragma unroll 1
        for (int ks = 0; ks < nst_v && ok; ks += 2) {
          if (!wait_bar(ctx, BAR(bl.fullv + slot), (seen >> slot) & 1u, ps + 3)) { ok = false; break; }
          if (!wait_bar(ctx, BAR(bl.fullv + slot + 1), (seen >> (slot + 1)) & 1u, ps + 3)) { ok = false; break; }
          seen ^= 3u << slot;
          tc_fence_after();
          const long long i0 = ctx.prof ? clock64() : 0;
          if (lane == 0) {
            const uint64_t a_desc = desc_hi | (rows_t_lo0 + (uint32_t)slot * (kSlabBytes >> 4));
            const uint32_t acc = accw + (uint32_t)(ks >> 1) * 16u;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {   // 16 tile rows per step: 2048 bytes down the slab, 32 bytes along P
              const uint64_t b_desc = desc_hi | (p_lo + (uint32_t)(kk >> 2) * (2048u >> 4) + (uint32_t)(kk & 3) * 2u);
              tc_mma_bf16(acc, a_desc + (uint32_t)kk * (2048u >> 4), b_desc, idesc_v, kk ? 1u : 0u);
            }
            tc_commit(BAR(bl.emptyv + (slot >> 1)));
            if (ks + 2 >= nst_v) tc_commit(BAR(bl.wfull + buf));
          }
          __syncwarp();
          if (ctx.prof && lane == 0) atomicAdd(ctx.prof + ps + 4, (unsigned long long)(clock64() - i0));
          slot += 2;
          if (slot == SV) slot = 0;
        }
      }
      ++it;
    }
    if (ctx.prof && lane == 0) ctx.prof[ps] = (unsigned long long)(clock64() - role_t0);
    if (!ok && lane == 0) {
      // giving up: the tensor-core operations this thread has issued may still be running and the CTA is about to
      // free its tensor memory; wait (again with a limit) until they have retired
      const uint32_t db = BAR(bl.drain + (kside ? 0 : 1));
      tc_commit(db);
      for (uint32_t i = 0; i < (1u << 22); ++i) if (mbar_try_wait(db, 0)) break;
    }
    __syncwarp();
  } else if (warp == 13) {
    // =============================== B_k slab loader (TMA) ===============================
    // B slab n goes to slot n % kNB, which held slab n - kNB.  That slab's MMAs are known to be complete
    //   - if it belongs to an earlier tile: when the previous tile's key accumulator was committed (kfull);
    //   - if it belongs to this tile: when the key-ring pair of its stage was released.
    // In both cases the barrier's previous phase is already known to be complete and its next phase cannot
    // complete before the slab being loaded is consumed, so the parity test is unambiguous.
    // Without padding slabs and with at least kNB slabs per tile the second rule also covers a slab of the previous
    // tile (the pair after next in the same ring position needs the slab being loaded): then the first slabs of a
    // tile do not have to wait for the end of the previous tile's key phase.
    const bool by_pair = nks_k == nst_k && nks_k >= kNB && kNB <= SK;
    // fault injection (tests of the give-up path): the slabs are never loaded, so the key-phase warp's wait for
    // them runs into its limit and the CTA winds down
    const bool no_b = (dev.inject & XKV_INJECT_FUSED_NO_B) != 0u;
    int bslot = 0, it = 0, slot = 0;
    uint32_t cnt_k = 0;                  // per slot pair: parity of the number of pairs that used it
    uint32_t fifo = 0;                   // per B slot, 4 bits: slot pair (3) and phase parity (1) of the slab it holds
    bool ok = true;
    TileIter cur;
    iter_begin(cur);
    while (ok && lane == 0 && iter_next(cur, no_op, no_op)) {
      const int head_row = (int)((((size_t)cur.b * dev.G + cur.l) * dev.H_kv + cur.g) * kDP);
      uint32_t my = 0;
#pragma unroll 1
      for (int ks = 0; ks < nks_k; ++ks) {
        int sl = slot + ks;
        while (sl >= SK) sl -= SK;
        if ((ks & 1) == 0) {             // key stages start on even slots: entering a slot pair
          const int pr = sl >> 1;
          my = (uint32_t)pr | (((cnt_k >> pr) & 1u) << 3);
          cnt_k ^= 1u << pr;
        }
        if (ks >= kNB || (by_pair && it > 0)) {
          const uint32_t e = (fifo >> (4 * bslot)) & 15u;
          if (!wait_bar(ctx, BAR(bl.emptyk + (int)(e & 7u)), e >> 3, 17)) { ok = false; break; }
        } else if (it > 0 && it * nks_k + ks >= kNB) {
          if (!wait_bar(ctx, BAR(bl.kfull + ((it - 1) & 1)), (uint32_t)(((it - 1) >> 1) & 1), 18)) { ok = false; break; }
        }
        fifo = (fifo & ~(15u << (4 * bslot))) | (my << (4 * bslot));
        if (!no_b) {
          mbar_expect_tx(BAR(bl.bfull + bslot), kSlabBytes);
          tma_load_2d(bring + (uint32_t)bslot * kSlabBytes, &bk_map, ks * 64, head_row, BAR(bl.bfull + bslot));
        }
        if (++bslot == kNB) bslot = 0;
      }
      // (a padding slab after an odd number of real slabs sits in the pair that was entered for the last real one)
      slot += nst_k;
      while (slot >= SK) slot -= SK;
      ++it;
    }
  } else if (warp < 4) {
    // =============================== key epilogue: rope, logits, softmax statistics, weights ===============================
    const int j = tid;                                  // tile row = TMEM lane
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    const float scale2 = dev.att_scale * kLog2e;
    const int rmask = (1 << dev.rope_shift) - 1;
    float m_run[NR], l_thr[NR];
    int it = 0;
    bool ok = true;
    uint32_t grp_par = 0;
    const int ps = warp == 0 ? 24 : -1000;
    int pbuf = 0;                                       // position buffer of the tile (four in rotation)
    const long long role_t0 = clock64();
    // where this row's weights go in the bf16 operand tile: [row block j/64][head][64 rows], 128-byte swizzle
    const uint32_t p_off = (uint32_t)(j >> 6) * 2048u + (uint32_t)(j & 7) * 2u;
    const uint32_t p_unit = (uint32_t)((j & 63) >> 3);
    // barrier among the 128 threads of this role, with the same bounded wait as every other wait
    auto group_sync = [&]() {
      mbar_arrive(BAR(bl.grp));
      if (!wait_bar(ctx, BAR(bl.grp), grp_par, ps + 3)) ok = false;
      grp_par ^= 1u;
    };
    TileIter cur;
    iter_begin(cur);
    auto flush = [&](int py) {   // end of a segment: write (m, l) of every head to the problem's partial slot
      float tot[NR];
#pragma unroll
      for (int h = 0; h < NR; ++h) {
        float v = l_thr[h];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        tot[h] = v;
      }
      group_sync();                                     // red_s[0] is free (last tile's readers are done)
      if (lane == 0) {
#pragma unroll
        for (int h = 0; h < NR; ++h) red_s[warp * NR + h] = tot[h];
      }
      group_sync();
      if (j < n_rep) {
        float* part = part_of(py, cur.prob) + (size_t)j * (dev.r_v + 2) + dev.r_v;
        float ls = 0.0f, mm = -INFINITY;
#pragma unroll
        for (int h = 0; h < NR; ++h) {
          if (h == j) { ls = red_s[h] + red_s[NR + h] + red_s[2 * NR + h] + red_s[3 * NR + h]; mm = m_run[h]; }
        }
        part[0] = mm;
        part[1] = ls;
      }
    };
    auto on_leave = [&]() { flush(cur.py); };
    auto on_enter = [&]() {
#pragma unroll
      for (int h = 0; h < NR; ++h) { m_run[h] = -INFINITY; l_thr[h] = 0.0f; }
      const __nv_bfloat16* qg = q + (((long long)cur.l * dev.batch + cur.b) * dev.H_q + (long long)cur.g * n_rep) * DH;
      // 16-byte pieces, all of a thread's loads issued before the first is used (heads beyond n_rep are zero)
      {
        constexpr int kPieces = NR * DH / 8, kPer = (kPieces + 127) / 128;
        const uint4* qv = reinterpret_cast<const uint4*>(qg);
        uint4 u[kPer];
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
          const int pc = j + 128 * i;
          u[i] = (pc < kPieces && pc * 8 < n_rep * DH) ? __ldg(qv + pc) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
          const int pc = j + 128 * i;
          if (pc < kPieces) {
            float4 a, b;
            a.x = __uint_as_float(u[i].x << 16); a.y = __uint_as_float(u[i].x & 0xffff0000u);
            a.z = __uint_as_float(u[i].y << 16); a.w = __uint_as_float(u[i].y & 0xffff0000u);
            b.x = __uint_as_float(u[i].z << 16); b.y = __uint_as_float(u[i].z & 0xffff0000u);
            b.z = __uint_as_float(u[i].w << 16); b.w = __uint_as_float(u[i].w & 0xffff0000u);
            *reinterpret_cast<float4*>(q_s + pc * 8) = a;
            *reinterpret_cast<float4*>(q_s + pc * 8 + 4) = b;
          }
        }
      }
      group_sync();
    };
    while (ok && iter_next(cur, on_leave, on_enter)) {
      const int buf = it & 1;
      const uint32_t par = (uint32_t)((it >> 1) & 1);
      if (!wait_bar(ctx, BAR(bl.posfull + pbuf), (uint32_t)((it >> 2) & 1), ps + 1)) { ok = false; break; }   // positions published
      if (!wait_bar(ctx, BAR(bl.kfull + buf), par, ps + 2)) { ok = false; break; }
      tc_fence_after();
      const int pos = pos_s[pbuf * kTile + j];
      if (++pbuf == 4) pbuf = 0;
      const int pp = pos < 0 ? 0 : pos;
      float z[NR];
#pragma unroll
      for (int h = 0; h < NR; ++h) z[h] = 0.0f;
      const uint32_t acc = tmem + lane_base + (uint32_t)(buf * 128);
      if (rope_smem && algn_s[buf * 4 + warp]) {
        key_logits<DH, NR, true, true>(acc, hi_s + (size_t)(buf * 16 + (j >> 3)) * kRopeStride,
                                       lo_s + (size_t)(pp & 7) * kRopeStride, q_s, z);
      } else {
        const LogitsOut<NR> o = dev.use_rope
            ? key_logits_rare<DH, NR, true>(acc, dev.rope_hi + (size_t)(pp >> dev.rope_shift) * HALF,
                                            dev.rope_lo + (size_t)(pp & rmask) * HALF, q_s)
            : key_logits_rare<DH, NR, false>(acc, nullptr, nullptr, q_s);
#pragma unroll
        for (int h = 0; h < NR; ++h) z[h] = o.z[h];
      }
      tc_fence_before();
      mbar_arrive(BAR(bl.kempty + buf));                // accumulator may be overwritten
      mbar_arrive(BAR(bl.rfree + buf));                 // positions and rotary rows of this tile are consumed
      // tile max per head over the 128 rows
      // (one redux.sync per head on the order-preserving integer image of the float: exact, and a fraction of
      // the code of a shuffle tree)
      float tmax[NR];
#pragma unroll
      for (int h = 0; h < NR; ++h) {
        z[h] = pos < 0 ? -INFINITY : z[h] * scale2;
        int zi = __float_as_int(z[h]);
        zi ^= (zi >> 31) & 0x7fffffff;
        int mi = __reduce_max_sync(0xffffffffu, zi);
        mi ^= (mi >> 31) & 0x7fffffff;
        tmax[h] = __int_as_float(mi);
      }
      float* red = red_s + (it & 1) * 4 * NR;
      if (lane == 0) {
#pragma unroll
        for (int h = 0; h < NR; ++h) red[h * 4 + warp] = tmax[h];   // [head][warp]: one 16-byte load per head below
      }
      group_sync();
      if (!ok) break;
      // the weights buffer and the rescale factors of tile it-2 must have been consumed
      if (!wait_bar(ctx, BAR(bl.wempty + buf), par ^ 1u, ps + 4)) { ok = false; break; }
      uint8_t* Pw = P_gen + buf * kPBytes + p_off;
#pragma unroll
      for (int h = 0; h < NR; ++h) {
        const float4 t4 = *reinterpret_cast<const float4*>(red + h * 4);
        const float tm = fmaxf(fmaxf(t4.x, t4.y), fmaxf(t4.z, t4.w));
        const float m_new = fmaxf(m_run[h], tm);
        const float alpha = (m_run[h] == -INFINITY) ? 0.0f : ex2_approx(m_run[h] - m_new);
        const float p = (m_new == -INFINITY) ? 0.0f : ex2_approx(z[h] - m_new);
        const __nv_bfloat16 pb = __float2bfloat16(p);
        l_thr[h] = l_thr[h] * alpha + __bfloat162float(pb);   // the denominator sums the weights as they are used
        m_run[h] = m_new;
        if (h < n_rep) *reinterpret_cast<__nv_bfloat16*>(Pw + h * 128 + ((p_unit ^ (uint32_t)(h & 7)) << 4)) = pb;
        if (j == h) alpha_s[buf * NR + h] = alpha;
      }
      fence_proxy_async();                              // the weights are read by the tensor core
      mbar_arrive(BAR(bl.pfull + buf));
      ++it;
    }
    if (ok && cur.py >= 0) flush(cur.py);
    if (ctx.prof && j == 0) ctx.prof[24] = (unsigned long long)(clock64() - role_t0);
  } else {
    // =============================== value epilogue: running W = W * alpha + W_tile ===============================
    const int mm = tid - 128;                           // rank column inside a 128-column block = TMEM lane
    const uint32_t lane_base = (uint32_t)((warp - 4) * 32) << 16;
    const int nblk = (dev.r_v + 127) >> 7;
    float w[WB][NR];
    const int ps = warp == 4 ? 32 : -1000;
    const long long role_t0 = clock64();
    int it = 0;
    bool ok = true;
    TileIter cur;
    iter_begin(cur);
    auto flush = [&](int py) {
      float* part = part_of(py, cur.prob);
#pragma unroll
      for (int bk = 0; bk < WB; ++bk) {
        const int col = bk * 128 + mm;
        if (bk < nblk && col < dev.r_v) {
#pragma unroll
          for (int h = 0; h < NR; ++h) if (h < n_rep) part[(size_t)h * (dev.r_v + 2) + col] = w[bk][h];
        }
      }
    };
    auto on_leave = [&]() { flush(cur.py); };
    auto on_enter = [&]() {
#pragma unroll
      for (int bk = 0; bk < WB; ++bk)
#pragma unroll
        for (int h = 0; h < NR; ++h) w[bk][h] = 0.0f;
    };
    while (ok && iter_next(cur, on_leave, on_enter)) {
      const int buf = it & 1;
      const uint32_t par = (uint32_t)((it >> 1) & 1);
      if (!wait_bar(ctx, BAR(bl.wfull + buf), par, ps + 1)) { ok = false; break; }
      tc_fence_after();
      float al[NR];
#pragma unroll
      for (int h = 0; h < NR; ++h) al[h] = alpha_s[buf * NR + h];
      const uint32_t acc = tmem + lane_base + 256u + (uint32_t)(buf * 128);
#pragma unroll
      for (int bk = 0; bk < WB; ++bk) {
        if (bk < nblk) {
          float v[NR];
          tmem_ld<NR>(acc + (uint32_t)(bk * 16), v);
          tc_wait_ld();
#pragma unroll
          for (int h = 0; h < NR; ++h) w[bk][h] = fmaf(w[bk][h], al[h], v[h]);
        }
      }
      tc_fence_before();
      mbar_arrive(BAR(bl.wempty + buf));
      ++it;
    }
    if (ok && cur.py >= 0) flush(cur.py);
    if (ctx.prof && mm == 0) ctx.prof[32] = (unsigned long long)(clock64() - role_t0);
  }

  // wind down: nothing of this CTA may still touch shared or tensor memory
  asm volatile("cp.async.wait_all;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  if (warp == 12) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// Partials of a problem -> out, lse.  grid.x = problems * n_rep, 1024 threads.  m is in log2 units.
// W_h = sum_seg 2^(m_seg - M) W_seg[h], L = sum_seg 2^(m_seg - M) l_seg, then
// out_h[d] = (1/L) sum_m W_h[m] B_v[m][g*d_h + d]   (Eq. 3 applied once to the weighted sum of basis rows).
// DH/8 threads read one 16-byte piece each of a B_v row; 1024/(DH/8) rows are in flight per pass.
constexpr int kMergeThreads = 1024;
constexpr int kMergeMaxSeg = 160;                     // a problem never has more segments than there are CTAs + 1
template <int DH>
__global__ void __launch_bounds__(kMergeThreads)
merge_segments_kernel(GroupDev dev, Sched sc, TailParts tail, __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
  extern __shared__ float m_s[];                      // [r_v] weights-times-basis, then [rows per pass][DH] partial sums
  __shared__ float wgt_s[kMergeMaxSeg];
  __shared__ float twgt_s[kTailMaxSplit];             // weights of the partial results over the uncompressed tail
  __shared__ float ML_s[2];
  constexpr int TPR = DH / 8, RPP = kMergeThreads / TPR;
  const int n_rep = dev.n_rep, r = dev.r_v;
  float* w_s = m_s;
  float* red = m_s + ((r + 3) & ~3);
  const int tid = threadIdx.x;
  const int h = blockIdx.x % n_rep, py = blockIdx.x / n_rep;
  const int per_layer = dev.batch * dev.H_kv;
  const int g = py % dev.H_kv, b = (py / dev.H_kv) % dev.batch, l = sc.l0 + py / per_layer;
  const long long prob = ((long long)l * dev.batch + b) * dev.H_kv + g;
  const long long first = (long long)py * sc.tpp;
  const int c0 = cta_of_tile(first, sc.n_ctas, sc.n_tiles), c1 = cta_of_tile(first + sc.tpp - 1, sc.n_ctas, sc.n_tiles);
  const int nseg = min(c1 - c0 + 1, kMergeMaxSeg);
  const size_t stride = (size_t)n_rep * (r + 2);
  // the B_v pieces do not depend on the partials: start those loads before anything else
  const int rg = tid / TPR, dg = tid % TPR;
  const size_t ld = (size_t)dev.H_kv * DH;
  const __nv_bfloat16* Bv = dev.B_v + (((size_t)b * dev.G + l) * r) * ld + (size_t)g * DH + dg * 8;
  constexpr int kPre = 8;                             // rows of B_v held in registers per thread
  uint4 pre[kPre];
#pragma unroll
  for (int i = 0; i < kPre; ++i) {
    const int m = rg + i * RPP;
    pre[i] = m < r ? *reinterpret_cast<const uint4*>(Bv + (size_t)m * ld) : make_uint4(0, 0, 0, 0);
  }
  grid_dependency_wait();                             // the partials come from the kernel launched before this one
  grid_dependency_launch();                           // the next kernel of the stream may start its own set-up
  const float* part = dev.part + ((size_t)prob * sc.n_slots) * stride + (size_t)h * (r + 2);
  const int nts = tail.part ? min(tail.n_split, kTailMaxSplit) : 0;
  const size_t tstride = (size_t)n_rep * (DH + 2);
  const float* tpart = tail.part ? tail.part + ((size_t)py * tail.n_split) * tstride + (size_t)h * (DH + 2) : nullptr;
  // this thread's column of the first segments' partial sums: fetched together with the statistics below, so
  // that the merge costs one round trip to L2 instead of two
  constexpr int kSegPre = 8;
  static_assert(kMaxBlocks * 128 <= kMergeThreads, "one rank column per thread");
  float pv[kSegPre];
#pragma unroll
  for (int s = 0; s < kSegPre; ++s) pv[s] = (s < nseg && tid < r) ? __ldcg(part + s * stride + tid) : 0.0f;
  if (tid < 32) {                                     // one warp: maxima, weights of the segments, denominator
    // maxima and denominators of this lane's segments in one batch of loads
    constexpr int kPer = (kMergeMaxSeg + 31) / 32;
    float sm[kPer], sl[kPer];
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
      const int s = tid + 32 * i;
      sm[i] = s < nseg ? __ldcg(part + s * stride + r) : -INFINITY;
      sl[i] = s < nseg ? __ldcg(part + s * stride + r + 1) : 0.0f;
    }
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < kPer; ++i) mx = fmaxf(mx, sm[i]);
    for (int s = tid; s < nts; s += 32) mx = fmaxf(mx, tpart[s * tstride + DH]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float Ls = 0.0f;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
      const int s = tid + 32 * i;
      if (s < nseg) {
        const float w = (sm[i] == -INFINITY || mx == -INFINITY) ? 0.0f : exp2f(sm[i] - mx);
        wgt_s[s] = w;
        Ls += w * sl[i];
      }
    }
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
  if (tid < r) {                                      // r <= kMergeThreads
    float acc = 0.0f;
#pragma unroll
    for (int s = 0; s < kSegPre; ++s) if (s < nseg) acc = fmaf(wgt_s[s], pv[s], acc);
    for (int s = kSegPre; s < nseg; ++s) acc = fmaf(wgt_s[s], part[s * stride + tid], acc);
    w_s[tid] = acc;
  }
  __syncthreads();
  float acc[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) acc[e] = 0.0f;
  auto add_row = [&](const uint4& v, float w) {
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      acc[2 * e] = fmaf(w, __uint_as_float(u[e] << 16), acc[2 * e]);
      acc[2 * e + 1] = fmaf(w, __uint_as_float(u[e] & 0xffff0000u), acc[2 * e + 1]);
    }
  };
#pragma unroll
  for (int i = 0; i < kPre; ++i) {
    const int m = rg + i * RPP;
    if (m < r) add_row(pre[i], w_s[m]);
  }
#pragma unroll 4
  for (int m = rg + kPre * RPP; m < r; m += RPP) add_row(*reinterpret_cast<const uint4*>(Bv + (size_t)m * ld), w_s[m]);
#pragma unroll
  for (int e = 0; e < 8; ++e) red[rg * DH + dg * 8 + e] = acc[e];
  __syncthreads();
  // two-level sum over the row groups: 1024 threads fold RPP partials to 8 per column, then DH threads finish
  constexpr int FOLD = kMergeThreads / DH;            // 8 (d_h = 128) or 16 (d_h = 64) threads per column
  {
    const int d = tid % DH, f = tid / DH;
    float o = 0.0f;
#pragma unroll 4
    for (int i = f; i < RPP; i += FOLD) o += red[i * DH + d];
    // the partial results over the uncompressed tail are already in output space; spread over all threads, so
    // that their loads are one round trip and not a chain of them
#pragma unroll 4
    for (int s = f; s < nts; s += FOLD) o = fmaf(twgt_s[s], tpart[s * tstride + d], o);
    __syncthreads();
    red[f * DH + d] = o;
  }
  __syncthreads();
  if (tid < DH) {
    float o = 0.0f;
#pragma unroll
    for (int f = 0; f < FOLD; ++f) o += red[f * DH + tid];
    const float M = ML_s[0], L = ML_s[1];
    const long long qh = ((long long)l * dev.batch + b) * dev.H_q + (long long)g * n_rep + h;
    out[qh * DH + tid] = __float2bfloat16(L > 0.0f ? o / L : 0.0f);
    if (lse && tid == 0) lse[qh] = L > 0.0f ? (M + log2f(L)) * kLn2 : -INFINITY;
  }
}

// The same merge for windows with many problems: one CTA per (problem, group of HG query heads), 512 threads.
// With one CTA per head a window of 128 problems x 7 heads is six waves of CTAs that each read the problem's B_v
// block again; here every B_v row a thread fetches serves all HG heads.  Same arithmetic per head as above; the
// sum over the rows of B_v is folded by one shuffle and one pass through shared memory.
constexpr int kMergeMultiThreads = 512;
template <int DH, int HG>
__global__ void __launch_bounds__(kMergeMultiThreads)
merge_segments_multi_kernel(GroupDev dev, Sched sc, TailParts tail, __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
  extern __shared__ float m_s[];                      // [HG][r4] weighted sums of basis rows, [HG][warps][DH] partial outputs
  __shared__ float wgt_s[HG][kMergeMaxSeg];
  __shared__ float twgt_s[HG][kTailMaxSplit];
  __shared__ float ML_s[HG][2];
  constexpr int TPR = DH / 8, RPP = kMergeMultiThreads / TPR, NW = kMergeMultiThreads / 32;
  const int n_rep = dev.n_rep, r = dev.r_v, r4 = (r + 3) & ~3;
  float* w_s = m_s;
  float* red = m_s + HG * r4;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ngrp = (n_rep + HG - 1) / HG;
  const int h0 = (blockIdx.x % ngrp) * HG, py = blockIdx.x / ngrp;
  const int nh = min(HG, n_rep - h0);
  const int per_layer = dev.batch * dev.H_kv;
  const int g = py % dev.H_kv, b = (py / dev.H_kv) % dev.batch, l = sc.l0 + py / per_layer;
  const long long prob = ((long long)l * dev.batch + b) * dev.H_kv + g;
  const long long first = (long long)py * sc.tpp;
  const int c0 = cta_of_tile(first, sc.n_ctas, sc.n_tiles), c1 = cta_of_tile(first + sc.tpp - 1, sc.n_ctas, sc.n_tiles);
  const int nseg = min(c1 - c0 + 1, kMergeMaxSeg);
  const size_t stride = (size_t)n_rep * (r + 2);
  const int rg = tid / TPR, dg = tid % TPR;
  const size_t ld = (size_t)dev.H_kv * DH;
  const __nv_bfloat16* Bv = dev.B_v + (((size_t)b * dev.G + l) * r) * ld + (size_t)g * DH + dg * 8;
  constexpr int kPre = HG <= 4 ? 8 : 4;               // rows of B_v requested before the partials are waited for
  uint4 pre[kPre];
#pragma unroll
  for (int i = 0; i < kPre; ++i) {
    const int m = rg + i * RPP;
    pre[i] = m < r ? *reinterpret_cast<const uint4*>(Bv + (size_t)m * ld) : make_uint4(0, 0, 0, 0);
  }
  grid_dependency_wait();
  grid_dependency_launch();
  const float* part0 = dev.part + ((size_t)prob * sc.n_slots) * stride + (size_t)h0 * (r + 2);
  const int nts = tail.part ? min(tail.n_split, kTailMaxSplit) : 0;
  const size_t tstride = (size_t)n_rep * (DH + 2);
  const float* tpart0 = tail.part ? tail.part + ((size_t)py * tail.n_split) * tstride + (size_t)h0 * (DH + 2) : nullptr;
  if (warp < nh) {                                    // warp h: maxima, weights of the segments, denominator of head h0 + h
    const float* part = part0 + (size_t)warp * (r + 2);
    const float* tpart = tpart0 ? tpart0 + (size_t)warp * (DH + 2) : nullptr;
    constexpr int kPer = (kMergeMaxSeg + 31) / 32;
    float sm[kPer], sl[kPer];
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
      const int sg = lane + 32 * i;
      sm[i] = sg < nseg ? __ldcg(part + sg * stride + r) : -INFINITY;
      sl[i] = sg < nseg ? __ldcg(part + sg * stride + r + 1) : 0.0f;
    }
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < kPer; ++i) mx = fmaxf(mx, sm[i]);
    for (int sg = lane; sg < nts; sg += 32) mx = fmaxf(mx, tpart[sg * tstride + DH]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float Ls = 0.0f;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
      const int sg = lane + 32 * i;
      if (sg < nseg) {
        const float w = (sm[i] == -INFINITY || mx == -INFINITY) ? 0.0f : exp2f(sm[i] - mx);
        wgt_s[warp][sg] = w;
        Ls += w * sl[i];
      }
    }
    for (int sg = lane; sg < nts; sg += 32) {
      const float ms = tpart[sg * tstride + DH];
      const float w = (ms == -INFINITY || mx == -INFINITY) ? 0.0f : exp2f(ms - mx);
      twgt_s[warp][sg] = w;
      Ls += w * tpart[sg * tstride + DH + 1];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) Ls += __shfl_xor_sync(0xffffffffu, Ls, o);
    if (lane == 0) { ML_s[warp][0] = mx; ML_s[warp][1] = Ls; }
  }
  __syncthreads();
  // weighted sums of the segments' partial sums, one rank column per thread and pass, segments in ascending order
  // (the loads of the first four segments of all heads are issued before the first of them is used: one trip to L2
  // per column, not one per head and segment)
  for (int col = tid; col < r; col += kMergeMultiThreads) {
    constexpr int kSegBatch = 4;
    float v[HG][kSegBatch];
#pragma unroll
    for (int h = 0; h < HG; ++h)
#pragma unroll
      for (int sg = 0; sg < kSegBatch; ++sg)
        v[h][sg] = (h < nh && sg < nseg) ? __ldcg(part0 + (size_t)h * (r + 2) + col + sg * stride) : 0.0f;
#pragma unroll
    for (int h = 0; h < HG; ++h) {
      if (h < nh) {
        const float* part = part0 + (size_t)h * (r + 2) + col;
        float acc = 0.0f;
#pragma unroll
        for (int sg = 0; sg < kSegBatch; ++sg) if (sg < nseg) acc = fmaf(wgt_s[h][sg], v[h][sg], acc);
        for (int sg = kSegBatch; sg < nseg; ++sg) acc = fmaf(wgt_s[h][sg], __ldcg(part + sg * stride), acc);
        w_s[h * r4 + col] = acc;
      }
    }
  }
  __syncthreads();
  float acc[HG][8];
#pragma unroll
  for (int h = 0; h < HG; ++h)
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[h][e] = 0.0f;
  auto add_row = [&](const uint4& v, int m) {
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
    float x[8];
#pragma unroll
    for (int e = 0; e < 4; ++e) { x[2 * e] = __uint_as_float(u[e] << 16); x[2 * e + 1] = __uint_as_float(u[e] & 0xffff0000u); }
#pragma unroll
    for (int h = 0; h < HG; ++h) {
      const float w = h < nh ? w_s[h * r4 + m] : 0.0f;
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[h][e] = fmaf(w, x[e], acc[h][e]);
    }
  };
#pragma unroll
  for (int i = 0; i < kPre; ++i) {
    const int m = rg + i * RPP;
    if (m < r) add_row(pre[i], m);
  }
  // the remaining rows four at a time, their loads issued together
  for (int m0 = rg + kPre * RPP; m0 < r; m0 += 4 * RPP) {
    uint4 nx[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int m = m0 + u * RPP;
      nx[u] = m < r ? *reinterpret_cast<const uint4*>(Bv + (size_t)m * ld) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int m = m0 + u * RPP;
      if (m < r) add_row(nx[u], m);
    }
  }
  // a warp holds two row groups (lanes 0..15 and 16..31 with the same columns): fold them, then one partial per warp
#pragma unroll
  for (int h = 0; h < HG; ++h)
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[h][e] += __shfl_xor_sync(0xffffffffu, acc[h][e], TPR);
  static_assert(TPR == 16 || TPR == 8, "row groups per warp");
  if constexpr (TPR == 8) {
#pragma unroll
    for (int h = 0; h < HG; ++h)
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[h][e] += __shfl_xor_sync(0xffffffffu, acc[h][e], 16);
  }
  if (lane < TPR) {
#pragma unroll
    for (int h = 0; h < HG; ++h)
#pragma unroll
      for (int e = 0; e < 8; ++e) red[(h * NW + warp) * DH + lane * 8 + e] = acc[h][e];
  }
  __syncthreads();
  for (int o = tid; o < nh * DH; o += kMergeMultiThreads) {
    const int h = o / DH, d = o - h * DH;
    float v = 0.0f;
#pragma unroll
    for (int w = 0; w < NW; ++w) v += red[(h * NW + w) * DH + d];
    if (tpart0) {
      const float* tpart = tpart0 + (size_t)h * (DH + 2);
      for (int sg = 0; sg < nts; ++sg) v = fmaf(twgt_s[h][sg], tpart[sg * tstride + d], v);
    }
    const float M = ML_s[h][0], L = ML_s[h][1];
    const long long qh = ((long long)l * dev.batch + b) * dev.H_q + (long long)g * n_rep + h0 + h;
    out[qh * DH + d] = __float2bfloat16(L > 0.0f ? v / L : 0.0f);
    if (lse && d == 0) lse[qh] = L > 0.0f ? (M + log2f(L)) * kLn2 : -INFINITY;
  }
}

template <int DH, int NR>
constexpr size_t fused_smem_bytes() {
  return 1024 + (size_t)(ring_slots<DH, NR>() + kNB) * kSlabBytes + misc_smem_bytes<DH, NR>();
}

template <int DH, int NR, int WB>
cudaError_t launch_fused_t(const xkv_group* grp, int l0, int l1, const __nv_bfloat16* q, const int32_t* sel_idx,
                           const int32_t* sel_cnt, int k_cap, __nv_bfloat16* out, float* lse, cudaStream_t s, TailParts tail) {
  const GroupDev& dev = grp->dev;
  const int problems = (l1 - l0) * dev.batch * dev.H_kv;
  Sched sc;
  sc.l0 = l0;
  sc.tpp = (k_cap + kTile - 1) / kTile;
  sc.n_tiles = problems * sc.tpp;
  sc.n_ctas = sc.n_tiles < grp->sm_count ? sc.n_tiles : grp->sm_count;
  sc.n_slots = fused_slots(grp);
  sc.k_cap = k_cap;
  sc.prof = grp->prof;
  static_assert(bar_layout(ring_slots<DH, NR>()).total <= 3 * 16 + kNB + 24, "barrier space");
  static_assert(kNB >= 2 && kNB < ring_slots<DH, NR>(), "B ring must be shorter than the row ring");
  static_assert(NR * WB <= 64 && WB <= kMaxBlocks, "value epilogue registers");
  const size_t smem = fused_smem_bytes<DH, NR>();
  CUtensorMap mk;
  memcpy(&mk, grp->bk_tmap, sizeof(mk));
  cudaError_t e;
  if (grp->prof) {     // the variant with the diagnostic counters compiled in
    if (dev.Aq_k) return cudaErrorNotSupported;        // no diagnostic variant of the quantised gather
    e = ensure_dyn_smem<sr_fused_kernel<DH, NR, WB, true, 0>>(smem, grp->device);
    if (e != cudaSuccess) return e;
    e = launch_pdl(sr_fused_kernel<DH, NR, WB, true, 0>, dim3(sc.n_ctas), dim3(kThreads), smem, s, mk, dev, sc, q, sel_idx, sel_cnt);
  } else if (dev.Aq_k && dev.quant_bits == 3) {
    e = ensure_dyn_smem<sr_fused_kernel<DH, NR, WB, false, 3>>(smem, grp->device);
    if (e != cudaSuccess) return e;
    e = launch_pdl(sr_fused_kernel<DH, NR, WB, false, 3>, dim3(sc.n_ctas), dim3(kThreads), smem, s, mk, dev, sc, q, sel_idx, sel_cnt);
  } else if (dev.Aq_k) {
    e = ensure_dyn_smem<sr_fused_kernel<DH, NR, WB, false, 4>>(smem, grp->device);
    if (e != cudaSuccess) return e;
    e = launch_pdl(sr_fused_kernel<DH, NR, WB, false, 4>, dim3(sc.n_ctas), dim3(kThreads), smem, s, mk, dev, sc, q, sel_idx, sel_cnt);
  } else {
    e = ensure_dyn_smem<sr_fused_kernel<DH, NR, WB, false, 0>>(smem, grp->device);
    if (e != cudaSuccess) return e;
    e = launch_pdl(sr_fused_kernel<DH, NR, WB, false, 0>, dim3(sc.n_ctas), dim3(kThreads), smem, s, mk, dev, sc, q, sel_idx, sel_cnt);
  }
  count_launch(kFamFused);
  if (e != cudaSuccess) return e;
  // one CTA per query head while those CTAs fit the SMs about twice over; beyond that one CTA per group of heads
  constexpr int HG = NR <= 4 ? 4 : 8;
  bool multi = false;
  if ((long long)problems * dev.n_rep <= 2LL * grp->sm_count) {
    const size_t msmem = sizeof(float) * (((size_t)dev.r_v + 3) / 4 * 4 + (size_t)(kMergeThreads / (DH / 8)) * DH);
    e = ensure_dyn_smem<merge_segments_kernel<DH>>(msmem, grp->device);
    if (e != cudaSuccess) return e;
    e = launch_pdl(merge_segments_kernel<DH>, dim3(problems * dev.n_rep), dim3(kMergeThreads), msmem, s, dev, sc, tail, out, lse);
  } else {
    const size_t msmem = sizeof(float) * ((size_t)HG * (((size_t)dev.r_v + 3) / 4 * 4) + (size_t)HG * (kMergeMultiThreads / 32) * DH);
    const int ngrp = (dev.n_rep + HG - 1) / HG;
    e = ensure_dyn_smem<merge_segments_multi_kernel<DH, HG>>(msmem, grp->device);
    if (e != cudaSuccess) return e;
    e = launch_pdl(merge_segments_multi_kernel<DH, HG>, dim3(problems * ngrp), dim3(kMergeMultiThreads), msmem, s, dev, sc, tail, out, lse);
    multi = true;
  }
  if (e != cudaSuccess) return e;
  count_launch(multi ? kFamMergeMulti : kFamMerge);
  return cudaGetLastError();
}

}  // namespace

// A problem never has more segments than there are CTAs + 1; the merge kernel's tables hold kMergeMaxSeg of them.
bool fused_sm_count_ok(int sm_count) { return sm_count >= 1 && sm_count + 1 <= kMergeMaxSeg; }

int fused_slots(const xkv_group* grp) {
  const int tpp_max = (grp->k_cap_max + kTile - 1) / kTile;
  return (tpp_max < grp->sm_count ? tpp_max : grp->sm_count) + 1;
}

size_t fused_part_floats(const xkv_group* grp) {
  const xkv_group_config& c = grp->cfg;
  return (size_t)c.G * c.batch * c.H_kv * fused_slots(grp) * (size_t)(c.H_q / c.H_kv) * (c.r_v + 2);
}

// The tensor-core path covers r_v up to 1024 (512 with more than 8 query heads per KV head).
bool fused_supported(const xkv_group* grp) {
  const int n_rep = grp->dev.n_rep, blocks = (grp->dev.r_v + 127) / 128;
  return blocks <= (n_rep <= 8 ? 8 : 4);
}

cudaError_t launch_fused(const xkv_group* grp, int l0, int l1, const __nv_bfloat16* q, const int32_t* sel_idx,
                         const int32_t* sel_cnt, int k_cap, __nv_bfloat16* out, float* lse, cudaStream_t s, TailParts tail) {
  const int n_rep = grp->dev.n_rep, blocks = (grp->dev.r_v + 127) / 128;   // WB: the smallest variant that holds r_v
#define XKV_DISPATCH(DH)                                                                                 \
  if (n_rep <= 4 && blocks <= 4) return launch_fused_t<DH, 4, 4>(grp, l0, l1, q, sel_idx, sel_cnt, k_cap, out, lse, s, tail);  \
  if (n_rep <= 4) return launch_fused_t<DH, 4, 8>(grp, l0, l1, q, sel_idx, sel_cnt, k_cap, out, lse, s, tail);  \
  if (n_rep <= 8 && blocks <= 4) return launch_fused_t<DH, 8, 4>(grp, l0, l1, q, sel_idx, sel_cnt, k_cap, out, lse, s, tail);  \
  if (n_rep <= 8) return launch_fused_t<DH, 8, 8>(grp, l0, l1, q, sel_idx, sel_cnt, k_cap, out, lse, s, tail);  \
  return launch_fused_t<DH, 16, 4>(grp, l0, l1, q, sel_idx, sel_cnt, k_cap, out, lse, s, tail);
  if (grp->dev.d_h == 128) { XKV_DISPATCH(128) }
  XKV_DISPATCH(64)
#undef XKV_DISPATCH
}

}  // namespace xkv
