// C ABI of libxkv: argument checking, handle life cycle, dispatch to the kernels.
#include <cuda.h>
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <new>

#include "xkv_internal.cuh"

namespace xkv {

static thread_local int g_last_cuda_error = 0;
static std::atomic<uint64_t> g_launches[kFamCount];

void set_cuda_error(cudaError_t e) { g_last_cuda_error = (int)e; }
void count_launch(KernelFamily family, int n) { g_launches[family].fetch_add((uint64_t)n, std::memory_order_relaxed); }

static int check_config(const xkv_group_config* c, bool need_ptrs) {
  if (!c) return XKV_ERR_INVALID_ARG;
  if (c->struct_size != sizeof(xkv_group_config)) return XKV_ERR_INVALID_ARG;
  if (c->G < 1 || c->batch < 1 || c->T < 1 || c->T >= (1 << 24)) return XKV_ERR_INVALID_ARG;
  if (c->H_kv < 1 || c->H_q < 1 || c->H_q % c->H_kv != 0) return XKV_ERR_INVALID_ARG;
  if (c->H_q / c->H_kv > kMaxRep) return XKV_ERR_INVALID_ARG;
  if (c->d_h != 64 && c->d_h != 128) return XKV_ERR_INVALID_ARG;
  if (c->r_k < 8 || c->r_v < 8 || c->r_k % 8 || c->r_v % 8) return XKV_ERR_INVALID_ARG;
  if (c->r_k > 8192 || c->r_v > 8192) return XKV_ERR_INVALID_ARG;
  if (c->chunk < 0 || c->chunk > 4096) return XKV_ERR_INVALID_ARG;
  if (c->k_max < 1) return XKV_ERR_INVALID_ARG;
  {
    // everything derived from k_max (row strides, tile counts, scratch sizes) has to stay in 32-bit range:
    // a budget beyond the context selects every row, so nothing larger than T rounded up to chunks is useful
    const int64_t ch = c->chunk ? c->chunk : 8;
    const int64_t k_cap = ((int64_t)c->k_max + ch - 1) / ch * ch;
    if (k_cap + (int64_t)XKV_MAX_OUTLIERS * ch >= ((int64_t)1 << 30)) return XKV_ERR_INVALID_ARG;
    // landmark rows are addressed by a 32-bit TMA coordinate; problems of a call are a grid dimension
    const int64_t n_c = ((int64_t)c->T + ch - 1) / ch;
    if ((int64_t)c->batch * c->G * c->H_kv * n_c >= ((int64_t)1 << 31)) return XKV_ERR_UNSUPPORTED;
    if ((int64_t)c->batch * c->G * c->H_kv > 65535) return XKV_ERR_UNSUPPORTED;
  }
  if (!(c->softmax_scale >= 0.0f) || isinf(c->softmax_scale)) return XKV_ERR_INVALID_ARG;
  if (isnan(c->rope_base) || isinf(c->rope_base)) return XKV_ERR_INVALID_ARG;
  if (need_ptrs) {
    // A_k / A_v may be NULL: the handle then serves reconstruct+attend only after xkv_group_set_quantized_bases
    if (!c->B_k || !c->B_v || (!c->A_k) != (!c->A_v)) return XKV_ERR_INVALID_ARG;
    const uintptr_t m = (uintptr_t)c->A_k | (uintptr_t)c->A_v | (uintptr_t)c->B_k | (uintptr_t)c->B_v |
                        (uintptr_t)c->landmarks;
    if (m & 15u) return XKV_ERR_INVALID_ARG;   // 16-byte vector loads and TMA need this
  }
  return XKV_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

// 2-D bf16 tensor [rows][cols] (cols fastest), box = box_rows x 64 columns, 128-byte swizzle.
static bool encode_rows64(void* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc((CUtensorMap*)out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims,
                   strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// 2-D bf16 tensor [rows][cols] with a row pitch of `pitch` elements, box = box_rows x 64 columns, 128-byte swizzle.
bool encode_bf16_map(void* out, const void* base, uint64_t rows, uint64_t cols, uint64_t pitch, uint32_t box_rows) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {pitch * 2};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc((CUtensorMap*)out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims,
                   strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool encode_landmark_map(void* out, const void* base, uint64_t rows, uint64_t cols) {
  return encode_rows64(out, base, rows, cols, kLandmarkBoxRows);
}

}  // namespace xkv

using namespace xkv;

#define XKV_TRY_CUDA(expr)                 \
  do {                                     \
    cudaError_t e_ = (expr);               \
    if (e_ != cudaSuccess) {               \
      set_cuda_error(e_);                  \
      (void)cudaGetLastError();            \
      st = (e_ == cudaErrorMemoryAllocation) ? XKV_ERR_OOM : XKV_ERR_CUDA; \
      goto fail;                           \
    }                                      \
  } while (0)

extern "C" {

const char* xkv_strerror(int s) {
  switch (s) {
    case XKV_OK: return "ok";
    case XKV_ERR_INVALID_ARG: return "invalid argument";
    case XKV_ERR_UNSUPPORTED: return "unsupported configuration";
    case XKV_ERR_ARCH: return "device is not sm_100 (B200)";
    case XKV_ERR_CUDA: return "CUDA runtime error";
    case XKV_ERR_OOM: return "out of device memory";
    case XKV_ERR_INDEX_RANGE: return "a selected row index was outside [0,T) and was skipped";
    case XKV_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out";
    case XKV_ERR_TOO_LARGE: return "problem exceeds the fixed scratch of the allocation-free entry point";
    default: return "unknown status";
  }
}

int xkv_last_cuda_error(void) { return g_last_cuda_error; }
uint64_t xkv_kernel_launch_count(void) {
  uint64_t n = 0;
  for (int f = 0; f < kFamCount; ++f) n += g_launches[f].load(std::memory_order_relaxed);
  return n;
}
int xkv_debug_launch_counts(uint64_t* counts) {
  if (!counts) return XKV_ERR_INVALID_ARG;
  for (int f = 0; f < kFamCount; ++f) counts[f] = g_launches[f].load(std::memory_order_relaxed);
  return XKV_OK;
}
int xkv_debug_set_fault_injection(xkv_group* g, uint32_t mask) {
  if (!g || (mask & ~(XKV_INJECT_SCAN_NO_LOAD | XKV_INJECT_FUSED_NO_B))) return XKV_ERR_INVALID_ARG;
  g->dev.inject = mask;
  return XKV_OK;
}

int xkv_group_bytes(const xkv_group_config* cfg, uint64_t* factor_bytes, uint64_t* landmark_bytes) {
  int st = check_config(cfg, false);
  if (st != XKV_OK) return st;
  const uint64_t c = cfg->chunk ? cfg->chunk : 8;
  const uint64_t d = (uint64_t)cfg->H_kv * cfg->d_h, T = cfg->T, G = cfg->G, B = cfg->batch;
  if (factor_bytes)
    *factor_bytes = B * 2 * (T * cfg->r_k + G * cfg->r_k * d + T * cfg->r_v + G * cfg->r_v * d);
  if (landmark_bytes) *landmark_bytes = B * 2 * G * ((T + c - 1) / c) * d;
  return XKV_OK;
}

int xkv_group_create(const xkv_group_config* cfg, void* stream, xkv_group** out) {
  if (!out) return XKV_ERR_INVALID_ARG;
  *out = nullptr;
  int st = check_config(cfg, true);
  if (st != XKV_OK) return st;
  cudaStream_t s = (cudaStream_t)stream;
  xkv_group* g = new (std::nothrow) xkv_group();
  if (!g) return XKV_ERR_OOM;
  memset(g, 0, sizeof(*g));
  g->cfg = *cfg;
  if (g->cfg.chunk == 0) g->cfg.chunk = 8;
  {
    cudaDeviceProp prop;
    XKV_TRY_CUDA(cudaGetDevice(&g->device));
    XKV_TRY_CUDA(cudaGetDeviceProperties(&prop, g->device));
    if (prop.major != 10) { st = XKV_ERR_ARCH; goto fail; }
    g->sm_count = prop.multiProcessorCount;
    if (!fused_sm_count_ok(g->sm_count)) { st = XKV_ERR_UNSUPPORTED; goto fail; }   // the segment merge's table size
  }
  {
    GroupDev& d = g->dev;
    const xkv_group_config& c = g->cfg;
    d.G = c.G; d.batch = c.batch; d.T = c.T; d.H_kv = c.H_kv; d.H_q = c.H_q; d.d_h = c.d_h;
    d.r_k = c.r_k; d.r_v = c.r_v; d.c = c.chunk; d.n_c = (c.T + c.chunk - 1) / c.chunk;
    d.n_rep = c.H_q / c.H_kv;
    // fine table of 8 positions (one landmark chunk); coarser splits keep the coarse table under 64 MB
    d.rope_shift = 3;
    while (((size_t)((c.T >> d.rope_shift) + 1) * (c.d_h / 2) * sizeof(float2)) > ((size_t)64 << 20)) d.rope_shift += 3;
    d.n_hi = (c.T + (1 << d.rope_shift) - 1) >> d.rope_shift;
    d.sel_scale = 1.0f / sqrtf((float)c.d_h);
    d.att_scale = c.softmax_scale > 0.0f ? c.softmax_scale : 1.0f / sqrtf((float)c.d_h);
    d.use_rope = c.rope_base > 0.0f;
    d.lm_const = 1;
    d.A_k = (const __nv_bfloat16*)c.A_k; d.A_v = (const __nv_bfloat16*)c.A_v;
    d.landmarks = (const __nv_bfloat16*)c.landmarks;
    g->k_cap_max = (int)(((int64_t)c.k_max + c.chunk - 1) / c.chunk) * c.chunk;

    const size_t heads = (size_t)c.batch * c.G * c.H_kv;
    const size_t btk = heads * kDP * c.r_k * sizeof(__nv_bfloat16);
    const size_t btv = heads * kDP * c.r_v * sizeof(__nv_bfloat16);
    const size_t pooled = c.landmarks ? heads * d.n_c * sizeof(float) : 0;
    const size_t hi = (size_t)d.n_hi * (c.d_h / 2) * sizeof(float2);
    const size_t lo = ((size_t)1 << d.rope_shift) * (c.d_h / 2) * sizeof(float2);
    const size_t pf0 = attend_part_floats(g), pf1 = fused_part_floats(g);
    const size_t part = (pf0 > pf1 ? pf0 : pf1) * sizeof(float);
    void* p = nullptr;
#define XKV_ALLOC(dst, type, bytes)                        \
    do {                                                   \
      XKV_TRY_CUDA(cudaMalloc(&p, (bytes) ? (bytes) : 16)); \
      g->owned[g->n_owned++] = p;                          \
      dst = (type)p;                                       \
      g->workspace_bytes += (bytes);                       \
    } while (0)
    __nv_bfloat16 *Bt_k, *Bt_v, *Bv_copy; float2 *rhi, *rlo;
    XKV_ALLOC(Bt_k, __nv_bfloat16*, btk);
    XKV_ALLOC(Bt_v, __nv_bfloat16*, btv);
    XKV_ALLOC(Bv_copy, __nv_bfloat16*, (size_t)c.batch * c.G * c.r_v * c.H_kv * c.d_h * sizeof(__nv_bfloat16));
    XKV_ALLOC(d.pooled, float*, pooled);
    XKV_ALLOC(rhi, float2*, hi);
    XKV_ALLOC(rlo, float2*, lo);
    XKV_ALLOC(d.part, float*, part);
    XKV_ALLOC(d.flags, unsigned int*, 256);
#undef XKV_ALLOC
    d.Bt_k = Bt_k; d.Bt_v = Bt_v; d.B_v = Bv_copy; d.rope_hi = rhi; d.rope_lo = rlo;
    XKV_TRY_CUDA(cudaMemcpyAsync(Bv_copy, c.B_v, (size_t)c.batch * c.G * c.r_v * c.H_kv * c.d_h * sizeof(__nv_bfloat16),
                                 cudaMemcpyDeviceToDevice, s));
    XKV_TRY_CUDA(cudaMemsetAsync(d.flags, 0, 256, s));
    XKV_TRY_CUDA(launch_repack_b((const __nv_bfloat16*)c.B_k, Bt_k, c.batch, c.G, c.r_k, c.H_kv, c.d_h, s));
    XKV_TRY_CUDA(launch_repack_b((const __nv_bfloat16*)c.B_v, Bt_v, c.batch, c.G, c.r_v, c.H_kv, c.d_h, s));
    XKV_TRY_CUDA(launch_rope_tables(rhi, rlo, d.n_hi, d.rope_shift, c.d_h, c.rope_base > 0 ? (double)c.rope_base : 1.0, s));
    XKV_TRY_CUDA(cudaStreamSynchronize(s));

    if (c.landmarks) {
      const uint64_t rows = (uint64_t)heads * d.n_c;
      g->has_lm_tmap = encode_landmark_map(g->lm_tmap, c.landmarks, rows, (uint64_t)c.d_h) ? 1 : 0;
      if (!g->has_lm_tmap) { st = XKV_ERR_CUDA; goto fail; }
    }
    // Tensor maps over the repacked B blocks (row pitch r*2 bytes is a multiple of 16 because r % 8 == 0;
    // a slab that reaches past column r is zero-filled by the copy engine).
    g->has_b_tmap = encode_rows64(g->bk_tmap, Bt_k, heads * kDP, (uint64_t)c.r_k, kDP) &&
                    encode_rows64(g->bv_tmap, Bt_v, heads * kDP, (uint64_t)c.r_v, kDP);
    if (!g->has_b_tmap) { st = XKV_ERR_CUDA; goto fail; }
    {
      const char* e = getenv("XKV_ATTEND_IMPL");
      g->attend_impl = (e && e[0] == 't') ? 1 : 0;
      const char* te = getenv("XKV_TAIL_IMPL");
      g->tail_impl = (te && te[0] == 'c') ? 1 : 0;
      const char* pe = getenv("XKV_FUSED_PROF");
      if (pe && pe[0] == '1') {
        XKV_TRY_CUDA(cudaMalloc(&p, (size_t)g->sm_count * 64 * sizeof(unsigned long long)));
        g->owned[g->n_owned++] = p;
        g->prof = (unsigned long long*)p;
        XKV_TRY_CUDA(cudaMemset(p, 0, (size_t)g->sm_count * 64 * sizeof(unsigned long long)));
      }
    }
  }
  *out = g;
  return XKV_OK;
fail:
  for (int i = 0; i < g->n_owned; ++i) cudaFree(g->owned[i]);
  delete g;
  return st;
}

int xkv_group_destroy(xkv_group* g) {
  if (!g) return XKV_OK;
  int st = XKV_OK;
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) { set_cuda_error(e); st = XKV_ERR_CUDA; }
  for (int i = 0; i < g->n_owned; ++i) cudaFree(g->owned[i]);
  delete g;
  return st;
}

int xkv_group_workspace_bytes(const xkv_group* g, uint64_t* bytes) {
  if (!g || !bytes) return XKV_ERR_INVALID_ARG;
  *bytes = g->workspace_bytes;
  return XKV_OK;
}

int xkv_group_status(xkv_group* g, uint32_t* device_flags, void* stream) {
  if (!g) return XKV_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  unsigned int f = 0;
  cudaError_t e = cudaMemcpyAsync(&f, g->dev.flags, sizeof(f), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(g->dev.flags, 0, sizeof(f), s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) { set_cuda_error(e); return XKV_ERR_CUDA; }
  if (device_flags) *device_flags = f;
  if (f & XKV_FLAG_TIMEOUT) return XKV_ERR_TIMEOUT;
  if (f & XKV_FLAG_INDEX_RANGE) return XKV_ERR_INDEX_RANGE;
  return XKV_OK;
}

int xkv_sr_select_static(const xkv_select_static_config* cfg, int layer_begin, int layer_end, const void* q,
                         int32_t k, int32_t* sel_idx, int32_t* sel_cnt, void* stream) {
  return select_static(cfg, layer_begin, layer_end, q, k, sel_idx, sel_cnt, (cudaStream_t)stream);
}

int xkv_debug_read_profile(xkv_group* g, uint64_t* out, int max_words) {
  if (!g || !out || max_words < 0) return XKV_ERR_INVALID_ARG;
  if (!g->prof) return XKV_ERR_UNSUPPORTED;
  size_t n = (size_t)g->sm_count * 64;
  if ((size_t)max_words < n) n = (size_t)max_words;
  cudaError_t e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemcpy(out, g->prof, n * sizeof(uint64_t), cudaMemcpyDeviceToHost);
  if (e == cudaSuccess) e = cudaMemset(g->prof, 0, (size_t)g->sm_count * 64 * sizeof(uint64_t));
  if (e != cudaSuccess) { set_cuda_error(e); return XKV_ERR_CUDA; }
  return (int)n;
}

int xkv_sr_select(xkv_group* g, int layer_begin, int layer_end, const void* q, int32_t k, int32_t* sel_idx,
                  int32_t* sel_cnt, void* stream) {
  if (!g || !q || !sel_idx || !sel_cnt) return XKV_ERR_INVALID_ARG;
  if (!g->cfg.landmarks) return XKV_ERR_INVALID_ARG;
  if (layer_begin < 0 || layer_end > g->cfg.G || layer_begin >= layer_end) return XKV_ERR_INVALID_ARG;
  if (k < 1 || k > g->cfg.k_max) return XKV_ERR_INVALID_ARG;
  if (((uintptr_t)q & 15u) || ((uintptr_t)sel_idx & 3u) || ((uintptr_t)sel_cnt & 3u)) return XKV_ERR_INVALID_ARG;
  cudaError_t e = launch_select(g, layer_begin, layer_end, (const __nv_bfloat16*)q, k, sel_idx, sel_cnt,
                                (cudaStream_t)stream);
  if (e != cudaSuccess) { set_cuda_error(e); (void)cudaGetLastError(); return XKV_ERR_CUDA; }
  return XKV_OK;
}

int xkv_sr_reconstruct_attend(xkv_group* g, int layer_begin, int layer_end, const void* q,
                              const int32_t* sel_idx, const int32_t* sel_cnt, int32_t k_cap, void* out,
                              float* lse, void* stream) {
  if (!g || !q || !sel_idx || !sel_cnt || !out) return XKV_ERR_INVALID_ARG;
  if (layer_begin < 0 || layer_end > g->cfg.G || layer_begin >= layer_end) return XKV_ERR_INVALID_ARG;
  if (k_cap < 1 || k_cap > g->k_cap_max) return XKV_ERR_INVALID_ARG;
  if (!g->dev.A_k && !g->dev.Aq_k) return XKV_ERR_INVALID_ARG;      // created without bases and none set since
  if (((uintptr_t)q & 15u) || ((uintptr_t)out & 15u) || ((uintptr_t)sel_idx & 3u) ||
      ((uintptr_t)sel_cnt & 3u) || ((uintptr_t)lse & 3u))
    return XKV_ERR_INVALID_ARG;
  if (g->dev.Aq_k && (g->attend_impl || !fused_supported(g))) return XKV_ERR_UNSUPPORTED;   // codes: tensor-core path only
  cudaError_t e = (g->attend_impl || !fused_supported(g))
                      ? launch_reconstruct_attend(g, layer_begin, layer_end, (const __nv_bfloat16*)q, sel_idx, sel_cnt,
                                                  k_cap, (__nv_bfloat16*)out, lse, (cudaStream_t)stream)
                      : launch_fused(g, layer_begin, layer_end, (const __nv_bfloat16*)q, sel_idx, sel_cnt, k_cap,
                                     (__nv_bfloat16*)out, lse, (cudaStream_t)stream);
  if (e != cudaSuccess) { set_cuda_error(e); (void)cudaGetLastError(); return XKV_ERR_CUDA; }
  return XKV_OK;
}

int xkv_build_landmarks(const xkv_landmark_config* c, const void* keys, void* landmarks, float* min_cos,
                        int32_t n_outliers, int32_t* outliers, void* stream) {
  if (!c || c->struct_size != sizeof(xkv_landmark_config) || !keys || !landmarks) return XKV_ERR_INVALID_ARG;
  if (c->G < 1 || c->batch < 1 || c->T < 1 || c->T >= (1 << 24) || c->H_kv < 1 || (c->d_h != 64 && c->d_h != 128) ||
      c->H_kv * c->d_h > 4096 || c->chunk < 0 || c->chunk > 4096 || isnan(c->rope_base) || isinf(c->rope_base))
    return XKV_ERR_INVALID_ARG;
  if (n_outliers < 0 || n_outliers > XKV_MAX_OUTLIERS || (n_outliers > 0 && (!outliers || !min_cos))) return XKV_ERR_INVALID_ARG;
  if (256 % (c->H_kv * c->d_h / 16) != 0) return XKV_ERR_UNSUPPORTED;   // threads per key row must divide the CTA
  if (((uintptr_t)keys & 15u) || ((uintptr_t)landmarks & 15u)) return XKV_ERR_INVALID_ARG;   // 16-byte loads and stores
  if (((uintptr_t)keys & 1u) || ((uintptr_t)landmarks & 1u) || ((uintptr_t)min_cos & 15u) || ((uintptr_t)outliers & 3u))
    return XKV_ERR_INVALID_ARG;
  int device = 0, cc_major = 0;
  cudaError_t e = cudaGetDevice(&device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, device);
  if (e != cudaSuccess) { set_cuda_error(e); (void)cudaGetLastError(); return XKV_ERR_CUDA; }
  if (cc_major != 10) return XKV_ERR_ARCH;
  const int ch = c->chunk ? c->chunk : 8;
  const int n_c = (c->T + ch - 1) / ch;
  cudaStream_t s = (cudaStream_t)stream;
  e = launch_landmarks((const __nv_bfloat16*)keys, (__nv_bfloat16*)landmarks, min_cos, c->G, c->batch, c->T, c->H_kv,
                       c->d_h, ch, c->rope_base, s);
  if (e == cudaSuccess && n_outliers > 0)
    e = launch_topk_rows(min_cos, c->G * c->batch * c->H_kv, n_c, n_outliers, -1.0f, outliers, device, s);
  if (e != cudaSuccess) { set_cuda_error(e); (void)cudaGetLastError(); return XKV_ERR_CUDA; }
  return XKV_OK;
}

int xkv_group_set_outliers(xkv_group* g, const int32_t* outliers, int32_t n_outliers, void* stream) {
  if (!g || n_outliers < 0 || n_outliers > XKV_MAX_OUTLIERS) return XKV_ERR_INVALID_ARG;
  if (n_outliers > 0 && (!outliers || ((uintptr_t)outliers & 3u))) return XKV_ERR_INVALID_ARG;
  if (!g->cfg.landmarks) return XKV_ERR_INVALID_ARG;
  // nothing of this handle may be in flight while its scratch is replaced
  cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
  if (e != cudaSuccess) { set_cuda_error(e); return XKV_ERR_CUDA; }
  const int c = g->dev.c;
  const int old_cap = g->k_cap_max;
  g->k_cap_max = (int)(((int64_t)g->cfg.k_max + c - 1) / c) * c + n_outliers * c;
  if (g->k_cap_max > old_cap) {
    // the partial results of reconstruct+attend are sized by the largest row count of a selection
    const size_t pf0 = attend_part_floats(g), pf1 = fused_part_floats(g);
    const size_t bytes = (pf0 > pf1 ? pf0 : pf1) * sizeof(float);
    void* p = nullptr;
    e = cudaMalloc(&p, bytes ? bytes : 16);
    if (e != cudaSuccess) {
      g->k_cap_max = old_cap;
      set_cuda_error(e);
      (void)cudaGetLastError();
      return e == cudaErrorMemoryAllocation ? XKV_ERR_OOM : XKV_ERR_CUDA;
    }
    for (int i = 0; i < g->n_owned; ++i) {
      if (g->owned[i] == (void*)g->dev.part) { cudaFree(g->owned[i]); g->owned[i] = p; }
    }
    g->dev.part = (float*)p;
  }
  g->dev.outliers = n_outliers > 0 ? outliers : nullptr;
  g->dev.n_out = n_outliers;
  return XKV_OK;
}

int xkv_tail_workspace_bytes(const xkv_group* g, int32_t tail_cap, uint64_t* bytes) {
  if (!g || !bytes || tail_cap < 1 || tail_cap > XKV_TAIL_MAX_ROWS) return XKV_ERR_INVALID_ARG;
  *bytes = (uint64_t)tail_part_floats(g, tail_cap) * sizeof(float);
  return XKV_OK;
}

int xkv_sr_reconstruct_attend_tail(xkv_group* g, int layer_begin, int layer_end, const void* q,
                                   const int32_t* sel_idx, const int32_t* sel_cnt, int32_t k_cap,
                                   const void* tail_k, const void* tail_v, const int32_t* tail_len,
                                   int32_t tail_cap, void* workspace, uint64_t workspace_bytes, void* out,
                                   float* lse, void* stream) {
  if (!g || !q || !sel_idx || !sel_cnt || !out || !tail_k || !tail_v || !workspace) return XKV_ERR_INVALID_ARG;
  if (layer_begin < 0 || layer_end > g->cfg.G || layer_begin >= layer_end) return XKV_ERR_INVALID_ARG;
  if (k_cap < 1 || k_cap > g->k_cap_max) return XKV_ERR_INVALID_ARG;
  if (tail_cap < 1 || tail_cap > XKV_TAIL_MAX_ROWS) return XKV_ERR_INVALID_ARG;
  if (!g->dev.A_k && !g->dev.Aq_k) return XKV_ERR_INVALID_ARG;
  if (workspace_bytes < (uint64_t)tail_part_floats(g, tail_cap) * sizeof(float)) return XKV_ERR_INVALID_ARG;
  if (((uintptr_t)q & 15u) || ((uintptr_t)out & 15u) || ((uintptr_t)sel_idx & 3u) || ((uintptr_t)sel_cnt & 3u) ||
      ((uintptr_t)lse & 3u) || ((uintptr_t)tail_k & 15u) || ((uintptr_t)tail_v & 15u) || ((uintptr_t)tail_len & 3u) ||
      ((uintptr_t)workspace & 15u))
    return XKV_ERR_INVALID_ARG;
  if (g->attend_impl || !fused_supported(g)) return XKV_ERR_UNSUPPORTED;
  cudaStream_t s = (cudaStream_t)stream;
  cudaError_t e = launch_tail_partials(g, layer_begin, layer_end, (const __nv_bfloat16*)q, (const __nv_bfloat16*)tail_k,
                                       (const __nv_bfloat16*)tail_v, tail_len, tail_cap, (float*)workspace, s);
  if (e == cudaSuccess)
    e = launch_fused(g, layer_begin, layer_end, (const __nv_bfloat16*)q, sel_idx, sel_cnt, k_cap, (__nv_bfloat16*)out,
                     lse, s, TailParts{(const float*)workspace, tail_splits(tail_cap)});
  if (e != cudaSuccess) { set_cuda_error(e); (void)cudaGetLastError(); return XKV_ERR_CUDA; }
  return XKV_OK;
}

static int current_sm100_device(int* device) {
  int major = 0;
  cudaError_t e = cudaGetDevice(device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, *device);
  if (e != cudaSuccess) { set_cuda_error(e); (void)cudaGetLastError(); return XKV_ERR_CUDA; }
  return major == 10 ? XKV_OK : XKV_ERR_ARCH;
}

int xkv_clf_rank_l(const xkv_clf_config* cfg, int32_t* l) {
  if (!l) return XKV_ERR_INVALID_ARG;
  int v = 0;
  const int st = clf_rank_l(cfg, &v);
  if (st == XKV_OK) *l = v;
  return st;
}

int xkv_clf_workspace_bytes(const xkv_clf_config* cfg, uint64_t* bytes) {
  if (!bytes) return XKV_ERR_INVALID_ARG;
  return clf_workspace_bytes(cfg, bytes);
}

int xkv_clf_factorize(const xkv_clf_config* cfg, const void* X, const void* omega, void* workspace,
                      uint64_t workspace_bytes, void* A, void* B, float* sigma, void* stream) {
  if (!X || !omega || !workspace || !A || !B) return XKV_ERR_INVALID_ARG;
  if (((uintptr_t)X & 15u) || ((uintptr_t)omega & 15u) || ((uintptr_t)workspace & 255u) || ((uintptr_t)A & 15u) ||
      ((uintptr_t)B & 15u) || ((uintptr_t)sigma & 3u))
    return XKV_ERR_INVALID_ARG;
  uint64_t need = 0;
  int st = clf_workspace_bytes(cfg, &need);                  // also validates cfg
  if (st != XKV_OK) return st;
  if (workspace_bytes < need) return XKV_ERR_INVALID_ARG;
  int device = 0;
  st = current_sm100_device(&device);
  if (st != XKV_OK) return st;
  return clf_factorize(cfg, X, omega, workspace, workspace_bytes, A, B, sigma, device, (cudaStream_t)stream);
}

int xkv_debug_set_clf_fault_injection(uint32_t mask) {
  if (mask & ~XKV_INJECT_CLF_BARRIER) return XKV_ERR_INVALID_ARG;
  clf_set_fault_injection(mask);
  return XKV_OK;
}

int xkv_clf_status(const void* workspace, uint32_t* flags, void* stream) {
  if (!workspace) return XKV_ERR_INVALID_ARG;
  unsigned int f = 0;
  cudaStream_t s = (cudaStream_t)stream;
  cudaError_t e = cudaMemcpyAsync(&f, workspace, sizeof(f), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) { set_cuda_error(e); return XKV_ERR_CUDA; }
  if (flags) *flags = f;
  if (f & XKV_FLAG_TIMEOUT) return XKV_ERR_TIMEOUT;
  return XKV_OK;
}

int xkv_debug_gemm(const void* a, const void* b, int32_t M, int32_t N, int32_t K, float* C, uint32_t* flags, void* stream) {
  if (!a || !b || !C || !flags || M < 1 || N < 1 || K < 1 || (M % 8) || (K % 8)) return XKV_ERR_INVALID_ARG;
  if (((uintptr_t)a & 15u) || ((uintptr_t)b & 15u) || ((uintptr_t)C & 3u)) return XKV_ERR_INVALID_ARG;
  int device = 0;
  const int st = current_sm100_device(&device);
  if (st != XKV_OK) return st;
  cudaError_t e = clf_gemm(a, b, M, N, K, C, flags, device, (cudaStream_t)stream);
  if (e != cudaSuccess) { set_cuda_error(e); (void)cudaGetLastError(); return XKV_ERR_CUDA; }
  return XKV_OK;
}

// x and codes are required; meta only for 4 bits (the 3-bit records carry their scale and offset)
static int check_rtn_args(const void* x, const void* codes, const void* meta, int64_t rows, int32_t cols, int32_t bits) {
  if (bits < 1 || bits > 8) return XKV_ERR_INVALID_ARG;
  if (!x || !codes || rows < 0 || cols < 32 || cols % 32 != 0) return XKV_ERR_INVALID_ARG;
  if (((uintptr_t)x & 15u) || ((uintptr_t)codes & 15u) || ((uintptr_t)meta & 15u)) return XKV_ERR_INVALID_ARG;
  if (bits != 4 && bits != 3) return XKV_ERR_UNSUPPORTED;
  if (bits == 4 && !meta) return XKV_ERR_INVALID_ARG;
  return XKV_OK;
}

int xkv_quantize_rtn(const void* x, int64_t rows, int32_t cols, int32_t bits, void* codes, void* meta, void* stream) {
  const int st = check_rtn_args(x, codes, meta, rows, cols, bits);
  if (st != XKV_OK) return st;
  cudaError_t e = bits == 4 ? launch_quantize_rtn4((const __nv_bfloat16*)x, rows, cols, codes, meta, (cudaStream_t)stream)
                            : launch_quantize_rtn3((const __nv_bfloat16*)x, rows, cols, codes, (cudaStream_t)stream);
  if (e != cudaSuccess) { set_cuda_error(e); (void)cudaGetLastError(); return XKV_ERR_CUDA; }
  return XKV_OK;
}

int xkv_dequantize_rtn(const void* codes, const void* meta, int64_t rows, int32_t cols, int32_t bits, void* x, void* stream) {
  const int st = check_rtn_args(x, codes, meta, rows, cols, bits);
  if (st != XKV_OK) return st;
  cudaError_t e = bits == 4 ? launch_dequantize_rtn4(codes, meta, rows, cols, (__nv_bfloat16*)x, (cudaStream_t)stream)
                            : launch_dequantize_rtn3(codes, rows, cols, (__nv_bfloat16*)x, (cudaStream_t)stream);
  if (e != cudaSuccess) { set_cuda_error(e); (void)cudaGetLastError(); return XKV_ERR_CUDA; }
  return XKV_OK;
}

int xkv_group_set_quantized_bases(xkv_group* g, const void* codes_k, const void* meta_k, const void* codes_v,
                                  const void* meta_v, int32_t bits) {
  if (!g) return XKV_ERR_INVALID_ARG;
  if (!codes_k && !meta_k && !codes_v && !meta_v) {
    g->dev.Aq_k = g->dev.Aq_v = nullptr; g->dev.Am_k = g->dev.Am_v = nullptr; g->dev.quant_bits = 0;
    return XKV_OK;
  }
  if (bits < 1 || bits > 8) return XKV_ERR_INVALID_ARG;
  if (bits != 4 && bits != 3) return XKV_ERR_UNSUPPORTED;
  if (!codes_k || !codes_v || (bits == 4 && (!meta_k || !meta_v))) return XKV_ERR_INVALID_ARG;
  if (((uintptr_t)codes_k | (uintptr_t)meta_k | (uintptr_t)codes_v | (uintptr_t)meta_v) & 15u) return XKV_ERR_INVALID_ARG;
  if (g->cfg.r_k % 32 != 0 || g->cfg.r_v % 32 != 0 || !fused_supported(g)) return XKV_ERR_UNSUPPORTED;
  g->dev.Aq_k = (const uint8_t*)codes_k; g->dev.Am_k = (const uint32_t*)meta_k;
  g->dev.Aq_v = (const uint8_t*)codes_v; g->dev.Am_v = (const uint32_t*)meta_v;
  g->dev.quant_bits = bits;
  return XKV_OK;
}

int xkv_dense_workspace_bytes(const xkv_group* g, int32_t cap, uint64_t* bytes) {
  if (!g || !bytes || cap < 1 || cap > XKV_DENSE_MAX_ROWS) return XKV_ERR_INVALID_ARG;
  if (!dense_supported(g, cap)) return XKV_ERR_UNSUPPORTED;
  *bytes = (uint64_t)tail_part_floats(g, cap) * sizeof(float);
  return XKV_OK;
}

int xkv_dense_attend(xkv_group* g, int layer_begin, int layer_end, const void* q, const void* K, const void* V,
                     const int32_t* len, int32_t cap, void* workspace, uint64_t workspace_bytes, void* out, float* lse,
                     void* stream) {
  if (!g || !q || !K || !V || !workspace || !out) return XKV_ERR_INVALID_ARG;
  if (layer_begin < 0 || layer_end > g->cfg.G || layer_begin >= layer_end) return XKV_ERR_INVALID_ARG;
  if (cap < 1 || cap > XKV_DENSE_MAX_ROWS) return XKV_ERR_INVALID_ARG;
  if (!dense_supported(g, cap)) return XKV_ERR_UNSUPPORTED;
  if (workspace_bytes < (uint64_t)tail_part_floats(g, cap) * sizeof(float)) return XKV_ERR_INVALID_ARG;
  if (((uintptr_t)q & 15u) || ((uintptr_t)out & 15u) || ((uintptr_t)lse & 3u) || ((uintptr_t)K & 15u) ||
      ((uintptr_t)V & 15u) || ((uintptr_t)len & 3u) || ((uintptr_t)workspace & 15u))
    return XKV_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  cudaError_t e = launch_tail_partials(g, layer_begin, layer_end, (const __nv_bfloat16*)q, (const __nv_bfloat16*)K,
                                       (const __nv_bfloat16*)V, len, cap, (float*)workspace, s);
  if (e == cudaSuccess)
    e = launch_dense_merge(g, layer_begin, layer_end, (const float*)workspace, cap, (__nv_bfloat16*)out, lse, s);
  if (e != cudaSuccess) { set_cuda_error(e); (void)cudaGetLastError(); return XKV_ERR_CUDA; }
  return XKV_OK;
}

}  // extern "C"
