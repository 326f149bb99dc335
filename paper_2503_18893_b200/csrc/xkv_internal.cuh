// Internal declarations shared by the translation units of libxkv (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include <atomic>

#include "xkv.h"

namespace xkv {

constexpr int kDP = 128;          // rows of a repacked B head block (d_h padded to 128 with zeros)
constexpr int kMaxRep = 16;       // query heads per KV head
constexpr int kAttTile = 128;     // selected rows per attention tile
constexpr int kLandmarkBoxRows = 64;   // landmark rows per TMA box = chunks scored per CTA of the landmark scan
constexpr int kTailSplitRows = 128;     // tail rows per partial result
constexpr int kTailMaxSplit = XKV_TAIL_MAX_ROWS / kTailSplitRows;
constexpr int kMaxSplit = 64;     // most partial results per (layer, sequence, head) problem

// Device-side description of one window; a copy lives in the handle and is passed by value.
struct GroupDev {
  int G, batch, T, H_kv, H_q, d_h, r_k, r_v, c, n_c, n_rep;
  int rope_shift;                   // fine rotary table covers 2^rope_shift consecutive positions
  int n_hi;                         // entries per frequency of the coarse table: ceil(T / 2^rope_shift)
  float sel_scale;                  // 1/sqrt(d_h) computed on the host (Algorithm 2, line 2)
  float att_scale;                  // softmax scale of the attention
  int use_rope;
  const __nv_bfloat16* A_k;         // [batch][T][r_k]
  const __nv_bfloat16* A_v;         // [batch][T][r_v]
  const __nv_bfloat16* landmarks;   // [batch][G][H_kv][n_c][d_h]
  const __nv_bfloat16* Bt_k;        // [batch][G][H_kv][kDP][r_k]  transposed head blocks, zero padded
  const __nv_bfloat16* Bt_v;        // [batch][G][H_kv][kDP][r_v]
  const __nv_bfloat16* B_v;         // [batch][G][r_v][H_kv*d_h]   owned copy in the caller's layout
  const float2* rope_hi;            // [n_hi][d_h/2]          (cos, sin) of (p_hi << rope_shift) * theta_i
  const float2* rope_lo;            // [2^rope_shift][d_h/2]  (cos, sin) of p_lo * theta_i
  float* pooled;                    // [G][batch][H_kv][n_c] pooled landmark scores
  float* part;                      // attention partials, see xkv_attend.cu
  unsigned int* flags;              // device flag word
  const int32_t* outliers;          // [G][batch][H_kv][n_out] static outlier chunk ids (Algorithm 2 line 5), or nullptr
  int n_out;
  int quant_bits;                   // 0: bf16 bases; 4: codes + scale/offset words; 3: 16-byte records in Aq_* (Am_* unused)
  const uint8_t* Aq_k;              // codes of A_k [batch][T][r_k/2], or nullptr (then the bf16 bases are gathered)
  const uint8_t* Aq_v;              // [batch][T][r_v/2]
  const uint32_t* Am_k;             // scale/offset words [batch][T][r_k/32]
  const uint32_t* Am_v;             // [batch][T][r_v/32]
  int lm_const;                     // 1: the landmarks do not change while the handle lives (loads may run ahead of the stream)
  unsigned int inject;              // XKV_INJECT_* bits (xkv_debug_set_fault_injection); 0 in normal use
};

}  // namespace xkv

struct xkv_group {
  xkv_group_config cfg;
  xkv::GroupDev dev;
  int device;
  int sm_count;
  int k_cap_max;                    // ceil(k_max/c)*c
  size_t workspace_bytes;
  void* owned[12];
  int n_owned;
  alignas(64) unsigned char lm_tmap[128];   // CUtensorMap for the landmark scan
  int has_lm_tmap;
  alignas(64) unsigned char bk_tmap[128];   // CUtensorMap over Bt_k rows
  alignas(64) unsigned char bv_tmap[128];   // CUtensorMap over Bt_v rows
  int has_b_tmap;
  unsigned long long* prof;         // diagnostic cycle counters of the fused kernel, or nullptr
  int attend_impl;                  // 0: tensor-core fused kernel, 1: plain tile kernel
  int tail_impl;                    // 0: tensor-core tail partials where they apply (d_h = 128), 1: CUDA-core kernel
};

namespace xkv {

void set_cuda_error(cudaError_t e);

// Launch with programmatic stream serialization: the kernel may begin while the previous kernel of the stream
// drains; it must execute griddepcontrol.wait before it reads anything an earlier kernel may have written.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}
// Kernel families of the launch accounting (xkv_debug_launch_counts reports one counter per family).
enum KernelFamily {
  kFamScan = XKV_KERNEL_SCAN, kFamTopk = XKV_KERNEL_TOPK, kFamFused = XKV_KERNEL_FUSED, kFamMerge = XKV_KERNEL_MERGE,
  kFamTile = XKV_KERNEL_TILE, kFamTailTc = XKV_KERNEL_TAIL_TC, kFamTailCuda = XKV_KERNEL_TAIL_CUDA,
  kFamLandmarks = XKV_KERNEL_LANDMARKS, kFamPrep = XKV_KERNEL_PREP, kFamDense = XKV_KERNEL_DENSE, kFamClf = XKV_KERNEL_CLF, kFamMergeMulti = XKV_KERNEL_MERGE_MULTI,
  kFamCount = XKV_KERNEL_FAMILIES
};
void count_launch(KernelFamily family, int n = 1);

// cudaFuncAttributeMaxDynamicSharedMemorySize of one kernel, set once per device instead of on every launch (the
// attribute is sticky; re-issuing it costs host time on the launch path).  `Kernel` is the kernel's address, so
// every instantiation keeps its own record.
constexpr int kMaxDevices = 64;
template <auto Kernel>
inline cudaError_t ensure_dyn_smem(size_t bytes, int device) {
  static std::atomic<size_t> have[kMaxDevices];
  if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
  if (have[device].load(std::memory_order_acquire) >= bytes && bytes > 0) return cudaSuccess;
  // the default limit of 48 KB covers static and dynamic shared memory together
  static std::atomic<long> static_bytes{-1};
  long st = static_bytes.load(std::memory_order_acquire);
  if (st < 0) {
    cudaFuncAttributes attr;
    const cudaError_t ea = cudaFuncGetAttributes(&attr, Kernel);
    if (ea != cudaSuccess) return ea;
    st = (long)attr.sharedSizeBytes;
    static_bytes.store(st, std::memory_order_release);
  }
  if (bytes + (size_t)st <= 48 * 1024) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(Kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess) have[device].store(bytes, std::memory_order_release);
  return e;
}

// xkv_prep.cu
cudaError_t launch_repack_b(const __nv_bfloat16* B, __nv_bfloat16* Bt, int batch, int G, int r, int H_kv,
                            int d_h, cudaStream_t s);
cudaError_t launch_rope_tables(float2* hi, float2* lo, int n_hi, int rope_shift, int d_h, double base,
                               cudaStream_t s);

// xkv_select.cu
cudaError_t launch_select(const xkv_group* grp, int l0, int l1, const __nv_bfloat16* q, int k,
                          int32_t* sel_idx, int32_t* sel_cnt, cudaStream_t s);

cudaError_t launch_topk_rows(const float* scores, int problems, int n, int k, float sign, int32_t* out, int device,
                             cudaStream_t s);

// xkv_landmarks.cu
cudaError_t launch_landmarks(const __nv_bfloat16* keys, __nv_bfloat16* landmarks, float* min_cos, int G, int batch, int T,
                             int H_kv, int d_h, int c, float rope_base, cudaStream_t s);

bool select_stride_ok(int64_t k, int c, int n_out);
int select_static(const xkv_select_static_config* c, int l0, int l1, const void* q, int32_t k, int32_t* sel_idx,
                  int32_t* sel_cnt, cudaStream_t s);
// xkv_api.cu: tensor map over [rows][cols] bf16 landmarks, kLandmarkBoxRows-row boxes of 64 columns, 128-byte swizzle
bool encode_landmark_map(void* out, const void* base, uint64_t rows, uint64_t cols);
// the same for a general bf16 matrix [rows][cols] with a row pitch (elements) and box_rows-row boxes of 64 columns
bool encode_bf16_map(void* out, const void* base, uint64_t rows, uint64_t cols, uint64_t pitch, uint32_t box_rows);

// xkv_attend.cu
size_t attend_part_floats(const xkv_group* grp);
cudaError_t launch_reconstruct_attend(const xkv_group* grp, int l0, int l1, const __nv_bfloat16* q,
                                      const int32_t* sel_idx, const int32_t* sel_cnt, int k_cap,
                                      __nv_bfloat16* out, float* lse, cudaStream_t s);

// xkv_tail.cu: partial attention results over an uncompressed tail, [problem of the call][split][head][d_h + 2]
struct TailParts {
  const float* part;   // nullptr: no tail
  int n_split;
};
int tail_splits(int tail_cap);
int tail_tiles_per_split(int tail_cap);
bool dense_supported(const xkv_group* grp, int cap);
cudaError_t launch_dense_merge(const xkv_group* grp, int l0, int l1, const float* part, int cap, __nv_bfloat16* out,
                               float* lse, cudaStream_t s);
size_t tail_part_floats(const xkv_group* grp, int tail_cap);
cudaError_t launch_tail_partials(const xkv_group* grp, int l0, int l1, const __nv_bfloat16* q, const __nv_bfloat16* tail_k,
                                 const __nv_bfloat16* tail_v, const int32_t* tail_len, int tail_cap, float* part,
                                 cudaStream_t s);

// xkv_quant.cu
cudaError_t launch_quantize_rtn4(const __nv_bfloat16* x, long long rows, int cols, void* codes, void* meta, cudaStream_t s);
cudaError_t launch_dequantize_rtn4(const void* codes, const void* meta, long long rows, int cols, __nv_bfloat16* x,
                                   cudaStream_t s);
cudaError_t launch_quantize_rtn3(const __nv_bfloat16* x, long long rows, int cols, void* rec, cudaStream_t s);
cudaError_t launch_dequantize_rtn3(const void* rec, long long rows, int cols, __nv_bfloat16* x, cudaStream_t s);

// xkv_clf.cu
int clf_rank_l(const xkv_clf_config* c, int* l);
int clf_workspace_bytes(const xkv_clf_config* c, uint64_t* bytes);
void clf_set_fault_injection(unsigned mask);
int clf_factorize(const xkv_clf_config* c, const void* X, const void* omega, void* workspace, uint64_t workspace_bytes,
                  void* A_out, void* B_out, float* sigma, int device, cudaStream_t s);
cudaError_t clf_gemm(const void* a, const void* b, int M, int N, int K, float* C, unsigned int* flags, int device,
                     cudaStream_t s);

// xkv_fused.cu
int fused_slots(const xkv_group* grp);
size_t fused_part_floats(const xkv_group* grp);
bool fused_supported(const xkv_group* grp);
bool fused_sm_count_ok(int sm_count);
cudaError_t launch_fused(const xkv_group* grp, int l0, int l1, const __nv_bfloat16* q, const int32_t* sel_idx,
                         const int32_t* sel_cnt, int k_cap, __nv_bfloat16* out, float* lse, cudaStream_t s,
                         TailParts tail = TailParts{nullptr, 0});

}  // namespace xkv
