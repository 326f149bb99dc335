/*
 * xkv.h -- C ABI of the xKV selective-reconstruction (SR) decode library for NVIDIA B200 (sm_100a).
 *
 * One handle describes one window of G adjacent transformer layers whose pre-RoPE key cache and
 * value cache were factorised across layers (paper Sec. 3.1, Eq. 1):
 *     [X_l0 ... X_l0+G-1] ~= A [B_l0 ... B_l0+G-1],   A = U Sigma (T x r),  B_l (r x d),  d = H_kv*d_h
 * once for keys (A_k, B_k, rank r_k) and once for values (A_v, B_v, rank r_v).
 *
 * A decode step for the layers of the window is two calls:
 *   xkv_sr_select              landmark-guided top-k chunk selection (App. B.1, Algorithm 2)
 *   xkv_sr_reconstruct_attend  X_hat[S,:] = A[S,:] B_{l,g} for keys and values (Sec. 3.2, Eq. 3),
 *                              rotary embedding of the rebuilt key rows, softmax attention over them.
 *
 * General rules
 *   - Every function returns an xkv_status; nothing throws, aborts or traps the GPU.
 *   - All data pointers are DEVICE pointers unless a parameter says "host".  The config struct,
 *     the handle and the out-parameters of create/status/bytes are host memory.
 *   - All work is enqueued on the CUDA stream passed in (a cudaStream_t cast to void*; NULL is the
 *     legacy default stream).  No call synchronises the device except create and destroy.
 *   - The handle BORROWS A_k, A_v, landmarks (the caller keeps them alive and unchanged while the
 *     handle is used) and copies B_k, B_v into a repacked buffer that it owns, together with its
 *     scratch (pooled scores, attention partials, rotary tables).  Calls on one handle must not
 *     overlap on the GPU: they share that scratch.
 *   - Conditions detected on the device (an index outside [0,T), a bounded wait that ran out) do not
 *     fault: the offending row is skipped or the tile abandoned, a bit is set in a device word, and
 *     xkv_group_status reports it after the caller has synchronised.
 *   - Index arithmetic is 64-bit; T < 2^24, d_h in {64,128}, r_k and r_v multiples of 8,
 *     H_q a multiple of H_kv with H_q/H_kv <= 16.
 */
#ifndef XKV_H_
#define XKV_H_

#include <stdint.h>

#if defined(__GNUC__)
#define XKV_API __attribute__((visibility("default")))
#else
#define XKV_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct xkv_group xkv_group; /* opaque */

typedef enum {
  XKV_OK = 0,
  XKV_ERR_INVALID_ARG = -1, /* NULL pointer, bad struct_size, sizes that break a rule above */
  XKV_ERR_UNSUPPORTED = -2, /* a legal but unimplemented combination */
  XKV_ERR_ARCH = -3,        /* current device is not compute capability 10.x */
  XKV_ERR_CUDA = -4,        /* a CUDA runtime call failed; see xkv_last_cuda_error */
  XKV_ERR_OOM = -5,         /* device allocation for the handle failed */
  XKV_ERR_INDEX_RANGE = -6, /* device flag: a selected row was outside [0,T) and was skipped */
  XKV_ERR_TIMEOUT = -7,     /* device flag: a bounded wait inside a kernel ran out */
  XKV_ERR_TOO_LARGE = -8    /* xkv_sr_select_static: the call needs more than its fixed scratch */
} xkv_status;

/* Bits of the device flag word returned by xkv_group_status. */
#define XKV_FLAG_INDEX_RANGE 1u
#define XKV_FLAG_TIMEOUT 2u
#define XKV_FLAG_CLF_BREAKDOWN 4u /* xkv_clf_factorize: a Cholesky pivot was not positive (reported by xkv_clf_status) */

/*
 * Problem statement for one window (names follow the paper; T is its L, G its W).
 * Layouts are row-major with the last index fastest; bf16 means the upper 16 bits of an IEEE fp32.
 */
typedef struct {
  uint32_t struct_size; /* sizeof(xkv_group_config); checked for ABI agreement */
  int32_t G;            /* layers in the window (paper W), >= 1 */
  int32_t batch;        /* sequences; each has its own factors (the SVD is computed per prompt) */
  int32_t T;            /* context rows (paper L), 1 <= T < 2^24 */
  int32_t H_kv, H_q;    /* KV heads and query heads; GQA map rho(h) = h / (H_q/H_kv) */
  int32_t d_h;          /* head width: 64 or 128 */
  int32_t r_k, r_v;     /* ranks of the key and value factorisation; multiples of 8 */
  int32_t chunk;        /* landmark chunk size c (0 means 8); n_c = ceil(T/c) */
  int32_t k_max;        /* largest token budget k that xkv_sr_select will be given */
  float rope_base;      /* > 0: rotate rebuilt key rows (rotate-half, theta_i = base^(-2i/d_h),
                           position = token row); <= 0: keys are used as reconstructed */
  float softmax_scale;  /* logit scale of the attention; 0 means 1/sqrt(d_h) */
  const void* A_k;      /* bf16 [batch][T][r_k]   shared token basis of the keys    (borrowed) */
  const void* A_v;      /* bf16 [batch][T][r_v]   shared token basis of the values  (borrowed) */
  const void* B_k;      /* bf16 [batch][G][r_k][H_kv*d_h]  per-layer reconstruction matrices; head g
                           owns columns g*d_h .. g*d_h+d_h-1 (Eq. 2).  Copied at create. */
  const void* B_v;      /* bf16 [batch][G][r_v][H_kv*d_h]  same for values.  Copied at create. */
  const void* landmarks; /* bf16 [batch][G][H_kv][n_c][d_h] chunk means of the post-RoPE keys
                            (Algorithm 1, lines 1-3); borrowed.  May be NULL if xkv_sr_select is
                            never called on this handle. */
} xkv_group_config;

/*
 * Validate the configuration, allocate the handle's device memory on the current device, repack
 * B_k/B_v and build the rotary tables (this work is enqueued on `stream` and waited for).
 * On success *out receives the handle.  Errors: INVALID_ARG, ARCH, OOM, CUDA.
 */
XKV_API int xkv_group_create(const xkv_group_config* cfg, void* stream, xkv_group** out);

/*
 * Algorithm 2 (App. B.1) for layers layer_begin <= l < layer_end of the window, every sequence and
 * every KV head g:
 *   P[h,j] = (sum_{i=0}^{d_h-1} q[h,i]*L[g,j,i]) * (1/sqrt(d_h))   fp32, i in ascending order
 *   S[j]   = max over the H_q/H_kv query heads h with rho(h) = g
 *   take the k_ch = min(ceil(k/c), n_c) chunks first in the order (S descending, j ascending;
 *   -0 equals +0), sort them ascending, expand chunk j to rows c*j .. min(c*j+c, T)-1.
 * q        bf16 [G][batch][H_q][d_h], post-RoPE decode queries (rows of layers outside the range are
 *          not read).
 * k        token budget, 1 <= k <= k_max.  k_cap = ceil(k/c)*c is the row stride of sel_idx
 *          ((ceil(k/c) + n_outliers)*c after xkv_group_set_outliers, see there).
 * sel_idx  out, int32 [G][batch][H_kv][k_cap]; entries at and beyond sel_cnt are set to -1.
 * sel_cnt  out, int32 [G][batch][H_kv]; number of rows (k_ch*c, less if the ragged last chunk is in).
 * Scores must be finite; the result for NaN inputs is unspecified (but in range).
 * Errors: INVALID_ARG (NULL, bad range, k out of range, handle without landmarks), CUDA.
 */
XKV_API int xkv_sr_select(xkv_group* grp, int layer_begin, int layer_end, const void* q, int32_t k,
                  int32_t* sel_idx, int32_t* sel_cnt, void* stream);

/*
 * Static outlier chunks (Algorithm 1 line 5 finds them at prefill; Algorithm 2 line 5 uses them): from now on
 * xkv_sr_select unites the top-k chunks of every (layer, sequence, KV head) with that head's outlier chunks.
 * outliers    int32 [G][batch][H_kv][n_outliers] chunk ids, device memory, BORROWED until the handle is destroyed
 *             or the list is replaced.  Ids outside [0, n_c) are ignored; a repeated id counts once.
 * n_outliers  0 <= n_outliers <= XKV_MAX_OUTLIERS; 0 (with any pointer) switches the union off.
 * With outliers the row stride of sel_idx is k_cap = (ceil(k/c) + n_outliers) * c, sel_cnt varies between
 * ceil(k/c)*c and k_cap (less by the ragged last chunk), rows stay ascending without repeats, and
 * xkv_sr_reconstruct_attend accepts k_cap up to (ceil(k_max/c) + n_outliers) * c.
 * The call waits for `stream` and may replace the handle's scratch: no work of this handle may be in flight on
 * another stream.  Errors: INVALID_ARG (also: handle without landmarks), OOM, CUDA.
 */
#define XKV_MAX_OUTLIERS 4096
XKV_API int xkv_group_set_outliers(xkv_group* grp, const int32_t* outliers, int32_t n_outliers, void* stream);

/*
 * Eq. 3 plus attention for layers layer_begin <= l < layer_end, every sequence, every KV head g:
 *   K_hat[S,:] = rope(A_k[S,:] B_k_{l,g}),  V_hat[S,:] = A_v[S,:] B_v_{l,g},
 *   out_h = softmax(scale * q_h K_hat^T) V_hat  for the query heads h with rho(h) = g.
 * sel_idx  int32 [G][batch][H_kv][k_cap], the first sel_cnt entries of each row list the token rows
 *          S.  They need not be sorted or chunk aligned; a repeated row counts as often as it
 *          appears.  A row outside [0,T) is skipped and XKV_FLAG_INDEX_RANGE is raised.
 * sel_cnt  int32 [G][batch][H_kv], 0 <= sel_cnt <= k_cap.  With sel_cnt = 0 the head's output is 0
 *          and its lse is -inf.
 * k_cap    row stride of sel_idx, 1 <= k_cap <= ceil(k_max/c)*c (the handle's scratch is sized by k_max).
 * out      bf16 [G][batch][H_q][d_h].
 * lse      optional (may be NULL) fp32 [G][batch][H_q]: natural-log sum of exp of the scaled logits,
 *          for merging with attention over rows kept outside the factorised cache.
 * Accumulation is fp32 from bf16 operands.  Errors: INVALID_ARG, CUDA.
 */
XKV_API int xkv_sr_reconstruct_attend(xkv_group* grp, int layer_begin, int layer_end, const void* q,
                              const int32_t* sel_idx, const int32_t* sel_cnt, int32_t k_cap,
                              void* out, float* lse, void* stream);

/*
 * xkv_sr_reconstruct_attend over the union of the selected reconstructed rows and an uncompressed tail:
 * the tokens generated during decoding are kept as plain K/V rows (Sec. 4 "Implementation details",
 * Sec. 7 "Long Generation Scenario") and every decode step attends to all of them.  One softmax over both
 * sets, evaluated as split partial results merged by their log-sum-exp.
 * tail_k, tail_v  bf16 [G][batch][H_kv][tail_cap][d_h], device, borrowed for the call; keys as the model
 *                 stores them (already rotated).
 * tail_len        int32 [batch], device, or NULL for tail_cap rows in every sequence; 0 <= tail_len <= tail_cap
 *                 (a larger value is clamped and XKV_FLAG_INDEX_RANGE is raised).
 * tail_cap        1 <= tail_cap <= XKV_TAIL_MAX_ROWS.
 * workspace       device scratch of at least xkv_tail_workspace_bytes(grp, tail_cap) bytes, 16-byte aligned,
 *                 owned by the caller, used only during the call's kernels.
 * The other arguments and the outputs are those of xkv_sr_reconstruct_attend.  With sel_cnt = 0 and
 * tail_len = 0 the head's output is 0 and its lse is -inf.
 * Errors: INVALID_ARG, UNSUPPORTED (shapes the tensor-core path does not cover), CUDA.
 */
#define XKV_TAIL_MAX_ROWS 32768
XKV_API int xkv_tail_workspace_bytes(const xkv_group* grp, int32_t tail_cap, uint64_t* bytes);
XKV_API int xkv_sr_reconstruct_attend_tail(xkv_group* grp, int layer_begin, int layer_end, const void* q,
                                           const int32_t* sel_idx, const int32_t* sel_cnt, int32_t k_cap,
                                           const void* tail_k, const void* tail_v, const int32_t* tail_len,
                                           int32_t tail_cap, void* workspace, uint64_t workspace_bytes,
                                           void* out, float* lse, void* stream);

/*
 * Cross-layer factorisation on the GPU (Sec. 3.1, Eq. 1): for one sequence and one cache (keys or values), the
 * rank-r factors A = U Sigma (T x r) and B_l (r x d per layer) of X = [X_l0 ... X_l0+G-1] (T x G d), by the
 * randomised SVD the paper describes for prefill (App. "Custom SVD Kernel": power iterations as 16-bit tensor-core
 * matrix products, shifted Cholesky QR instead of Householder QR).  Steps: Z <- omega; (power_iters + 1) times
 * Y = X Z, U = X^T Y, Z = orth(U) (two passes of Cholesky QR with a relative diagonal shift, five for the last
 * iterate; Gram matrix, factor and solve in fp64); then the
 * Rayleigh-Ritz step on span(Z): M = Z^T X^T X Z = P Lambda P^T (Jacobi), V = Z P_r, B = V^T rounded to bf16,
 * A = X bf16(V), sigma = sqrt(Lambda).  The result approximates the optimum of Eq. 1 (it is not unique up to signs and
 * rotations inside equal singular values: compare residuals, never factors).
 * cfg       host struct: T rows, G layers, d columns per layer (G*d a multiple of 64), rank r (multiple of 8),
 *           oversample p (0 means 32; l = r + p rounded up to a multiple of 64, at most G*d), power_iters q (0..8).
 * X         bf16 [T][G*d] (the layers' caches side by side, layer l in columns l*d .. l*d+d-1), device, 16-byte aligned.
 * omega     bf16 [G*d][l] random test matrix drawn by the caller (standard normal), device; l from xkv_clf_rank_l.
 * workspace device scratch of at least xkv_clf_workspace_bytes(cfg) bytes, 256-byte aligned, caller-owned.
 * A         out bf16 [T][r];  B out bf16 [G][r][d] (the layout of xkv_group_config.B_k for one sequence);
 * sigma     out fp32 [r], optional.
 * The call allocates nothing and enqueues everything on `stream`.  xkv_clf_status (after the caller has synchronised,
 * or blocking on `stream`) reads the flag word of the workspace: XKV_FLAG_TIMEOUT, XKV_FLAG_CLF_BREAKDOWN.
 * The first 256 bytes of the workspace are that flag block (32-bit words); besides word 0 (the flags) a caller may
 * read word 11, the number of Jacobi sweeps the last call ran (a diagnostic: at most 12); the rest is internal.
 * The Jacobi sweeps are one cooperative launch (all its CTAs resident at once), so the device must not be fully
 * occupied by kernels that wait for this one.
 * Errors: INVALID_ARG, UNSUPPORTED (l too large for the eigen-solver: l <= 2048), ARCH, CUDA.
 */
typedef struct {
  uint32_t struct_size; /* sizeof(xkv_clf_config) */
  int32_t T, G, d, r;
  int32_t oversample;   /* p; 0 means 32 */
  int32_t power_iters;  /* q */
} xkv_clf_config;
XKV_API int xkv_clf_rank_l(const xkv_clf_config* cfg, int32_t* l);
XKV_API int xkv_clf_workspace_bytes(const xkv_clf_config* cfg, uint64_t* bytes);
XKV_API int xkv_clf_factorize(const xkv_clf_config* cfg, const void* X, const void* omega, void* workspace,
                              uint64_t workspace_bytes, void* A, void* B, float* sigma, void* stream);
XKV_API int xkv_clf_status(const void* workspace, uint32_t* flags, void* stream);
/* Diagnostic: the tensor-core product of the factorisation alone, C (M x N, fp32) = A B^T for A bf16 [K][M] and
 * B bf16 [N][K] (M, K multiples of 8); flags: one device word (XKV_FLAG_TIMEOUT). */
XKV_API int xkv_debug_gemm(const void* a, const void* b, int32_t M, int32_t N, int32_t K, float* C, uint32_t* flags,
                           void* stream);

/*
 * Round-to-nearest quantisation of factors (App. "Integrate with Quantization": RTN on the compressed cache; the
 * printed 25.7x at 4 bits is the 8.03x of the 16-bit factors times 16/5, i.e. one bit of overhead per scalar).
 * Groups of 32 consecutive scalars of a row share a bf16 scale and a bf16 offset:
 *   zero = bf16(min), scale = bf16((max - min)/15), code = clip(rint((x - zero)/scale), 0, 15)   (fp32, ties to even)
 *   x_hat = bf16(code*scale + zero), the exact value rounded once.
 * x      bf16 [rows][cols], device, 16-byte aligned; cols a multiple of 32.
 * codes  [rows][cols/2] bytes, 16-byte aligned.  Inside every 32-bit word (scalars e0..e7) nibble k of the low half
 *        is e_2k and nibble k of the high half is e_2k+1.
 * meta   uint32 [rows][cols/32]: scale in the low 16 bits, offset in the high 16 bits.
 * bits   4, or 3 (the paper's other setting: 8.03x -> 32.12x).  With 3 bits the step is (max - min)/7, codes clip at
 *        7, and a group is ONE 16-byte record in `codes` ([rows][cols/32] records, cols/2 bytes per row as for 4 bits;
 *        `meta` is not used and may be NULL): {meta word, w0, w1, w2}; word w_j holds scalars 10j..10j+9 as five
 *        pairs, (w_j >> 3k) & 0x00070007 = (e_10j+2k, e_10j+2k+1); bits 15 of w0, w1, w2 hold scalar 30 and bits 31
 *        scalar 31, least significant bit in w0.  Other widths: UNSUPPORTED.
 * xkv_dequantize_rtn writes x_hat (for the small per-layer matrices B, which a handle takes as bf16).
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA.
 */
XKV_API int xkv_quantize_rtn(const void* x, int64_t rows, int32_t cols, int32_t bits, void* codes, void* meta, void* stream);
XKV_API int xkv_dequantize_rtn(const void* codes, const void* meta, int64_t rows, int32_t cols, int32_t bits, void* x,
                               void* stream);

/*
 * From now on xkv_sr_reconstruct_attend (and the _tail variant) gathers the token bases from 4-bit or 3-bit codes and
 * dequantises them on the way into shared memory (Eq. 3 on x_hat); a gathered row costs r/2 + r/8 bytes (4 bits) or
 * r/2 bytes (3 bits) instead of 2r.  The handle's A_k / A_v (which xkv_group_create then accepts as NULL) are no longer read.
 * codes_k, meta_k  quantised A_k: [batch][T][r_k/2] bytes and uint32 [batch][T][r_k/32] (layout of xkv_quantize_rtn
 *                  with rows = batch*T), device, BORROWED until the handle is destroyed; likewise codes_v, meta_v.
 * bits             4 or 3 (with 3 the meta pointers are not used and may be NULL); r_k and r_v must be multiples of 32.
 *                  All-NULL pointers switch back to the bf16 bases.
 * Errors: INVALID_ARG, UNSUPPORTED (ranks, or a shape the tensor-core path does not cover).
 */
XKV_API int xkv_group_set_quantized_bases(xkv_group* grp, const void* codes_k, const void* meta_k, const void* codes_v,
                                          const void* meta_v, int32_t bits);

/*
 * Plain decode attention over an UNCOMPRESSED bf16 cache: out_h = softmax(scale * q_h K^T) V for the query heads of
 * every (layer, sequence, KV head).  This is the baseline that selective reconstruction is measured against (Sec. 5,
 * "Efficiency Studies": full attention reads the whole cache, SR removes the term that grows with the context); it
 * runs the kernels of the uncompressed tail with several tiles per CTA and a merge of its own.
 * K, V       bf16 [G][batch][H_kv][cap][d_h], device, borrowed for the call; keys as the model stores them (rotated).
 * len        int32 [batch], device, or NULL for cap rows in every sequence (clamped to cap, flag raised, as for the tail).
 * cap        1 <= cap <= XKV_DENSE_MAX_ROWS; beyond XKV_TAIL_MAX_ROWS only d_h = 128 is served (else UNSUPPORTED).
 * workspace  device scratch of at least xkv_dense_workspace_bytes(grp, cap) bytes, 16-byte aligned, caller-owned.
 * The handle supplies the shapes (G, batch, heads, d_h) and the softmax scale; its factors are not read.
 * With len = 0 a head's output is 0 and its lse is -inf.  Errors: INVALID_ARG, UNSUPPORTED, CUDA.
 */
#define XKV_DENSE_MAX_ROWS (1 << 22)
XKV_API int xkv_dense_workspace_bytes(const xkv_group* grp, int32_t cap, uint64_t* bytes);
XKV_API int xkv_dense_attend(xkv_group* grp, int layer_begin, int layer_end, const void* q, const void* K, const void* V,
                             const int32_t* len, int32_t cap, void* workspace, uint64_t workspace_bytes, void* out,
                             float* lse, void* stream);

/*
 * Algorithm 1 (App. B.1), the prefill side of the selector, for every sequence, layer and KV head g:
 *   landmark[j]  = mean over the rows x of chunk j of rope(K[x]),  chunk j = rows c*j .. min(c*j+c, T)-1   (lines 1-3)
 *   min_cos[j]   = min over those rows of cos(rope(K[x]), landmark[j])  (fp32, the unrounded mean; a zero vector
 *                  has cosine 0)                                                                        (line 4)
 *   outliers     = the n_outliers chunks with the smallest min_cos, ties to the lowest chunk id, ids ascending,
 *                  padded with -1 if n_outliers > n_c                                                    (line 5)
 * No handle and no allocation: everything the call needs is passed in.
 * keys        bf16 [batch][G][T][H_kv*d_h] (head g owns columns g*d_h .. g*d_h+d_h-1), device.  With
 *             rope_base > 0 the rows are rotated here (rotate-half, position = row, angles formed in fp64);
 *             with rope_base <= 0 they are taken as already rotated.
 * landmarks   out bf16 [batch][G][H_kv][n_c][d_h]: the layout xkv_group_config.landmarks expects.
 * min_cos     out fp32 [G][batch][H_kv][n_c]; may be NULL if n_outliers == 0.
 * outliers    out int32 [G][batch][H_kv][n_outliers]: the layout xkv_group_set_outliers expects; NULL if none.
 * Limits: d_h in {64, 128}; H_kv * d_h / 16 (threads per key row) must divide 256, i.e. H_kv * d_h is a power of
 * two between 64 and 4096 (else UNSUPPORTED); keys and landmarks 16-byte aligned; 0 <= n_outliers <=
 * XKV_MAX_OUTLIERS; 1 <= T < 2^24.
 * Errors: INVALID_ARG, UNSUPPORTED, ARCH, CUDA.
 */
typedef struct {
  uint32_t struct_size; /* sizeof(xkv_landmark_config) */
  int32_t G, batch, T, H_kv, d_h;
  int32_t chunk;        /* c (0 means 8) */
  float rope_base;
} xkv_landmark_config;
XKV_API int xkv_build_landmarks(const xkv_landmark_config* cfg, const void* keys, void* landmarks, float* min_cos,
                                int32_t n_outliers, int32_t* outliers, void* stream);

/* Free the handle and the device memory it owns (synchronises the device first). NULL is allowed. */
XKV_API int xkv_group_destroy(xkv_group* grp);

/*
 * Read the device flag word (host out-parameter, may be NULL) with a blocking copy on `stream`
 * and clear it.  Returns XKV_OK, or the status of the most severe flag (TIMEOUT over INDEX_RANGE).
 */
XKV_API int xkv_group_status(xkv_group* grp, uint32_t* device_flags, void* stream);

/*
 * Memory accounting of one window (App. C, "Compressed-cache memory" and "Landmark memory"),
 * in bytes of bf16 storage: factor_bytes = batch*2*(T*r_k + G*r_k*d + T*r_v + G*r_v*d),
 * landmark_bytes = batch*2*G*ceil(T/c)*d.  Host-only; needs no device.  Out-pointers may be NULL.
 */
XKV_API int xkv_group_bytes(const xkv_group_config* cfg, uint64_t* factor_bytes, uint64_t* landmark_bytes);

/*
 * Scratch bytes the handle owns on the device (pooled scores, attention partials, rotary tables,
 * repacked B), host out-parameter.
 */
XKV_API int xkv_group_workspace_bytes(const xkv_group* grp, uint64_t* bytes);

/* Static, human-readable name of a status code. Never NULL. */
XKV_API const char* xkv_strerror(int status);

/* The last CUDA runtime error code seen by this library on the calling thread (0 if none). */
XKV_API int xkv_last_cuda_error(void);

/* Number of kernels the library has launched since load (all handles); for launch accounting. */
XKV_API uint64_t xkv_kernel_launch_count(void);

/*
 * The same count split by kernel family: counts[f] = launches of family f since load (host array of
 * XKV_KERNEL_FAMILIES words).  Tests use it to tell which of two implementations of a step ran.
 */
#define XKV_KERNEL_SCAN 0      /* landmark scores + pooling (Algorithm 2 lines 2-3) */
#define XKV_KERNEL_TOPK 1      /* top-k chunks (Algorithm 2 lines 1, 4, 5) */
#define XKV_KERNEL_FUSED 2     /* gather + reconstruct + attention on the tensor core (Eq. 3) */
#define XKV_KERNEL_MERGE 3     /* log-sum-exp merge of attention partials, value projection */
#define XKV_KERNEL_TILE 4      /* the plain (CUDA-core) reconstruct + attention kernels */
#define XKV_KERNEL_TAIL_TC 5   /* uncompressed-tail / dense attention partials on the tensor core */
#define XKV_KERNEL_TAIL_CUDA 6 /* the same partials on CUDA cores */
#define XKV_KERNEL_LANDMARKS 7 /* Algorithm 1 */
#define XKV_KERNEL_PREP 8      /* handle set-up: repacking, rotary tables */
#define XKV_KERNEL_DENSE 9     /* merge of dense-attention partials (xkv_dense_attend) */
#define XKV_KERNEL_CLF 10      /* cross-layer factorisation (xkv_clf_factorize) */
#define XKV_KERNEL_MERGE_MULTI 11 /* the same merge with one CTA per group of query heads (windows of many problems) */
#define XKV_KERNEL_FAMILIES 12
XKV_API int xkv_debug_launch_counts(uint64_t* counts);

/*
 * Host-side fault injection for tests of the give-up path (nothing here faults, traps or hangs the GPU: a wait
 * that can never be satisfied runs into its limit, the kernel raises XKV_FLAG_TIMEOUT and returns).
 *   XKV_INJECT_SCAN_NO_LOAD   the landmark scan does not issue its loads and waits only briefly for them; the
 *                             pooled scores keep whatever they held, so the selection that follows is arbitrary
 *                             (but in range).
 *   XKV_INJECT_FUSED_NO_B     the reconstruct+attend kernel does not load the reconstruction matrices and
 *                             waits only briefly; its output for that call is unspecified.
 * mask = 0 restores normal operation; later calls on the handle are then correct again.
 */
#define XKV_INJECT_SCAN_NO_LOAD 1u
#define XKV_INJECT_FUSED_NO_B 2u
XKV_API int xkv_debug_set_fault_injection(xkv_group* grp, uint32_t mask);
/*
 * The same for xkv_clf_factorize, which has no handle: the mask applies to every later call of the process until it
 * is set back to 0.
 *   XKV_INJECT_CLF_BARRIER    one CTA of the Jacobi kernel does not arrive at the first grid barrier, and the wait of
 *                             that kernel's barriers is shortened to about a millisecond; the other CTAs give up,
 *                             the workspace's flag word gets XKV_FLAG_TIMEOUT (xkv_clf_status returns
 *                             XKV_ERR_TIMEOUT) and the factors of that call are unspecified.
 */
#define XKV_INJECT_CLF_BARRIER 4u
XKV_API int xkv_debug_set_clf_fault_injection(uint32_t mask);

/*
 * Chunk selection for callers that must not allocate device memory.  (The paper has no counterpart: this is a
 * packaging variant of xkv_sr_select, same arithmetic, same outputs.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a serving loop whose memory pool owns
 * every byte of the device, under an allocator that forbids side allocations, or in a process that may only
 * use memory handed to it.  xkv_group_create allocates (pooled scores, repacked matrices, tables); this entry
 * point takes no handle and allocates nothing, neither with cudaMalloc/cudaFree nor through any library.
 *
 * Where the scratch lives: the pooled landmark scores go to a fixed array inside the library image
 * (XKV_STATIC_SELECT_MAX_SCORES floats, 4 MiB, plus 256 bytes of flag words).  Every GPU that loads the library
 * carries that array until the process exits.  A call needs G*batch*H_kv*ceil(T/c) scores; if that is more than
 * the array holds, the call does nothing and returns XKV_ERR_TOO_LARGE.
 *
 * First call on a device: the library looks up the array's device address (once per device, for the device
 * that is current at the call) before it launches anything.  Make that first call outside any stream capture.
 *
 * Sharing: all calls on a device use the same array, which keeps the previous call's scores; the flag words are
 * cleared at the start of each call.  Two calls whose kernels overlap on the GPU (different streams, or
 * different host threads) race on it: serialise them.  Device-side give-ups (a bounded wait that ran out) are
 * not reported by this entry point.
 *
 * cfg       host struct; landmarks as in xkv_group_config (bf16 [batch][G][H_kv][n_c][d_h], device, 16-byte aligned).
 * other arguments, outputs and tie rules: exactly those of xkv_sr_select (k_cap = ceil(k/c)*c is the row stride).
 * Errors: INVALID_ARG, TOO_LARGE, ARCH, CUDA.
 */
#define XKV_STATIC_SELECT_MAX_SCORES (1u << 20)
typedef struct {
  uint32_t struct_size; /* sizeof(xkv_select_static_config) */
  int32_t G, batch, T, H_kv, H_q, d_h;
  int32_t chunk;        /* 0 means 8 */
  const void* landmarks;
} xkv_select_static_config;
XKV_API int xkv_sr_select_static(const xkv_select_static_config* cfg, int layer_begin, int layer_end, const void* q,
                                 int32_t k, int32_t* sel_idx, int32_t* sel_cnt, void* stream);

/*
 * Diagnostic.  If the environment variable XKV_FUSED_PROF=1 was set when the handle was created, the
 * reconstruct+attend kernel adds, per CTA, the cycles each warp role spent waiting on each of its
 * hand-offs (64 counters per CTA; the layout is documented beside the kernel).  Synchronises the device,
 * copies up to max_words counters to `out` (host) and clears them.  Returns the number of words copied,
 * XKV_ERR_UNSUPPORTED if profiling was not requested, or another negative status.
 */
XKV_API int xkv_debug_read_profile(xkv_group* grp, uint64_t* out, int max_words);

#ifdef __cplusplus
}
#endif
#endif /* XKV_H_ */
