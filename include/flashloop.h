/*
 * flashloop.h -- C ABI of the B200 (sm_100a) FlashLoop loop-r prefill library.
 *
 * The library implements one step of "FlashLoop: Fast and Memory-Efficient Looped Transformers via
 * Lazy Updates": the prefill of loop r > 1 of one layer, i.e.
 *   (1) cross-loop token scoring and top-k token selection        (Section 4.1, Appendix D.1, Eq. 5)
 *   (2) column-sparse attention replacement                       (Section 4.2, Appendix D.2, Eq. 6-7)
 *   (3) quantization of the cross-loop K/V residuals              (Section 4.3, Appendix D.3, Eq. 8)
 *   (4) dequantize-and-add reconstruction of K/V inside attention (Section 4.3, last paragraph; App. G)
 * plus the dense source loop that produces the statistics loop 2 starts from (Eq. 2, Eq. 6 with m_C = 1).
 *
 * Conventions
 *  - Plain C. Every pointer is a DEVICE pointer unless its comment says "host". All device buffers are
 *    owned by the caller, must be 16-byte aligned, and must stay valid until the stream has run the call.
 *  - Every call validates its arguments on the host, enqueues its kernels on `stream` (a cudaStream_t
 *    passed as void*) and returns without synchronising. Return value: FL_OK or a negative fl_status.
 *    Nothing is launched when an argument is rejected.
 *  - No call allocates device memory: every buffer, scratch included, is the caller's.
 *  - Results are deterministic: the same inputs give bit-identical outputs.
 *  - Row-major tensors; [n, H, dh] means n rows of H heads of dh elements, dh fastest.
 *    "storage type" is fl_shape.dtype: FL_BF16 (2 bytes) or FL_F32 (4 bytes).
 *  - Notation: L tokens, H heads, dh head dimension, d = H*dh, A^(r) active-token set of loop r,
 *    nb = ceil(L / q_block) query blocks of q_block consecutive token positions,
 *    S[h,b] the key columns selected for head h and block b, T_i = { j in S[h, block(i)] : j <= i }.
 *    G^(r) is the hidden state entering loop r (the paper's H^(r-1)).
 */
#ifndef FLASHLOOP_H_
#define FLASHLOOP_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define FL_API __attribute__((visibility("default")))
#else
#define FL_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  FL_OK = 0,
  FL_ERR_INVALID_ARG = -1, /* null / misaligned pointer, size out of range, inconsistent store */
  FL_ERR_UNSUPPORTED = -2, /* a valid request this build has no kernel for (e.g. head_dim 96) */
  FL_ERR_WORKSPACE = -3,   /* the workspace handed to fl_set_workspace is too small to be of any use */
  FL_ERR_CUDA = -4,        /* a CUDA runtime call failed (launch error, wrong device, ...) */
  FL_ERR_TIMEOUT = -5      /* reported through the device status word: a bounded wait ran out */
} fl_status;

enum { FL_BF16 = 0, FL_F32 = 1 };
#define FL_MAX_LOOPS 32 /* residual streams per store: loops 2 .. FL_MAX_LOOPS+1 */

/* Opaque context: device ordinal, SM count, cached TMA tensor maps (host memory). Not thread-safe per context. */
typedef struct fl_ctx fl_ctx;
FL_API int fl_create(fl_ctx** out /* host */, int device);
FL_API int fl_destroy(fl_ctx* ctx);
FL_API const char* fl_status_string(int status); /* host string, static storage */
FL_API int fl_version(void);

/* Fixed per model / configuration. */
typedef struct {
  int32_t L;        /* tokens in the prompt, >= 1 */
  int32_t n_heads;  /* H >= 1 */
  int32_t head_dim; /* dh in {64, 128} */
  int32_t dtype;    /* FL_BF16 or FL_F32: storage type of hidden states, Q, K, V, O and the K/V base */
  int32_t q_block;  /* query-block width in token positions, >= 1 (1 = the per-position rule of Eq. 6) */
  int32_t bits;     /* residual code width: 2, 4, 8, or 16 = codec off (rows stored in storage type) */
  int32_t group;    /* codec group: consecutive head_dim elements sharing scale and offset;
                       one of 8, 16, 32, 64, 128 and a divisor of head_dim */
  float eps;        /* Eq. 5 epsilon (added to the norm, not to its square) */
  float sm_scale;   /* logit scale, normally 1/sqrt(head_dim) */
} fl_shape;

/* One loop's residual payload for K or for V (Eq. 8: only active rows carry payload).
 * Row t belongs to token position active_idx[t] of that loop; slot_of_pos inverts the map.
 *   bits in {2,4,8}: codes [n_rows, H, dh*bits/8] bytes, little-endian inside a byte (element
 *                    (8/bits)*t+u occupies bits [u*bits, (u+1)*bits) of byte t);
 *                    scale, zero [n_rows, H, dh/group] IEEE fp16 bit patterns;
 *                    value = code * scale + zero (one binary32 rounding).
 *   bits == 16     : codes [n_rows, H, dh] in storage type holds the loop's rows themselves;
 *                    scale and zero are ignored (may be NULL).
 * rows_prev / rows_cur (optional, for the K and the V stream of a loop alike; rows_cur may be set without
 * rows_prev, not the reverse; bf16 storage only, ignored otherwise): [n_rows, H, dh] storage type, 16-byte aligned. A transient workspace, not
 * part of the cache: fl_quant_kv_residual of loop r, which has both values in registers, leaves there the
 * reconstructed rows of the stream's tokens before and after the loop's residual, Xhat^(r-1) and Xhat^(r)
 * (Eq. 4 / Eq. 8 chain in binary32, rounded once to the storage type), and fl_loop_attention of the same loop
 * gathers the selected columns that are active in loop r from them instead of dequantizing those columns again.
 * A call that reuses the carried old term (fl_attn_carry.reuse) reads rows_cur only, so a loop that is known to
 * reuse may lend rows_cur alone and save the quantizer the other write; a recomputing call that finds rows_cur
 * alone rebuilds the columns itself, as if neither were there.
 * The buffers may be reused for the next loop or layer once that attention call has been issued on the stream.
 * This is a choice of this implementation; the paper reconstructs inside its attention kernel. */
typedef struct {
  void* codes;
  uint16_t* scale;
  uint16_t* zero;
  const int32_t* slot_of_pos; /* [L]: row of this stream holding the position, or -1 */
  void* rows_prev;
  void* rows_cur;
  int32_t n_rows;
  int32_t reserved_;
} fl_kv_stream;

/* Per-layer K/V store: loop-1 base (storage type, all L rows) plus one residual stream per later loop.
 * k_res[r-2] / v_res[r-2] hold loop r and describe the same rows (equal n_rows and slot_of_pos contents).
 * Reconstruction (Eq. 4 / Eq. 8), in binary32 and in loop order:
 *   Xhat^(r)_i = ((base_i + D_2) + D_3) + ... over the loops <= r in which position i was active. */
typedef struct {
  void* k_base;
  void* v_base; /* [L, H, dh] */
  fl_kv_stream k_res[FL_MAX_LOOPS];
  fl_kv_stream v_res[FL_MAX_LOOPS];
  int32_t n_streams; /* streams filled so far: loops 2 .. n_streams+1 */
  int32_t reserved_;
} fl_kv_store; /* host struct holding device pointers */

/* Stage 1 -- Eq. 5. Scores the candidate rows and keeps the top k.
 *   s_i = ||G^(r)_i - G^(r-1)_i||_2 / (||G^(r)_i||_2 + eps), accumulated in binary32 over d = H*dh;
 *   A^(r) = the min(k, n_cand) candidates with the largest s, ties to the lowest position.
 * h_prev, h_cur : [L, d] storage type.  cand: ascending positions [n_cand], or NULL for all L rows
 * (then n_cand must equal L).  Outputs: scores f32 [n_cand] (aligned with cand), active_idx int32
 * [min(k, n_cand)] ascending, slot_of_pos int32 [L] (rank in active_idx, or -1).
 * Inputs must be finite. Errors: null pointers, k < 1, n_cand < 1 or > L, loop_r < 2; FL_ERR_UNSUPPORTED unless
 * d = H*dh is a multiple of 256 (a warp reads a row in 256-element steps). `status` is accepted for symmetry and never
 * written: this call has no bounded device wait and checks nothing on the device. */
FL_API int fl_select_tokens(fl_ctx* ctx, const fl_shape* shape, int loop_r, const void* h_prev, const void* h_cur,
                     const int32_t* cand, int32_t n_cand, int32_t k, float* scores, int32_t* active_idx,
                     int32_t* slot_of_pos, int32_t* status, void* stream);

/* Active-row execution (Appendix G, the item on executing only the active tokens):
 * gather: dst[t, :] = src[idx[t], :];  scatter: dst[idx[t], :] = src[t, :], other rows untouched.
 * row_bytes must be a positive multiple of 16; idx ascending without repeats; n >= 0. */
FL_API int fl_gather_rows(fl_ctx* ctx, const void* src, const int32_t* idx, int32_t n, int64_t row_bytes, void* dst,
                   void* stream);
FL_API int fl_scatter_update(fl_ctx* ctx, const void* src, const int32_t* idx, int32_t n, int64_t row_bytes,
                      void* dst, void* stream);

/* Projection of the active rows (Section 4.4 and Appendix G: the selected token rows are gathered so that the
 * projections remain regular GEMMs, and results return to their positions). One tensor-core GEMM whose A operand is
 * gathered by row index and whose epilogue writes or adds into indexed rows:
 *   for t in [0, n):  y[dst(t), :] = (accumulate ? y[dst(t), :] : 0) + x[src(t), :] . w^T
 * with src(t) = src_idx[t] (or t when src_idx is NULL) and dst(t) = dst_idx[t] (or t when dst_idx is NULL).
 * x: bf16 [x_rows, d_in]; w: bf16 [d_out, d_in] (a linear layer's weight, e.g. the stacked Q, K, V weights);
 * y: bf16 [y_rows, d_out]; all row-major, device memory, 16-byte aligned, owned by the caller; y must not overlap
 * x or w. Products accumulate in binary32 over d_in; each output element is rounded to bf16 once (after the add
 * when accumulate = 1). Index lists: device int32 [n], values inside their matrix, dst_idx without repeats; rows of y
 * that are not listed are left untouched. With src_idx = the active list this replaces fl_gather_rows + a GEMM on the
 * compact rows; with dst_idx = the active list and accumulate = 1 it is the output projection with the residual add
 * scattered back.
 * Errors: FL_ERR_INVALID_ARG for null or misaligned pointers, n < 0, n beyond a matrix that has no index list,
 * accumulate not 0 or 1, y aliasing an input; FL_ERR_UNSUPPORTED unless d_in is a multiple of 64 and d_out a multiple
 * of 8, or when the device offers no tensor maps (nothing is launched). n = 0 returns FL_OK without a launch.
 * `status` (device int32, may be NULL) receives FL_ERR_TIMEOUT if a bounded wait inside the kernel ran out; y is then
 * undefined. */
FL_API int fl_project_rows(fl_ctx* ctx, const void* x, int64_t x_rows, const int32_t* src_idx, int32_t n, int32_t d_in,
                    const void* w, int32_t d_out, void* y, int64_t y_rows, const int32_t* dst_idx,
                    int32_t accumulate, int32_t* status, void* stream);

/* Stacked Q/K/V projection of the active rows with the residual codec as the epilogue of its K and V columns
 * (Section 4.4: cache update and quantization fused into the producing kernel; Appendix G: Q, K and V in one GEMM).
 * One launch replaces fl_gather_rows + the projection GEMM + fl_quant_kv_residual:
 *   [q | k | v] = x[active_idx[t], :] . w_qkv^T          (w_qkv: bf16 [3d, d], rows 0..d-1 -> Q, d..2d-1 -> K, 2d..3d-1 -> V)
 *   q_out[t, :] = bf16(q);  k, v rounded to bf16 and then coded exactly as fl_quant_kv_residual codes them, against
 *   the reconstruction of loop_r - 1 (base + earlier streams of `store`), into stream loop_r - 2 of `store`
 *   (codes, scale, zero, and rows_prev / rows_cur when the stream lends them).
 * x: bf16 [x_rows, d] (the hidden states); q_out: bf16 [n_active, d]; kv_out: optional bf16 [n_active, 2d] that
 * receives the new K | V rows as the codec saw them (NULL: they are never written anywhere). The codes are those of the
 * GEMM's own bf16 outputs: a different GEMM (other accumulation order) may round a value differently and so code it
 * differently; given kv_out they are bit-exact against the reference codec.
 * Errors: as fl_quant_kv_residual and fl_project_rows; FL_ERR_UNSUPPORTED unless the storage type is bf16, bits < 16,
 * group >= 32 and d is a multiple of 256. `status` receives FL_ERR_TIMEOUT if a bounded wait ran out. */
FL_API int fl_project_qkv_quant(fl_ctx* ctx, const fl_shape* shape, int loop_r, const void* x, int64_t x_rows,
                         const int32_t* active_idx, int32_t n_active, const void* w_qkv, void* q_out, void* kv_out,
                         const fl_kv_store* store, int32_t* status, void* stream);

/* Stage 3 -- Eq. 8 with the quantizer of Appendix E (asymmetric, group-wise, min/max).
 * For each active row i = active_idx[t], X in {K, V}, head, group of `group` elements, in binary32:
 *   delta = X^(r)_i - Xhat^(r-1)_i            (Xhat^(r-1) rebuilt from base + streams of loops < r)
 *   zero  = fp16 round-down(min delta);  range = max delta - zero
 *   scale = range == 0 ? 0 : fp16 round-up(range / (2^bits - 1))
 *   code  = scale == 0 ? 0 : clamp(round-half-even((delta - zero) / scale), 0, 2^bits - 1)
 * and writes stream r (store->k_res[loop_r-2], v_res[loop_r-2]; codes/scale/zero pre-allocated by the
 * caller for n_rows == n_active, slot_of_pos already filled for loop r). |delta| must stay below 65504.
 * With bf16 storage and the stream's rows_prev / rows_cur set (K and V alike) it also writes, per active row,
 * Xhat^(r-1)_i and Xhat^(r)_i = Xhat^(r-1)_i + (code * scale + zero), each rounded once to bf16.
 * k_new, v_new: [n_active, H, dh] storage type. store is a host struct; store->n_streams must be
 * >= loop_r - 1 (the stream being written counts). Errors: loop_r < 2 or > FL_MAX_LOOPS+1, bad bits or
 * group, null buffers, n_rows mismatch; FL_ERR_UNSUPPORTED unless d = H*dh is a multiple of 256, and of 2048 beyond
 * 2048 (whole warps must walk a row together: the group reductions are sub-warp shuffles). n_active == 0 is a no-op.
 * `status` is accepted for symmetry and never written. */
FL_API int fl_quant_kv_residual(fl_ctx* ctx, const fl_shape* shape, int loop_r, const void* k_new, const void* v_new,
                         const int32_t* active_idx, int32_t n_active, const fl_kv_store* store,
                         int32_t* status, void* stream);

/* Dense source loop -- Eq. 2 for all L rows, causal, plus what loop 2 needs (Eq. 6 with m_C = 1):
 *   o [L, H, dh] storage type;  lse f32 [H, L] = log sum_{j<=i} exp(sm_scale q_i.k_j);
 *   col_scores f32 [H, nb, L]: col_scores[h,b,j] = sum_{i in block b, i >= j} p_ij for j <= last row of
 *   block b (entries beyond are not written). lse and col_scores may be NULL (col_scores needs lse). */
FL_API int fl_dense_loop_attention(fl_ctx* ctx, const fl_shape* shape, const void* q, const void* k, const void* v,
                            void* o, float* lse, float* col_scores, int32_t* status, void* stream);

/* Eq. 6: per (head, block) S = TopK_c over the candidate columns, ties to the lowest column.
 *   cand_cols == NULL : dense source. col_scores is [H, nb, L]; block b's candidates are columns
 *                       0 .. min(L, (b+1)*q_block)-1.
 *   cand_cols != NULL : sparse source. cand_cols int32 [H, nb, n_cand] ascending with cand_cnt[H, nb] valid
 *                       entries each; col_scores is [H, nb, n_cand], aligned with cand_cols.
 * Outputs: col_idx int32 [H, nb, c] ascending, padded with -1; col_cnt int32 [H, nb] = min(c, candidates).
 * n_cand is the row stride of the candidate arrays (L for a dense source). `status` is accepted for symmetry and never
 * written. */
FL_API int fl_select_columns(fl_ctx* ctx, const fl_shape* shape, const float* col_scores, const int32_t* cand_cols,
                      const int32_t* cand_cnt, int32_t n_cand, int32_t c, int32_t* col_idx, int32_t* col_cnt,
                      int32_t* status, void* stream);

/* Optional workspace for fl_loop_attention / fl_loop_attention_indexed (device memory of the caller, 256-byte
 * aligned; the paper has no counterpart: it is a scheduling aid of this implementation). The attention launch has one
 * CTA per (head, query block) problem and the problems cost about the same, so a problem count that is not a multiple
 * of the SM count ends in a partly empty wave. With a workspace of fl_loop_attention_workspace_bytes() bytes (0 when a
 * split cannot help the shape), the problems of that last wave are given to two CTAs each; the one that finishes
 * first leaves its partial accumulators there and the other adds them to its own, so the result does not depend on
 * which came first beyond the rounding order of that one addition. fl_set_workspace clears the arrival counters at the
 * head of the buffer on `stream` (every launch leaves them cleared, also one that reported FL_ERR_TIMEOUT through the
 * status word; the outputs of such a launch are undefined); the buffer must stay valid until fl_destroy or the next
 * fl_set_workspace (NULL detaches it). Attention calls of one context that may overlap in time (different
 * streams) must not share a workspace. */
FL_API int fl_loop_attention_workspace_bytes(fl_ctx* ctx, const fl_shape* shape, int64_t* bytes /* host */);
FL_API int fl_set_workspace(fl_ctx* ctx, void* workspace /* device */, int64_t bytes, void* stream);

/* Stages 2 + 4 -- Eq. 7 (equivalently Eq. 3) over the reconstructed K/V (Eq. 4 / Eq. 8): rows of tokens that are
 * active in loop r are read from the stream's rows_prev / rows_cur when fl_quant_kv_residual of loop r has left them
 * there (store->k_res[loop_r-2] and v_res[loop_r-2], all four buffers set), everything else is rebuilt inside the
 * kernel from the base and the residual streams.
 * For head h, active row t (position i = active_idx[t], block b), T_i = { j in col_idx[h,b,:] : j <= i }:
 *   p_old_j = exp(sm_scale q_old_t . Khat^(r-1)_j - lse_prev[h,i])       previous loop's probabilities
 *   m_i     = sum_{T_i} p_old_j                                          cached global mass
 *   p_new_j = m_i softmax_{T_i}(sm_scale q_new_t . Khat^(r)_j)
 *   o_out_t = o_prev_t - sum p_old_j Vhat^(r-1)_j + sum p_new_j Vhat^(r)_j
 *   lse_out[h,i] = logsumexp_{T_i}(sm_scale q_new_t . Khat^(r)_j) - log m_i
 *   col_scores_next[h,b,u] = sum over the block's active rows of p_new for column col_idx[h,b,u]
 * Rows with empty T_i keep o and lse. Khat^(r-1) uses streams of loops < r, Khat^(r) adds loop r
 * (store->n_streams >= loop_r - 1). q_new, q_old, o_prev, o_out: [n_active, H, dh] storage type;
 * lse_prev, lse_out: f32 [H, L] indexed by position (only active rows are read / written).
 * o_out may alias o_prev and lse_out may alias lse_prev. col_scores_next f32 [H, nb, c] or NULL. */
FL_API int fl_loop_attention(fl_ctx* ctx, const fl_shape* shape, int loop_r, const void* q_new, const void* q_old,
                      const int32_t* active_idx, int32_t n_active, const fl_kv_store* store,
                      const int32_t* col_idx, const int32_t* col_cnt, int32_t c, const float* lse_prev,
                      float* lse_out, const void* o_prev, void* o_out, float* col_scores_next,
                      int32_t* status, void* stream);

/* The same operation (Eq. 7 / Eq. 3 with Eq. 8 inside the kernel) on position-indexed stores, which removes the
 * gathers of Q^(r-1), O^(r-1) and the scatters of O^(r), Q^(r) around it (the gather / update steps of Appendix G):
 *   q_store_in  [L, H, dh]: row active_idx[t] holds q_old_t
 *   q_store_out [L, H, dh]: row active_idx[t] receives q_new_t (NULL: not written; may be q_store_in)
 *   o_store_in  [L, H, dh]: row active_idx[t] holds o_prev_t
 *   o_store_out [L, H, dh]: row active_idx[t] receives o_out_t (may be o_store_in)
 *   lse_in, lse_out f32 [H, L] by position (may be the same)
 * Rows of inactive positions are neither read nor written. q_new is [n_active, H, dh] as above. Tensor path only:
 * returns FL_ERR_UNSUPPORTED (nothing launched) unless dtype is FL_BF16, head_dim is 128 and c <= 3072, or when
 * the context was created with FL_FORCE_SIMT=1; callers then gather, call fl_loop_attention and scatter. */
FL_API int fl_loop_attention_indexed(fl_ctx* ctx, const fl_shape* shape, int loop_r, const void* q_new,
                              const void* q_store_in, void* q_store_out, const int32_t* active_idx, int32_t n_active,
                              const fl_kv_store* store, const int32_t* col_idx, const int32_t* col_cnt, int32_t c,
                              const float* lse_in, float* lse_out, const void* o_store_in, void* o_store_out,
                              float* col_scores_next, int32_t* status, void* stream);

/* Old-term economy for fl_loop_attention_indexed (Eq. 7 against Eq. 3: the old term of loop r is the cached
 * p^(r-1) Vhat^(r-1) over the selected columns, which is loop r-1's NEW term whenever the column set of the row's
 * (head, block) is unchanged since loop r-1 and the row was active in it; Eq. 6's cached mass m_i then carries over
 * unchanged too). With
 *   B_i = o^(w-1)_i - sum_{T_i} p_old_j Vhat^(w-1)_j      (the row's background, fixed at the last loop w that
 *                                                          recomputed the old term)
 * every later loop over the same sets is  o^(r)_i = B_i + sum_{T_i} p_new_j Vhat^(r)_j,  p_new = m_i softmax_{T_i}(.).
 *   bg_store [L, H, dh] storage type, by position; mass f32 [H, L] by position. Caller-owned, 16-byte aligned,
 *   distinct from the O stores; only rows / entries of active positions are touched.
 *   reuse == 0: the call computes what fl_loop_attention_indexed computes and also WRITES, for every active row,
 *               B_i (rounded once to the storage type) and m_i (0 for a row with empty T_i, whose B_i is o_prev_i).
 *   reuse != 0: the call READS B_i and m_i and computes the new term only: q_store_in, o_store_in and lse_in are not
 *               read (they may be NULL). Rows with m_i == 0 get o_out = B_i; their lse_out entry is copied from
 *               lse_in when that is given and left alone otherwise.
 * The caller guarantees, for a reuse call: col_idx / col_cnt are those of the call that wrote the buffers, and every
 * active row was active in that call (nested token sets, Appendix D.1). After the column sets are pruned the next
 * call must recompute (reuse == 0). The result differs from the recomputing form only by rounding (B is rounded to
 * the storage type once instead of the output of every loop). */
typedef struct {
  void* bg_store;
  float* mass;
  int32_t reuse;
  int32_t reserved_;
} fl_attn_carry;

/* fl_loop_attention_indexed with the carried old term; carry == NULL makes it that call exactly. Arguments, results
 * and errors otherwise as fl_loop_attention_indexed; additionally FL_ERR_INVALID_ARG when a buffer of `carry` is NULL,
 * misaligned or one of the O stores. */
FL_API int fl_loop_attention_indexed_carry(fl_ctx* ctx, const fl_shape* shape, int loop_r, const void* q_new,
                                    const void* q_store_in, void* q_store_out, const int32_t* active_idx,
                                    int32_t n_active, const fl_kv_store* store, const int32_t* col_idx,
                                    const int32_t* col_cnt, int32_t c, const float* lse_in, float* lse_out,
                                    const void* o_store_in, void* o_store_out, const fl_attn_carry* carry /* host */,
                                    float* col_scores_next, int32_t* status, void* stream);

/* fl_loop_attention_indexed with the workspace of its last-wave split (see fl_set_workspace) taken from a fixed array
 * that is part of the library's device image, for callers that cannot lend device memory (code that runs where
 * cudaMalloc is off limits: inside a region whose memory was budgeted up front, or under an allocator the caller does
 * not control); the context's own workspace, if any, is ignored by this call. The paper has no counterpart. The call
 * allocates and frees nothing. The array is 19.7 MB and every device that loads the library holds its own copy until
 * the process exits, whether this entry point is used or not. Its address is looked up on the first call per device
 * (cudaGetSymbolAddress, which answers for the CURRENT device: that call, like every later one, must be made with the
 * context's device current, else FL_ERR_CUDA and nothing is cached or launched); make that first call before any
 * stream capture. The arrival counters at the head of the array are cleared on `stream` before each launch, after the
 * arguments have passed the same host checks as fl_loop_attention_indexed (a rejected call enqueues nothing).
 * The array holds the partial results of at most 74 split problems (half of a B200's SMs); a shape whose split needs
 * more returns FL_ERR_WORKSPACE before anything is launched. There is one array per device and it keeps the last
 * call's contents: two of these calls that may overlap in time (different streams or contexts on one device) race on
 * it and must be serialised by the caller. Arguments, results and other errors as fl_loop_attention_indexed. */
FL_API int fl_loop_attention_indexed_static(fl_ctx* ctx, const fl_shape* shape, int loop_r, const void* q_new,
                                     const void* q_store_in, void* q_store_out, const int32_t* active_idx,
                                     int32_t n_active, const fl_kv_store* store, const int32_t* col_idx,
                                     const int32_t* col_cnt, int32_t c, const float* lse_in, float* lse_out,
                                     const void* o_store_in, void* o_store_out, float* col_scores_next,
                                     int32_t* status, void* stream);

/* Sparse decode attention -- Eq. 6-7 as Appendix D.2 writes them, for decode positions (Appendix G, the item on
 * sparse decode kernels): loop r >= 2 of n_queries single-token queries that follow the prompt, over the prompt's
 * store. Query t, head h has its OWN selected subset S = col_idx[t, h, :col_cnt[t, h]] (ascending positions of the
 * prompt, padded with -1; every one of them is causal for a decode position) and log-normaliser lse_prev[t, h] with
 * p_old_j = exp(sm_scale q_old . Khat^(r-1)_j - lse_prev) (a dense source loop gives lse_prev = logsumexp over all keys):
 *   m = sum_S p_old_j;  p_new_j = m softmax_S(sm_scale q_new . Khat^(r)_j);
 *   o_out = o_prev - sum_S p_old_j Vhat^(r-1)_j + sum_S p_new_j Vhat^(r)_j;  lse_out = logsumexp_S - log m;
 *   p_new_out[t, h, u] = p_new of column S[u] (the scores from which the next loop's subset is pruned; 0 beyond the
 *   count), or NULL.
 * K/V of the selected columns are rebuilt inside the kernel from the base and the residual streams (Eq. 8), rounded
 * to the storage type where attention consumes them. q_new, q_old, o_prev, o_out: [n_queries, H, dh] storage type
 * (o_out may alias o_prev); lse_prev, lse_out: f32 [n_queries, H] (may alias). A query with an empty subset keeps its
 * output and log-normaliser. The decode tokens' own K/V (the short full-precision tail of Appendix E) are not part of
 * this call. `status` is accepted for symmetry and never written. */
FL_API int fl_decode_attention(fl_ctx* ctx, const fl_shape* shape, int loop_r, const void* q_new, const void* q_old,
                        int32_t n_queries, const fl_kv_store* store, const int32_t* col_idx, const int32_t* col_cnt,
                        int32_t c, const float* lse_prev, float* lse_out, const void* o_prev, void* o_out,
                        float* p_new_out, int32_t* status, void* stream);

/* Quantized loop-1 base (Appendix E, "Quantization Setting"): the quantizer of the residual streams (asymmetric,
 * scale and offset from the group's minimum and maximum, shape->bits bits) applied to the base K and V of a layer, the
 * keys grouped PER CHANNEL (a group = `group` consecutive positions of one channel) and the values PER TOKEN (a group =
 * `group` consecutive channels of one position); the most recent `tail` positions stay in the storage type.
 * With Lq = max(0, L - tail), d = H*dh, all device buffers owned by the caller, 16-byte aligned:
 *   k_codes, v_codes : uint8 [Lq, d*bits/8]  packed like the residual codes (little-endian inside a byte)
 *   k_scale, k_zero  : fp16  [ceil(Lq/group), d]      (the last token group may be shorter)
 *   v_scale, v_zero  : fp16  [Lq, d/group]
 *   k_tail, v_tail   : storage type [L - Lq, d]        rows Lq .. L-1 as they are */
typedef struct {
  void* k_codes; void* k_scale; void* k_zero;
  void* v_codes; void* v_scale; void* v_zero;
  void* k_tail;  void* v_tail;
  int32_t group; /* 32, 64 or 128; must divide d */
  int32_t tail;  /* >= 0 */
} fl_kv_base_q; /* host struct holding device pointers */

/* Packs k, v ([L, H, dh] storage type) into `base`. Arithmetic as in fl_quant_kv_residual, in binary32:
 *   zero = fp16 round-down(min);  scale = fp16 round-up((max - zero) / (2^bits - 1)), 0 for a constant group;
 *   code = clamp(round-half-even((x - zero) / scale), 0, 2^bits - 1).
 * fl_dequant_kv_base writes rows of k_out, v_out ([L, H, dh] storage type): rows below Lq as
 * storage-round(fma(code, scale, zero)), the tail rows copied back. row_mask = NULL rebuilds every row; otherwise
 * (device uint32 [H, ceil(L/32)], bit t%32 of word [h][t/32]) only the (head, position) pairs whose bit is set, and
 * the rest of k_out / v_out is left untouched (the tail rows are always copied). The sparse loops then run on
 * k_out / v_out as their base: the packed form is what stays resident, the rebuilt rows are a transient copy of one
 * layer. fl_mark_base_rows fills such a mask with what the sparse loops of a layer read (Appendix D.2: attention
 * touches the selected columns only; Eq. 8: the residual chain starts from the base rows of the active positions):
 * for every head the first col_cnt[h, b] entries of col_idx[h, b, :] of all its blocks, plus active_idx[0..n_active).
 * It clears the mask first. A mask made with the active set of loop r also serves every later loop whose active set
 * is nested in it and whose column lists are subsets.
 * Errors: FL_ERR_INVALID_ARG for null or misaligned buffers, a group other than 32 / 64 / 128, tail < 0;
 * FL_ERR_UNSUPPORTED when shape->bits is 16, or d is not a multiple of 256 and of the group. `status` is never
 * written. fl_kv_base_q_bytes returns the bytes of the packed form (codes, metadata and tail, K and V). */
FL_API int fl_quant_kv_base(fl_ctx* ctx, const fl_shape* shape, const void* k, const void* v, const fl_kv_base_q* base,
                     int32_t* status, void* stream);
FL_API int fl_dequant_kv_base(fl_ctx* ctx, const fl_shape* shape, const fl_kv_base_q* base, const uint32_t* row_mask,
                       void* k_out, void* v_out, int32_t* status, void* stream);
FL_API int fl_mark_base_rows(fl_ctx* ctx, const fl_shape* shape, const int32_t* col_idx, const int32_t* col_cnt, int32_t c,
                      const int32_t* active_idx, int32_t n_active, uint32_t* row_mask, int32_t* status, void* stream);
FL_API int fl_kv_base_q_bytes(const fl_shape* shape, int32_t group, int32_t tail, int64_t* bytes);

/* The checked build (libflashloop_debug.so, compiled with -DFL_DEBUG_BOUNDS) validates, before every launch, the
 * index arrays the call is about to trust: row lists (range, strictly ascending), column lists against their counts
 * (range, ascending, counts within [0, c]), candidate lists, and the slot maps of the residual streams the call reads
 * (each value -1 or a row of its stream), and fl_select_tokens its two hidden-state matrices (every value finite). A small
 * kernel reads the arrays (never what they point to), the host waits for
 * its verdict, and on a violation the call returns FL_ERR_INVALID_ARG, writes that code to `status` when one was given
 * (also in the calls whose normal build never writes it) and launches nothing else. Nothing traps. The wait makes the
 * checked build slow and unusable inside a stream capture: it is for tests and debugging. Returns 1 in the checked
 * build, 0 otherwise. */
FL_API int fl_debug_bounds_enabled(void);

/* KV-cache accounting (Section 1's 48 GiB example; Section 4.3): bytes held for one layer by this store
 * after n_loops loops, and by a dense looped cache of n_loops loops. Host-only, no device access.
 * share_layers = number of layers sharing each loop's slot map and index list (>= 1). */
FL_API int fl_kv_store_bytes(const fl_shape* shape, const fl_kv_store* store, int n_loops, int share_layers,
                      int64_t* flashloop_bytes /* host */, int64_t* dense_bytes /* host */);

#ifdef __cplusplus
}
#endif
#endif /* FLASHLOOP_H_ */
