/*
 * spa.h - C boundary of the Select-and-Pack-Attention (SPA) block library for NVIDIA B200 (sm_100a).
 *
 * One SPA block (Ren et al., "Context-Aware Token Selection and Packing for Enhanced Vision
 * Transformer", Sec. 3.2): a linear gate scores every token (Eq. 4); tokens whose logit exceeds a
 * threshold are selected (deterministic form of Eq. 6); the selections of all images are packed
 * into one dense buffer ("Token Packing"); QKV projection, self-attention restricted to tokens of
 * the same image, and the output projection run on the packed buffer; results are scattered back
 * and unselected tokens pass through unchanged.
 *
 * Conventions shared by every call
 *   - All tensor pointers are DEVICE pointers owned by the caller, 16-byte aligned, unless a
 *     parameter is explicitly documented as a host pointer.  The library never allocates or
 *     frees device memory; scratch comes from the caller-provided `workspace`
 *     (spa_workspace_bytes() bytes, 256-byte aligned).
 *   - `stream` is a cudaStream_t passed as void*.  Calls validate their arguments on the host
 *     and return a negative spa_status synchronously; otherwise they enqueue work on `stream`
 *     and return SPA_OK without synchronising.
 *   - Conditions only the device can see (more selected tokens than `capacity`, a bounded wait
 *     that ran out) are recorded in the int32 `d_status` word (first error wins; the caller zeroes
 *     it) and the kernels finish cleanly.  `d_status` may be NULL.
 *   - Storage dtype T is float (SPA_F32) or bfloat16 (SPA_BF16); accumulation is always fp32.
 *     C*sizeof(T) and (C/H)*sizeof(T) must be multiples of 16 bytes; C/H must be 32 or 64.
 *   - Packed buffers have `capacity` rows allocated (capacity <= B*N); only the first
 *     N_p = cu_seqlens[B] rows are defined.  N_p lives on the device: no call reads it back.
 *   - Layouts are row-major with the last index contiguous: x[B][N][C], x_packed[capacity][C],
 *     qkv[capacity][3C] with column = which*C + h*(C/H) + e (which = 0,1,2 for q,k,v),
 *     attn_out[capacity][C] with column = h*(C/H) + e, lse[H][capacity], weights W[out][in].
 */
#ifndef SPA_H_
#define SPA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SPA_OK = 0,
  SPA_ERR_INVALID_ARG = -1, /* null pointer, non-positive size, misaligned pointer          */
  SPA_ERR_UNSUPPORTED = -2, /* dtype, head dimension or row size the kernels do not cover   */
  SPA_ERR_CAPACITY = -3,    /* device: more selected tokens than `capacity`                 */
  SPA_ERR_CUDA = -4,        /* a CUDA runtime call failed (see spa_last_cuda_error)         */
  SPA_ERR_TIMEOUT = -5,     /* device: a bounded wait expired                               */
  SPA_ERR_SCRATCH = -6      /* the problem needs more scratch than the built-in array holds */
} spa_status;

typedef enum { SPA_F32 = 0, SPA_BF16 = 1 } spa_dtype;

enum {
  SPA_FLAG_RESIDUAL = 1,  /* selected rows: y = x + z instead of y = z                     */
  SPA_FLAG_INPLACE = 2,   /* spa_unpack_scatter: y aliases x, only selected rows written   */
  SPA_FLAG_GATE_SCALE = 4,/* Eq. 5: packed rows are scaled by sigmoid(score)               */
  SPA_FLAG_SIMT_ONLY = 8, /* bf16 only: run the fp32-FMA kernels instead of the tensor-core ones */
  SPA_FLAG_NO_CTA_PAIRS = 16,/* wide linear layers: keep the one-CTA tensor-core kernels (no CTA pairs) */
  SPA_FLAG_UNFUSED = 32,  /* spa_block_fwd / spa_block_bwd: separate projection, scatter and gather kernels even
                             where the fused calls apply                                                      */
  SPA_FLAG_ONE_PASS_BWD = 64 /* attention backward (tensor-core problems): segments of at most 128 rows are handled by
                             a kernel that owns a whole segment and evaluates S, P, dP, dS once; the two-pass kernels
                             take the longer segments only.  Same results within the stated tolerances               */
};

typedef struct spa_params {
  int32_t B;          /* images in the batch                                             */
  int32_t N;          /* tokens per image                                                */
  int32_t C;          /* channels                                                        */
  int32_t H;          /* attention heads; head dimension d = C / H                       */
  int32_t dtype;      /* spa_dtype of x, weights, packed buffers                         */
  int32_t flags;      /* SPA_FLAG_* bits                                                 */
  int32_t capacity;   /* rows allocated in packed buffers, 1 <= capacity <= B*N          */
  float tau;          /* selection threshold on the gate logit                           */
  float softmax_scale;/* 0 selects 1/sqrt(d)                                             */
} spa_params;

/* Bytes of scratch the calls below that take `workspace` need for these parameters. */
size_t spa_workspace_bytes(const spa_params* p);

/* Gate and hard selection (Sec. 3.2, Eq. 4 and the thresholded form of Eq. 6).
 *   scores[b*N+n] = b_g + sum_c w_g[c] * x[b][n][c];  if s_up != NULL, scores = max(scores, s_up).
 *   mask[b*N+n]   = scores > tau ? 1 : 0   (strict).
 * x: T[B][N][C]; w_g: T[C]; b_g: host scalar; s_up: float[B*N] or NULL;
 * scores: float[B*N] out; mask: uint8[B*N] out. */
int spa_gate(const spa_params* p, const void* x, const void* w_g, float b_g, const float* s_up,
             float* scores, uint8_t* mask, void* stream);

/* Token packing (Sec. 3.2 "Token Packing"): stable compaction of the selected tokens, images in
 * batch order and tokens in raster order.
 *   cu_seqlens[0] = 0, cu_seqlens[b+1] = cu_seqlens[b] + popcount(mask[b][:]);
 *   idx[i] = flat position b*N+n of packed row i (ascending);  inv[b*N+n] = i or -1;
 *   x_packed[i][:] = x[idx[i]][:]   (times sigmoid(scores[idx[i]]) under SPA_FLAG_GATE_SCALE).
 * mask: uint8[B*N] (non-zero = selected); scores: float[B*N], only read under GATE_SCALE, else
 * may be NULL; x_packed: T[capacity][C] out; idx: int32[capacity] out; inv: int32[B*N] out or
 * NULL; cu_seqlens: int32[B+1] out.  If more than `capacity` tokens are selected the surplus rows
 * are dropped, cu_seqlens still holds the true counts and SPA_ERR_CAPACITY is recorded in d_status;
 * every later call clamps N_p to capacity.  B*N must not exceed 2^20. */
int spa_select_pack(const spa_params* p, const void* x, const uint8_t* mask, const float* scores,
                    void* x_packed, int32_t* idx, int32_t* inv, int32_t* cu_seqlens,
                    int32_t* d_status, void* stream);

/* spa_select_pack with each image's tokens visited in the order order[0], order[1], ... (int32[N], a
 * permutation of 0..N-1; the same for every image) instead of raster order: the cyclic shift of the feature
 * map that the paper applies every two blocks so that other tokens share a container (Sec. 1).  mask, scores,
 * idx and inv stay indexed by the original token, so every later call is unchanged; only the order of the
 * packed rows inside each image differs.  The order array is read on the device. */
int spa_select_pack_ordered(const spa_params* p, const void* x, const uint8_t* mask, const float* scores,
                            const int32_t* order, void* x_packed, int32_t* idx, int32_t* inv,
                            int32_t* cu_seqlens, int32_t* d_status, void* stream);

/* spa_gate (or spa_gate_prefill when y != NULL) and spa_select_pack in one pass over x (Sec. 3.2, Eq. 4, Eq. 6,
 * "Token Packing"): x is read once, the selected rows go from registers to x_packed.  Same outputs, bit for bit, as
 * the two calls.  Rows of at most 128 16-byte chunks (1024 bf16 or 512 fp32 channels): spa_gate_select_pack_supported
 * says whether the call applies, else it returns SPA_ERR_UNSUPPORTED.
 * pack_state: spa_pack_state_bytes() bytes of device memory that must be ZERO when the call starts; the kernel
 * leaves it zero again (also after an error), so the caller clears it once, after allocating it.  Two calls that
 * share one pack_state must not overlap on the GPU.  Tiles of tokens exchange their selected counts through it;
 * every wait on it is bounded (SPA_ERR_TIMEOUT in d_status when one runs out; the packed outputs are then undefined). */
size_t spa_pack_state_bytes(const spa_params* p);
int spa_gate_select_pack_supported(const spa_params* p);
int spa_gate_select_pack(const spa_params* p, const void* x, const void* w_g, float b_g, const float* s_up,
                         float* scores, uint8_t* mask, void* y, void* x_packed, int32_t* idx, int32_t* inv,
                         int32_t* cu_seqlens, void* pack_state, int32_t* d_status, void* stream);

/* Attention segments of the paper's own batching (Sec. 3.2 "Token Packing": the selected tokens fill containers of a
 * fixed length L = M^2, and the mask keeps a token from attending to tokens of other images): the packed buffer is cut
 * at every multiple of L and at every image boundary.  seg_offsets (device, int32[spa_container_max_segments() + 1])
 * receives the distinct cut positions in ascending order - 0 first, N_p last - padded with copies of N_p (empty
 * segments).  Pass it to the attention calls with n_seg = spa_container_max_segments(p, L) = B + capacity / L: nothing
 * is read back to the host, so the container variant runs inside the same recorded step as everything else.
 * B is limited to 4095 images (else SPA_ERR_UNSUPPORTED); L >= 1. */
int32_t spa_container_max_segments(const spa_params* p, int32_t L);
int spa_container_offsets(const spa_params* p, const int32_t* cu_seqlens, int32_t L, int32_t* seg_offsets,
                          void* stream);

/* QKV projection on the packed tokens (the 3LC^2 term of Eq. 9):
 *   qkv[i][j] = b_qkv[j] + sum_c W_qkv[j][c] * x_packed[i][c],  i < N_p, j < 3C.
 * W_qkv: T[3C][C]; b_qkv: T[3C] or NULL; qkv: T[capacity][3C] out. */
int spa_packed_qkv(const spa_params* p, const void* x_packed, const void* W_qkv, const void* b_qkv,
                   const int32_t* cu_seqlens, void* qkv, int32_t* d_status, void* stream);

/* Multi-head self-attention in which a packed token attends only to tokens of its own segment
 * (Sec. 3.2: the attention mask keeps tokens from attending to other images; the 2L^2C term).
 * For segment s = [seg_offsets[s], seg_offsets[s+1]) and head h, over rows i, j of the segment:
 *   S_ij = scale * q_i . k_j;  P = softmax_j(S);  attn_out_i = sum_j P_ij v_j;
 *   lse[h][i] = log sum_j exp(S_ij).
 * seg_offsets: int32[n_seg+1], ascending, seg_offsets[0] = 0; pass cu_seqlens and B for the
 * default same-image mask.  N_p = seg_offsets[n_seg].  attn_out: T[capacity][C]; lse: float[H][capacity]. */
int spa_packed_attention_fwd(const spa_params* p, const void* qkv, const int32_t* seg_offsets,
                             int32_t n_seg, void* attn_out, float* lse, int32_t* d_status,
                             void* stream);

/* Gradient of spa_packed_attention_fwd with respect to qkv (the paper trains through the block,
 * Sec. 1; it gives no derivation, this is the standard softmax-attention gradient):
 *   D_i = sum_e d_attn_out_ie * attn_out_ie;  P_ij = exp(S_ij - lse_i);
 *   dV_j = sum_i P_ij dO_i;  dS_ij = P_ij (dO_i . v_j - D_i);
 *   dQ_i = scale * sum_j dS_ij k_j;  dK_j = scale * sum_i dS_ij q_i.
 * dqkv: T[capacity][3C] out, same column layout as qkv.  workspace: scratch, may be NULL when
 * spa_workspace_bytes() is 0. */
int spa_packed_attention_bwd(const spa_params* p, const void* qkv, const void* attn_out,
                             const float* lse, const void* d_attn_out, const int32_t* seg_offsets,
                             int32_t n_seg, void* dqkv, void* workspace, int32_t* d_status,
                             void* stream);

/* Attention backward for callers that cannot hand over scratch memory.  (The paper has no
 * counterpart: this is a packaging variant of spa_packed_attention_bwd, same arithmetic.)
 *
 * Who needs it: code that runs where device allocation is off the table - inside a region that is
 * being recorded for later replay, inside a framework whose memory pool is frozen or owned by
 * someone else, in a plugin that is only handed its input and output tensors, or under a memory
 * budget fixed at start-up.  Such callers cannot call cudaMalloc (or any allocator built on it) to
 * obtain the `workspace` the regular call wants, so here the per-row scratch (D_i, one float per
 * head and packed row) lives in an array that is part of the library image itself.
 *
 * Limits and rules:
 *   - bf16 problems with head dimension 32 or 64 only (the tensor-core path); anything else returns
 *     SPA_ERR_UNSUPPORTED.
 *   - H * capacity * sizeof(float) must not exceed SPA_STATIC_SCRATCH_BYTES, else SPA_ERR_SCRATCH.
 *     Every GPU on which the library is loaded holds that many bytes until the process exits.
 *   - The call allocates nothing and frees nothing, on the device or through any library.
 *   - The first call on each device looks up the array's device address (once, with that device
 *     current); make that first call before any stream capture begins.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left.
 *     Nothing in it has to start at zero: each call writes every entry before reading it.  Two
 *     calls whose kernels overlap on the GPU (different streams, no ordering) race on it; keep
 *     calls to this entry point ordered with respect to one another.
 * Arguments are those of spa_packed_attention_bwd without `workspace`. */
#define SPA_STATIC_SCRATCH_BYTES (4u << 20)
int spa_packed_attention_bwd_static(const spa_params* p, const void* qkv, const void* attn_out,
                                    const float* lse, const void* d_attn_out,
                                    const int32_t* seg_offsets, int32_t n_seg, void* dqkv,
                                    int32_t* d_status, void* stream);

/* Output projection on the packed tokens:  z[i][j] = b_o[j] + sum_c W_o[j][c] * a[i][c].
 * a: T[capacity][C]; W_o: T[C][C]; b_o: T[C] or NULL; z: T[capacity][C] out. */
int spa_packed_proj(const spa_params* p, const void* a, const void* W_o, const void* b_o,
                    const int32_t* cu_seqlens, void* z, int32_t* d_status, void* stream);

/* Unpack: y[b][n][:] = z_packed[inv[b*N+n]][:] for selected tokens, x[b][n][:] otherwise
 * (Sec. 3.2: negative tokens are passed on unchanged).  SPA_FLAG_RESIDUAL adds x on selected rows.
 * Out of place (y != x) every row of y is written; under SPA_FLAG_INPLACE y must equal x and only
 * the selected rows are written. */
int spa_unpack_scatter(const spa_params* p, const void* z_packed, const void* x, const int32_t* idx,
                       const int32_t* inv, const int32_t* cu_seqlens, void* y, int32_t* d_status,
                       void* stream);

/* Transpose of spa_unpack_scatter:  dz_packed[i][:] = dY[idx[i]][:];  dX[t][:] = dY[t][:] for
 * unselected tokens t.  Selected rows of dX are left for spa_select_pack_bwd (under
 * SPA_FLAG_RESIDUAL they receive dY too, the term that the residual adds).  dX may equal dY
 * (nothing is copied then) or be NULL. */
int spa_unpack_scatter_bwd(const spa_params* p, const void* dY, const int32_t* idx,
                           const int32_t* inv, const int32_t* cu_seqlens, void* dz_packed, void* dX,
                           void* stream);

/* Transpose of the pack gather:  dX[idx[i]][:] = dx_packed[i][:]  (+ dY[idx[i]][:] under
 * SPA_FLAG_RESIDUAL; dY may be NULL otherwise). */
int spa_select_pack_bwd(const spa_params* p, const void* dx_packed, const void* dY,
                        const int32_t* idx, const int32_t* cu_seqlens, void* dX, void* stream);

/* Gradients of a packed linear layer out = a W^T + b with W: T[n_out][n_in]:
 *   da[i][:] = dout[i][:] W           (T[capacity][n_in], may be NULL)
 *   dW = dout^T a                     (float[n_out][n_in], may be NULL)
 *   db[j] = sum_i dout[i][j]          (float[n_out], may be NULL)
 * Sums over packed rows run in a fixed order: results are bitwise reproducible.
 * n_in and n_out must be multiples of 16 bytes / sizeof(T). */
int spa_packed_linear_bwd(const spa_params* p, const void* a, const void* W, const void* dout,
                          int32_t n_in, int32_t n_out, const int32_t* cu_seqlens, void* da,
                          float* dW, float* db, void* workspace, int32_t* d_status, void* stream);

/* Fused unpack (Sec. 3.2: selected tokens are replaced by the block's output, the others pass through).
 * The three calls below give the same results as spa_packed_proj + spa_unpack_scatter and as
 * spa_packed_linear_bwd + spa_select_pack_bwd, without the packed intermediate (z, dx_packed) and
 * without the separate scatter kernel: the matrix product writes its rows straight to their tokens.
 * Tensor-core problems only (bf16, C a multiple of 8, C >= 64): spa_fused_scatter_supported says
 * whether they apply; otherwise they return SPA_ERR_UNSUPPORTED and the unfused calls must be used. */
int spa_fused_scatter_supported(const spa_params* p);

/* spa_gate that also writes y[B][N][C] = x while it reads x (nothing is copied when y == x): the
 * pass-through rows of the fused unpack at no second read of x. */
int spa_gate_prefill(const spa_params* p, const void* x, const void* w_g, float b_g, const float* s_up,
                     float* scores, uint8_t* mask, void* y, void* stream);

/* dst[B][N][C] = src[B][N][C]: writes the pass-through rows ahead of the scatter (y = x in the
 * forward pass, dX = dY in the backward pass).  A no-op when dst == src. */
int spa_unpack_prefill(const spa_params* p, const void* src, void* dst, void* stream);

/* Output projection with the unpack scatter in its epilogue:  y[idx[i]][:] = b_o + W_o a[i][:]
 * (added to y[idx[i]][:] under SPA_FLAG_RESIDUAL).  y: T[B][N][C] must already hold x
 * (spa_gate_prefill, spa_unpack_prefill, or y aliasing x); rows of unselected tokens are not touched. */
int spa_packed_proj_scatter(const spa_params* p, const void* a, const void* W_o, const void* b_o,
                            const int32_t* idx, const int32_t* cu_seqlens, void* y, int32_t* d_status,
                            void* stream);

/* spa_packed_linear_bwd with the transpose of the pack gather in the epilogue of the input gradient:
 * dX[idx[i]][:] = dout[i][:] W  (added to dX[idx[i]][:] under SPA_FLAG_RESIDUAL, where dX must
 * already hold dY: spa_unpack_scatter_bwd copies those rows too when the flag is set).  n_in must equal C; dW, db and workspace as in spa_packed_linear_bwd. */
int spa_packed_linear_bwd_scatter(const spa_params* p, const void* a, const void* W, const void* dout,
                                  int32_t n_in, int32_t n_out, const int32_t* idx,
                                  const int32_t* cu_seqlens, void* dX, float* dW, float* db,
                                  void* workspace, int32_t* d_status, void* stream);

/* ---- Trainable selection (Sec. 3.2 multi-scale supervised selection, Eq. 4-5; Sec. 3.3 Eq. 10) ---------
 * With SPA_FLAG_GATE_SCALE the packed rows are Sigmoid(s) x (Eq. 5) and a gradient reaches the gate.  The hard
 * selection itself has no gradient.  Order of the calls in a backward pass: spa_select_loss (writes ds),
 * ..., spa_select_pack_bwd_gated (adds to ds), spa_gate_bwd (consumes ds).  All buffers are device memory. */

/* Bytes of scratch that spa_select_loss, spa_gate_bwd and spa_layer_norm_bwd need (per-CTA partial sums). */
size_t spa_train_workspace_bytes(const spa_params* p);

/* Scores of the previous, finer stage, float[B][2*rows][2*cols], max-pooled 2x2 to this stage's grid:
 * s_up float[B][rows*cols], the second argument of Max in Eq. 4. */
int spa_score_pool(const float* scores_prev, int32_t B, int32_t rows, int32_t cols, float* s_up, void* stream);

/* Selection loss of one block, Eq. 10: loss = -sum_t (y_t log p_t + (1 - y_t) log(1 - p_t)), p = Sigmoid(scores),
 * y = labels (uint8 0/1, [B*N]).  Writes ds[t] = alpha (p_t - y_t) for every token and, if loss != NULL, the
 * unweighted sum to *loss (device float).  labels == NULL: ds = 0 and loss = 0 (clears ds for the calls below). */
int spa_select_loss(const spa_params* p, const float* scores, const uint8_t* labels, float alpha, float* ds,
                    float* loss, void* workspace, void* stream);

/* Transpose of the pack gather under SPA_FLAG_GATE_SCALE:  dX[idx[i]][:] = Sigmoid(s) dx_packed[i][:]
 * (+ dY[idx[i]][:] under SPA_FLAG_RESIDUAL) and  ds[idx[i]] += Sigmoid'(s) (dx_packed[i] . x[idx[i]]),
 * s = scores[idx[i]].  Replaces spa_select_pack_bwd. */
int spa_select_pack_bwd_gated(const spa_params* p, const void* dx_packed, const void* x, const float* scores,
                              const void* dY, const int32_t* idx, const int32_t* cu_seqlens, void* dX,
                              float* ds, void* stream);

/* Backward of spa_gate given ds = gradient at the stored (post-Max) scores.  Where the linear layer supplied
 * the maximum (scores > s_up, or s_up == NULL):  dX[t][:] += ds[t] w_g,  dw_g = sum_t ds[t] x[t][:]  (float[C]),
 * db_g = sum_t ds[t] (device float, may be NULL); elsewhere ds_up[t] = ds[t] (float[B*N], may be NULL; zero where
 * the linear layer won).  Sums over tokens run in a fixed order.  C is limited to 128 16-byte chunks per row
 * (1024 bf16 or 512 fp32 channels); beyond that the call returns SPA_ERR_UNSUPPORTED. */
int spa_gate_bwd(const spa_params* p, const void* x, const void* w_g, const float* scores, const float* s_up,
                 const float* ds, void* dX, float* dw_g, float* db_g, float* ds_up, void* workspace,
                 void* stream);

/* ---- The rest of the pre-norm transformer block around SPA (Sec. 3.2: selected tokens go through attention,
 * the others straight to the feed-forward network).  The paper prints no formula for these standard parts;
 * they are: LayerNorm over the channels, linear layers over all tokens, the exact (erf) GELU. --------------- */

/* out[i][:] = b + W a[i][:] for the rows that cu_seqlens[B] counts (W: T[n_out][n_in], b: T[n_out] or NULL,
 * a: T[capacity][n_in], out: T[capacity][n_out]).  accumulate != 0 adds the result to what out holds (a residual
 * branch).  With cu_seqlens[b] = b*N the layer runs over every token.  spa_packed_linear_bwd is its backward. */
int spa_packed_linear(const spa_params* p, const void* a, const void* W, const void* b, int32_t n_in,
                      int32_t n_out, const int32_t* cu_seqlens, void* out, int32_t accumulate,
                      int32_t* d_status, void* stream);

/* y = (x - mean) * rstd * gamma + beta over the C channels of each of the B*N tokens; mean, rstd: float[B*N] out
 * (saved for the backward).  C is limited to 128 16-byte chunks per row (else SPA_ERR_UNSUPPORTED). */
int spa_layer_norm(const spa_params* p, const void* x, const void* gamma, const void* beta, float eps, void* y,
                   float* mean, float* rstd, void* stream);

/* Backward of spa_layer_norm: dx (+ add[t][:] if add != NULL: the gradient of a residual branch), dgamma and
 * dbeta (float[C], sums over tokens in a fixed order).  workspace: spa_train_workspace_bytes. */
int spa_layer_norm_bwd(const spa_params* p, const void* dy, const void* x, const void* gamma, const float* mean,
                       const float* rstd, const void* add, void* dx, float* dgamma, float* dbeta,
                       void* workspace, void* stream);

/* h = gelu(u) = u Phi(u) and du = dh * gelu'(u) over T[B*N][n_cols]; du may alias dh. */
int spa_gelu(const spa_params* p, const void* u, int32_t n_cols, void* h, void* stream);
int spa_gelu_bwd(const spa_params* p, const void* dh, const void* u, int32_t n_cols, void* du, void* stream);

/* ---- The block as one unit (Sec. 3.2: gate -> select and pack -> attention on the packed tokens -> unpack; Eq. 9
 * counts it as one).  spa_block_fwd and spa_block_bwd issue the calls above in order on `stream`; they choose the
 * fused calls where spa_fused_scatter_supported() allows (unless SPA_FLAG_UNFUSED), and spa_block_bwd runs the two
 * weight-gradient products on a second stream beside the attention backward when `overlap` is given.  Nothing
 * synchronises with the host, so both can be recorded into one CUDA graph.
 *
 * All pointers are device memory owned by the caller and sized as in the single calls (packed buffers: `capacity`
 * rows).  Which fields may be NULL:
 *   s_up, order, seg_offsets (NULL: the images are the attention segments), b_qkv, b_o, pack_state;
 *   z, dx_packed            when the fused calls apply (the products write y and dX rows themselves);
 *   every backward field    for spa_block_fwd;
 *   labels .. train_workspace unless `trainable` is non-zero.
 * The forward pass leaves scores, mask, cu_seqlens, idx, inv, x_packed, qkv, attn_out, lse for the backward pass. */
typedef struct spa_overlap spa_overlap;  /* a second stream and the two events that fork to it and join it */

typedef struct spa_block_buffers {
  /* inputs of the forward pass */
  const void* x;              /* T[B][N][C]                                                          */
  const void* w_g;            /* T[C]                                                                */
  float b_g;
  const float* s_up;          /* float[B*N] or NULL (Eq. 4)                                          */
  const void* W_qkv;          /* T[3C][C]                                                            */
  const void* b_qkv;          /* T[3C] or NULL                                                       */
  const void* W_o;            /* T[C][C]                                                             */
  const void* b_o;            /* T[C] or NULL                                                        */
  const int32_t* order;       /* int32[N] packing order of each image's tokens, or NULL (raster)     */
  const int32_t* seg_offsets; /* int32[n_seg+1] attention segments, or NULL (cu_seqlens, B)          */
  int32_t n_seg;
  /* results and intermediates of the forward pass */
  float* scores;              /* float[B*N]                                                          */
  uint8_t* mask;              /* uint8[B*N]                                                          */
  int32_t* cu_seqlens;        /* int32[B+1]                                                          */
  int32_t* idx;               /* int32[capacity]                                                     */
  int32_t* inv;               /* int32[B*N]                                                          */
  void* x_packed;             /* T[capacity][C]                                                      */
  void* qkv;                  /* T[capacity][3C]                                                     */
  void* attn_out;             /* T[capacity][C]                                                      */
  float* lse;                 /* float[H][capacity]                                                  */
  void* z;                    /* T[capacity][C]; unfused path only                                   */
  void* y;                    /* T[B][N][C]; equal to x under SPA_FLAG_INPLACE                       */
  /* backward pass */
  const void* dY;             /* T[B][N][C]                                                          */
  void* dz;                   /* T[capacity][C]                                                      */
  void* d_attn_out;           /* T[capacity][C]                                                      */
  void* dqkv;                 /* T[capacity][3C]                                                     */
  void* dx_packed;            /* T[capacity][C]; unfused path only                                   */
  void* dX;                   /* T[B][N][C]                                                          */
  float* dW_qkv;              /* float[3C][C]                                                        */
  float* db_qkv;              /* float[3C]                                                           */
  float* dW_o;                /* float[C][C]                                                         */
  float* db_o;                /* float[C]                                                            */
  void* workspace;            /* spa_workspace_bytes()                                               */
  void* workspace_side;       /* a second area of that size; needed when `overlap` is given          */
  void* pack_state;           /* spa_pack_state_bytes(), zeroed once by the caller, or NULL: gate and
                                 packing then run as two kernels                                     */
  spa_overlap* overlap;       /* spa_overlap_create(), or NULL: everything on `stream`               */
  int32_t* d_status;          /* device status word or NULL                                          */
  /* trainable selection (Eq. 4-5, Eq. 10): gradient to the gate */
  int32_t trainable;          /* non-zero: spa_block_bwd also runs the four calls of that section    */
  const uint8_t* labels;      /* uint8[B*N] or NULL (no selection loss)                              */
  float alpha;                /* weight of the selection loss                                        */
  float* ds;                  /* float[B*N]                                                          */
  float* ds_up;               /* float[B*N] or NULL                                                  */
  float* dw_g;                /* float[C]                                                            */
  float* db_g;                /* float[1] or NULL                                                    */
  float* loss;                /* float[1] or NULL                                                    */
  void* train_workspace;      /* spa_train_workspace_bytes()                                         */
  /* the paper's containers (Sec. 3.2 "Token Packing") */
  int32_t container_len;      /* L > 0: spa_block_fwd fills seg_offsets (which must then be a writable
                                 int32[spa_container_max_segments(p, L) + 1]) with the container cuts of the
                                 selection it has just packed and both passes use them; n_seg is ignored */
} spa_block_buffers;

/* A non-blocking stream and two events on the current device (host-side objects, no device memory).  Create one
 * per block that runs concurrently; destroy it when no work that uses it is in flight. */
int spa_overlap_create(spa_overlap** out);
int spa_overlap_destroy(spa_overlap* ov);

/* Forward pass of one block: y = x on unselected tokens, the projected attention output (plus x under
 * SPA_FLAG_RESIDUAL) on selected ones. */
int spa_block_fwd(const spa_params* p, const spa_block_buffers* b, void* stream);

/* Backward pass for the last spa_block_fwd on the same buffers: dX, dW_qkv, db_qkv, dW_o, db_o (and, when
 * `trainable`, ds, ds_up, dw_g, db_g, loss).  When it returns, every piece of work it enqueued, on either stream,
 * is ordered before whatever is enqueued on `stream` next. */
int spa_block_bwd(const spa_params* p, const spa_block_buffers* b, void* stream);

/* ---- Diagnostics (the paper has no counterpart) ----------------------------------------------------------------
 * spa_probe_exp2: n_ctas CTAs of 512 threads evaluate base-2 exponentials with the instruction the softmax kernels
 * use, 8 * iters per thread; *n_exp (host, may be NULL) receives the total count.  Timed by the caller, it gives the
 * exponential throughput that bounds attention at head dimension 32 (Eq. 9's 2L^2C term costs one exponential per
 * 4d flops).  sink: float[n_ctas], never written in practice.
 * spa_probe_wait_expiry: one warp waits on a barrier that nobody arrives at and gives up after `limit` polls
 * (<= 2^20): d_status receives SPA_ERR_TIMEOUT and *polls_done (device int32, may be NULL) the polls made.  Shows,
 * without any fault or hang, what every bounded wait of the kernels does when it runs out.
 * spa_probe_mma_issue: one CTA issues 32 back-to-back tensor-core products of a shape the attention kernels use
 * (M = 128, K = 16, bf16, zeroed operands; variant 0: both operands in shared memory, N = 64; 1: A in TMEM, N = 64;
 * 2, 3: shared memory, N = 128, 256) and commits them to a barrier; elected = 0: lane 0 of a warp issues alone,
 * 1: all lanes of the warp run the loop and one elected lane issues.  cycles (device uint32[2]) receives the fastest
 * of 20 repetitions: [0] SM clocks from the first product to the commit, [1] until the barrier completes.  The probe
 * takes all 512 TMEM columns of its SM while it runs: call it with nothing else in flight.  Its wait is bounded
 * (SPA_ERR_TIMEOUT in d_status). */
int spa_probe_exp2(int32_t n_ctas, int32_t iters, float* sink, unsigned long long* n_exp, void* stream);
int spa_probe_wait_expiry(int32_t limit, int32_t* d_status, int32_t* polls_done, void* stream);
int spa_probe_mma_issue(int32_t variant, int32_t elected, uint32_t* cycles, int32_t* d_status, void* stream);

/* Blocking read of the device status word: synchronises `stream` and returns its value. */
int spa_read_status(const int32_t* d_status, void* stream);

/* Static text for a spa_status value. */
const char* spa_status_string(int status);

/* Text of the last CUDA error a call of this library met on the calling thread ("" if none). */
const char* spa_last_cuda_error(void);

/* Number of kernels this library has enqueued in this process so far (host-side tally, all
 * threads; used to report launches per step). */
unsigned long long spa_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SPA_H_ */
