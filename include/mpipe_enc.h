/*
 * libmpipe_enc -- the data-parallel computation that the Mpipe "transpose" schedule relocates,
 * written for NVIDIA B200 (sm_100a).
 *
 * Under the schedule <transpose, 1f1b> (Section 4.2, "Instantiation") the modality encoder is a
 * Replicated region: every pipeline rank runs whole encoder microbatches, Fwd(enc, r, m) inside its
 * warm-up bubble and -- only if the encoder is trainable -- Bwd(enc, r, m) in the cool-down; the
 * encoder output then crosses the Replicated->Sharded seam of Table 2 ("Gather") into the first LLM
 * stage.  This library provides the kernels of that region's attention and of the local half of the
 * seam, over packed variable-length image-patch sequences (Section 2: resolutions, clip lengths and
 * pure-text samples vary from microbatch to microbatch):
 *
 *   mpipe_seg_plan          patch counts -> cu_seqlens + longest-first tile work-lists   (host, integers)
 *   mpipe_varlen_attn_fwd   per-image softmax attention, O and (if trained) row LSE      (device)
 *   mpipe_varlen_attn_bwd   dQ, dK, dV; a no-op when the encoder is frozen               (device)
 *   mpipe_merge_tokens      encoder tokens -> their placeholder rows of the LLM input    (device)
 *   mpipe_merge_tokens_bwd  gradient rows at the placeholders -> encoder; no-op if frozen (device)
 *
 * Conventions
 *   - Plain C ABI.  Every call returns an mpipe_status_t as int32_t; nothing throws or aborts.
 *   - "host" / "device" is stated for every pointer.  The caller owns all memory, the workspace and
 *     the CUDA stream; the library allocates no device memory.  Device calls enqueue work on `stream`
 *     (a cudaStream_t passed as void*, NULL = default stream) and return without synchronising.
 *     They may therefore be captured in a CUDA graph and replayed (per-kernel attributes are set on a
 *     kernel's first launch: make one plain call of each entry point before the capture).
 *   - Argument errors are detected on the host before anything is launched; outputs are untouched.
 *   - bf16 = bfloat16.  Token tensors are [tokens, heads, head_dim] with explicit token and head
 *     strides in ELEMENTS; head_dim is contiguous.  Base pointers must be 16-byte aligned and the
 *     strides multiples of 8 elements (TMA needs 16-byte aligned global strides).
 *   - `status_buf` (device int32[4], optional, zeroed by the caller) receives device-side findings:
 *     [0] = first non-zero mpipe_status_t seen by a kernel, [1] = detail (e.g. offending index),
 *     [2], [3] reserved.  Kernels never trap: a bounded wait that expires or an out-of-range index
 *     sets this word, skips the offending work and returns.
 *   - mode mirrors trainable(enc) of the paper's derive(): MPIPE_ENC_FROZEN deletes every optional
 *     backward event (Lemma 1 and the "same schedule, two footprints" paragraph of Section 4.2);
 *     the forward results are bit-identical in both modes (Corollary 1).
 */
#ifndef MPIPE_ENC_H_
#define MPIPE_ENC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    MPIPE_OK = 0,
    MPIPE_ERR_INVALID_ARG = 1, /* NULL / negative / misaligned / inconsistent argument            */
    MPIPE_ERR_UNSUPPORTED = 2, /* head_dim not in {64, 80}, tile_rows not a supported value       */
    MPIPE_ERR_WORKSPACE = 3,   /* workspace NULL or smaller than mpipe_attn_workspace_bytes()     */
    MPIPE_ERR_CUDA = 4,        /* a CUDA runtime / driver call failed (launch, tensor-map encode) */
    MPIPE_ERR_TIMEOUT = 5,     /* device: a bounded wait expired (reported through status_buf)    */
    MPIPE_ERR_INDEX = 6        /* device: merge position out of range (reported via status_buf)   */
} mpipe_status_t;

/* trainable(enc): the one model bit derive() reads for the encoder region (Section 4.2). */
typedef enum { MPIPE_ENC_FROZEN = 0, MPIPE_ENC_TRAINED = 1 } mpipe_enc_mode_t;

/* One tile of one segment.  Forward items tile the QUERY rows of a segment (rows = queries, kv_* =
 * the segment's whole key range); backward items tile the KEY/VALUE rows (rows = keys, kv_* = the
 * segment's whole query range, which is the same token range).  Heads are not listed: kernels
 * iterate item x head. */
typedef struct {
    int32_t seg;       /* segment (image / clip) index                      */
    int32_t tile;      /* tile index inside the segment                     */
    int32_t row_start; /* first packed row of the tile                      */
    int32_t row_len;   /* rows in the tile, 1..tile_rows                    */
    int32_t kv_start;  /* first packed row of the segment (= cu_seqlens[seg]) */
    int32_t kv_len;    /* tokens in the segment                             */
} mpipe_work_item_t;

/* Native tile heights of the kernels in this build (rows per work item). */
int32_t mpipe_fwd_tile_rows(void);
int32_t mpipe_bwd_tile_rows(void);

/*
 * (1) Segment planner -- host, integer only.  Not in the paper beyond the observation that the
 * encoder's work is known before the LLM pipeline starts (Section 1) and that the static schedule
 * has no run-time scheduling cost; it has to cost microseconds.
 *
 *   cu_seqlens[0] = 0, cu_seqlens[i+1] = cu_seqlens[i] + patch_counts[i];  *total_tokens = cu[n_seg];
 *   *max_seqlen = max patch count (0 if none).
 *   Items: segments ordered by patch count descending, ties by index ascending; empty segments
 *   (pure-text samples) are skipped; per segment tiles t = 0.. in order:
 *     { seg, t, cu[seg] + t*tile_rows, min(tile_rows, n - t*tile_rows), cu[seg], n }.
 *   Forward items use fwd_tile_rows, backward items bwd_tile_rows.  FROZEN => *n_bwd_items = 0.
 *
 * Two-call pattern: with fwd_items == NULL (resp. bwd_items == NULL) only the counts are written.
 * All pointers are HOST pointers.  cu_seqlens has room for n_seg + 1 entries.  patch_counts may be
 * NULL iff n_seg == 0.  Errors: negative count or n_seg, total >= 2^31, tile_rows <= 0, NULL outputs
 * -> MPIPE_ERR_INVALID_ARG.
 */
int32_t mpipe_seg_plan(const int32_t* patch_counts, int32_t n_seg, int32_t fwd_tile_rows, int32_t bwd_tile_rows,
                       int32_t mode, int32_t* cu_seqlens, int32_t* total_tokens, int32_t* max_seqlen,
                       mpipe_work_item_t* fwd_items, int32_t* n_fwd_items, mpipe_work_item_t* bwd_items,
                       int32_t* n_bwd_items);

/* Bytes of device workspace mpipe_varlen_attn_bwd needs (0 when FROZEN): an fp32 dQ accumulator
 * [tokens, heads, head_dim] and the fp32 row terms Delta [heads, tokens], each rounded up to 256 B. */
size_t mpipe_attn_workspace_bytes(int32_t total_tokens, int32_t n_heads, int32_t head_dim, int32_t mode);

/*
 * (2) Fwd(enc) attention (the relocated forward event of Section 4.2).  For every segment s with
 * packed rows [a, b) = [cu[s], cu[s+1]) and every head h, with S = softmax_scale * Q K^T restricted
 * to the segment (bidirectional, no mask inside it, nothing across segments):
 *     O[i,h,:] = sum_j softmax_j(S_ij) V[j,h,:],     LSE[h,i] = ln sum_j exp(S_ij).
 *
 *   q, k, v   device, bf16 [total_tokens, n_heads, head_dim], strides tok_stride_qkv / head_stride_qkv
 *   o         device, bf16, same shape, strides tok_stride_o / head_stride_o              (output)
 *   lse       device, fp32 [n_heads, total_tokens] contiguous; written only when TRAINED (required
 *             then); ignored when FROZEN                                                  (output)
 *   cu_seqlens_dev   device int32[n_seg + 1]   (copy of the plan; the kernels take every range from the
 *                    items, which carry the same boundaries, and do not read it)
 *   fwd_items_dev    device mpipe_work_item_t[n_fwd_items] from mpipe_seg_plan with
 *                    fwd_tile_rows = mpipe_fwd_tile_rows().  The host cannot inspect device memory at
 *                    launch time, so the kernel checks the whole list before it does anything else:
 *                    every item's row range and key range must be non-empty and lie inside
 *                    [0, total_tokens), the row range at most one tile.  If one does not (a plan made
 *                    for another total_tokens, a corrupted buffer) the plan is rejected as a whole:
 *                    status_buf[0] = MPIPE_ERR_INDEX, status_buf[1] = the index of a bad item, and the
 *                    kernel returns without reading or writing any tensor.
 *   total_tokens == 0 or n_fwd_items == 0: returns MPIPE_OK without launching.
 * Rows past a segment's end inside a tile are computed but never stored.  fp32 accumulation,
 * bf16 probabilities; results are deterministic run to run.
 */
int32_t mpipe_varlen_attn_fwd(const void* q, const void* k, const void* v, void* o, float* lse,
                              int64_t tok_stride_qkv, int64_t head_stride_qkv, int64_t tok_stride_o,
                              int64_t head_stride_o, const int32_t* cu_seqlens_dev, int32_t n_seg,
                              int32_t total_tokens, int32_t max_seqlen, const mpipe_work_item_t* fwd_items_dev,
                              int32_t n_fwd_items, int32_t n_heads, int32_t head_dim, float softmax_scale,
                              int32_t mode, int32_t* status_buf, void* stream);

/*
 * (3) Bwd(enc)? attention -- exists only when trainable(enc) (Lemma 1).  FROZEN: returns MPIPE_OK at
 * once, launches nothing, touches nothing.  TRAINED, per segment and head, with P = exp(S - LSE):
 *     Delta_i = sum_d dO[i,d] O[i,d];  dV = P^T dO;  dP = dO V^T;  dS = P o (dP - Delta);
 *     dQ = softmax_scale * dS K;       dK = softmax_scale * dS^T Q.
 *
 *   dout, o   device bf16 (o strides);  q, k, v device bf16 (qkv strides);  lse device fp32 [H, T]
 *   dq, dk, dv device bf16, strides tok_stride_grad / head_stride_grad                    (outputs)
 *   bwd_items_dev  from mpipe_seg_plan with bwd_tile_rows = mpipe_bwd_tile_rows()
 *   workspace      device, >= mpipe_attn_workspace_bytes(...), 256-byte aligned; contents are scratch
 *                  (fp32 dQ accumulator + Delta).  The alignment is a requirement of the TMA tensor map
 *                  through which the accumulator is updated.
 *   The item list is checked on the device exactly as in the forward (MPIPE_ERR_INDEX); a rejected plan leaves dk
 *   and dv untouched and dq all zeros (its accumulator is cleared and converted independently of the plan).
 * dQ is summed over key tiles in fp32 by the copy engine (TMA reduce-add from shared memory); the order
 * of those additions is not fixed, so the low bits of dQ may differ from run to run.  dK and dV are
 * reproducible at head_dim 64.
 */
int32_t mpipe_varlen_attn_bwd(const void* dout, const void* q, const void* k, const void* v, const void* o,
                              const float* lse, void* dq, void* dk, void* dv, int64_t tok_stride_qkv,
                              int64_t head_stride_qkv, int64_t tok_stride_o, int64_t head_stride_o,
                              int64_t tok_stride_grad, int64_t head_stride_grad, const int32_t* cu_seqlens_dev,
                              int32_t n_seg, int32_t total_tokens, int32_t max_seqlen,
                              const mpipe_work_item_t* bwd_items_dev, int32_t n_bwd_items, int32_t n_heads,
                              int32_t head_dim, float softmax_scale, int32_t mode, void* workspace,
                              size_t workspace_bytes, int32_t* status_buf, void* stream);

/*
 * The same backward for callers that are not allowed to allocate device memory.  (The paper has no
 * counterpart: it never discusses where kernel scratch comes from.)
 *
 * Who needs it: a pipeline runtime that hands out all device memory from a plan fixed before the
 * step and exposes no allocator to the code it runs in the bubbles; a host process whose device
 * memory belongs to another component's pool; a latency-critical loop in which cudaMalloc is
 * banned because it synchronises the whole device.  Such callers cannot produce the `workspace` of
 * mpipe_varlen_attn_bwd, so this variant keeps the scratch (fp32 dQ accumulator + Delta) inside the
 * library, in a fixed 32 MiB device array (mpipe_attn_bwd_static_scratch_bytes()).  Every GPU that
 * loads the library holds those 32 MiB until the process exits, used or not.
 *
 *   - Arguments, layouts, results and error behaviour are those of mpipe_varlen_attn_bwd, minus
 *     workspace / workspace_bytes.  Inputs and outputs are still the caller's buffers.
 *   - Limit: mpipe_attn_workspace_bytes(total_tokens, n_heads, head_dim, TRAINED) must not exceed
 *     the 32 MiB (e.g. 8000 tokens x 16 heads x 64).  Larger problems are refused with
 *     MPIPE_ERR_WORKSPACE before anything is launched; use mpipe_varlen_attn_bwd for them.
 *   - The call itself allocates nothing (no cudaMalloc / cudaFree, no allocating library routine).
 *     The first call on each device looks up the array's device address once, with that device
 *     current; make that first call before starting any stream capture.  A failed look-up returns
 *     MPIPE_ERR_CUDA.  With lazy module loading the CUDA runtime materialises the library's device
 *     code, this array included, when the first kernel of the library is used, and that first look-up
 *     may synchronise the device: do one warm-up call at start-up if neither is acceptable later.
 *     The per-device address cache is plain host memory: first calls on one device from several host
 *     threads at once are harmless (they store the same value) but are not ordered.
 *   - Argument errors are reported exactly as by mpipe_varlen_attn_bwd (the same checks run first);
 *     only then is the size compared with the limit.
 *   - All calls on a device share the one array, which keeps whatever the previous call left in
 *     it.  Nothing needs to be cleared by the caller: each call's first kernel zeroes the
 *     accumulator and rewrites Delta for its own problem.  Because the array is shared, two calls
 *     whose kernels may overlap on the GPU (different streams, no dependency between them) race on
 *     it and produce garbage: serialise them.
 */
size_t mpipe_attn_bwd_static_scratch_bytes(void);
int32_t mpipe_varlen_attn_bwd_static(const void* dout, const void* q, const void* k, const void* v, const void* o,
                                     const float* lse, void* dq, void* dk, void* dv, int64_t tok_stride_qkv,
                                     int64_t head_stride_qkv, int64_t tok_stride_o, int64_t head_stride_o,
                                     int64_t tok_stride_grad, int64_t head_stride_grad,
                                     const int32_t* cu_seqlens_dev, int32_t n_seg, int32_t total_tokens,
                                     int32_t max_seqlen, const mpipe_work_item_t* bwd_items_dev, int32_t n_bwd_items,
                                     int32_t n_heads, int32_t head_dim, float softmax_scale, int32_t mode,
                                     int32_t* status_buf, void* stream);

/*
 * (4) Local half of Coll(Gather, (enc, llm), m), the Replicated->Sharded seam of Table 2: encoder
 * token i is written over row positions[i] of the LLM input-embedding buffer, in place:
 *     llm_embeds[positions[i], 0:hidden] = enc_tokens[i, 0:hidden].
 * The forward seam is not gated by trainability, so `mode` is accepted and ignored.
 *
 *   enc_tokens  device bf16 [n_enc_tokens, hidden], row stride enc_row_stride elements
 *   llm_embeds  device bf16 [n_llm_tokens, hidden], row stride emb_row_stride elements   (in/out)
 *   positions_dev device int32[n_enc_tokens]; must be unique (precondition; see
 *               mpipe_validate_positions).  An index outside [0, n_llm_tokens) is skipped and
 *               reported as MPIPE_ERR_INDEX in status_buf.
 *   hidden must be a multiple of 8 and both buffers 16-byte aligned with strides multiples of 8.
 *   n_enc_tokens == 0: MPIPE_OK, nothing launched.
 */
int32_t mpipe_merge_tokens(const void* enc_tokens, int64_t enc_row_stride, void* llm_embeds, int64_t emb_row_stride,
                           const int32_t* positions_dev, int32_t n_enc_tokens, int32_t n_llm_tokens, int32_t hidden,
                           int32_t mode, int32_t* status_buf, void* stream);

/*
 * Local half of the reverse seam Coll(Scatter, (enc, llm), m)?, which fires only when some region
 * before the LLM is trainable (Lemma 1, gate (i)):  d_enc[i, :] = d_llm_embeds[positions[i], :].
 * FROZEN: returns MPIPE_OK at once and touches nothing.  Same layout rules as mpipe_merge_tokens;
 * d_enc is the output.
 */
int32_t mpipe_merge_tokens_bwd(const void* d_llm_embeds, int64_t emb_row_stride, void* d_enc, int64_t enc_row_stride,
                               const int32_t* positions_dev, int32_t n_enc_tokens, int32_t n_llm_tokens,
                               int32_t hidden, int32_t mode, int32_t* status_buf, void* stream);

/* Host helper: checks that HOST positions[0..n) are unique and inside [0, n_llm_tokens).
 * Returns MPIPE_OK, MPIPE_ERR_INDEX (out of range) or MPIPE_ERR_INVALID_ARG (duplicate / NULL). */
int32_t mpipe_validate_positions(const int32_t* positions, int32_t n, int32_t n_llm_tokens);

/*
 * The rest of the packed encoder layer -- what one Fwd(enc, r, m) event of the transpose schedule executes
 * besides attention (Section 4.2; the paper says only "ViT-style encoder", Section 2: the block below is the
 * pre-norm Transformer block of that family).  The forward is the whole layer of a FROZEN encoder (Lemma 1: no
 * backward events exist then); for a TRAINED one it also writes the LSE, and mpipe_encoder_layer_bwd below is its
 * backward.
 *
 *   mpipe_linear_fwd     C[M, N] = act(A[M, K] W[N, K]^T + bias[N]) + residual[M, N]; all bf16, device, row-major
 *                        with row strides lda / ldw / ldr / ldc in elements (multiples of 8, bases 16-byte
 *                        aligned), fp32 accumulation on the tensor cores, act = GELU (u Phi(u), erf form) when
 *                        flags has MPIPE_LINEAR_GELU, identity otherwise; bias and residual may be NULL.
 *                        N and K multiples of 8 (MPIPE_ERR_UNSUPPORTED otherwise); M == 0 launches nothing.
 *   mpipe_layernorm_fwd  y[t, :] = (x[t, :] - mean_t) * rsqrt(var_t + eps) * gamma + beta, biased variance, fp32
 *                        statistics; bf16 in and out, hidden a multiple of 8 and <= 2048.
 *   mpipe_rope_apply     rotary position encoding, rotate-half form, in place on q and k of a packed projection:
 *                        for each token t, head h and pair j < head_dim/2:
 *                          (x[j], x[j + head_dim/2]) <- (x[j] cos[t,j] - x[j+hd/2] sin[t,j], x[j+hd/2] cos[t,j] + x[j] sin[t,j]).
 *                        qk: bf16 device, q of token t at qk + t*tok_stride, its k at + k_offset, heads contiguous
 *                        (head stride = head_dim); cos/sin: fp32 device [n_tokens, head_dim/2] -- the caller builds
 *                        them (1-D, or 2-D with one half of the pairs per image axis); head_dim a multiple of 16.
 *                        The paper does not name a position encoding; this is the one the Qwen2-VL-like
 *                        configuration implies.  fp32 arithmetic, one rounding to bf16.
 *   mpipe_encoder_layer_fwd
 *        a = LN(x; ln1) ; qkv = a Wqkv^T + bqkv (columns q | k | v, each [n_heads][head_dim]) ;
 *        q, k <- rope(q, k) when rope_cos / rope_sin are given (both NULL: none) ;
 *        o = per-image softmax attention (mpipe_varlen_attn_fwd on strided views of qkv, same plan arguments) ;
 *        x1 = x + o Wo^T + bo ; m = LN(x1; ln2) ; y = x1 + GELU(m W1^T + b1) W2^T + b2.
 *        x, y: bf16 [n_tokens, hidden] contiguous, device; y may not alias x.  Weights: device bf16, nn.Linear
 *        layout [out, in], contiguous.  lse: fp32 [n_heads, n_tokens] when TRAINED, ignored when FROZEN.
 *        workspace: device, 256-byte aligned, >= mpipe_encoder_layer_workspace_bytes (MPIPE_ERR_WORKSPACE);
 *        caller-owned; after a TRAINED call it holds what mpipe_encoder_layer_bwd reads (see there), otherwise its contents are
 *        undefined afterwards.  In both modes the activation is applied to the fp32 accumulator of the fc1 projection;
 *        the TRAINED forward stores the pre-activation (bf16) from the same accumulator in the same launch, so y is
 *        bit-identical in the two modes (Corollary 1: freezing changes nothing in the forward).  Seven launches (eight
 *        with rope) on `stream`, no allocation, no sync.
 *        head_dim = hidden / n_heads must be one the attention kernels support (64, 80).
 * Device-side findings (a bounded wait that ran out) are reported through status_buf as for the attention calls.
 */
#define MPIPE_LINEAR_GELU 1

typedef struct {
    const void *ln1_gamma, *ln1_beta;   /* [hidden] */
    const void *w_qkv, *b_qkv;          /* [3*hidden, hidden], [3*hidden] */
    const void *w_o, *b_o;              /* [hidden, hidden], [hidden] */
    const void *ln2_gamma, *ln2_beta;   /* [hidden] */
    const void *w_fc1, *b_fc1;          /* [ffn, hidden], [ffn] */
    const void *w_fc2, *b_fc2;          /* [hidden, ffn], [hidden] */
} mpipe_layer_weights_t;

int32_t mpipe_linear_fwd(const void* a, const void* w, const void* bias, const void* residual, void* c, int32_t M,
                         int32_t N, int32_t K, int64_t lda, int64_t ldw, int64_t ldr, int64_t ldc, int32_t flags,
                         int32_t* status_buf, void* stream);
/* Input gradient of a projection y = x W^T (W [N, K]):  dx[M, K] = (dy[M, N] W[N, K]) o GELU'(gelu_input[M, K]) + residual[M, K].
 * gelu_input (the pre-activation u of the layer in front, whose output x = GELU(u) fed this projection) and residual
 * may be NULL; GELU'(u) = Phi(u) + u phi(u).  Same layout, alignment and error rules as mpipe_linear_fwd; W is read
 * as stored (no transposed copy). */
int32_t mpipe_linear_dgrad(const void* dy, const void* w, const void* gelu_input, const void* residual, void* dx, int32_t M,
                           int32_t N, int32_t K, int64_t lddy, int64_t ldw, int64_t ldu, int64_t ldr, int64_t lddx,
                           int32_t* status_buf, void* stream);
/* Weight gradient of a projection y = x W^T:  dw[N, K] += dy[n_tokens, N]^T x[n_tokens, K], accumulated in fp32 into the
 * caller's gradient buffer (fp32 device [N, lddw], lddw a multiple of 4; the caller zeroes it at the start of a step
 * and every microbatch adds to it).  dy, x: bf16 device, row strides multiples of 8, bases 16-byte aligned; N, K
 * multiples of 8.  The token range is split over CTAs and partial tiles are added with TMA reductions, so the
 * summation order (and the last bits) can differ from run to run. */
int32_t mpipe_linear_wgrad(const void* dy, const void* x, float* dw, int32_t n_tokens, int32_t N, int32_t K, int64_t lddy,
                           int64_t ldx, int64_t lddw, int32_t* status_buf, void* stream);
int32_t mpipe_layernorm_fwd(const void* x, const void* gamma, const void* beta, void* y, int32_t n_tokens,
                            int32_t hidden, int64_t ldx, int64_t ldy, float eps, void* stream);
int32_t mpipe_rope_apply(void* qk, int64_t tok_stride, int64_t k_offset, const float* cos_table, const float* sin_table,
                         int32_t n_tokens, int32_t n_heads, int32_t head_dim, void* stream);
/* Backward pieces of the layer (exist only for a trainable encoder, Lemma 1):
 *   mpipe_rope_apply_bwd     the transpose of mpipe_rope_apply (rotation by the opposite angles), in place on dq, dk.
 *   mpipe_layernorm_bwd      with xhat = (x - mean) rstd and g = dy * gamma:
 *                              dx = rstd * (g - mean(g) - xhat * mean(g * xhat)) + dres      (dres may be NULL)
 *                              dgamma[j] += sum_t dy[t,j] xhat[t,j],  dbeta[j] += sum_t dy[t,j]   (fp32, accumulated)
 *                            x, dy, dres, dx: bf16 [n_tokens, hidden]; mean / rstd are recomputed from x.
 *   mpipe_colsum_accumulate  out[j] += sum_t a[t, j] in fp32: the bias gradient of a projection from its dy.
 * The fp32 accumulations use atomics: their last bits can differ from run to run. */
int32_t mpipe_rope_apply_bwd(void* dqk, int64_t tok_stride, int64_t k_offset, const float* cos_table, const float* sin_table,
                             int32_t n_tokens, int32_t n_heads, int32_t head_dim, void* stream);
int32_t mpipe_layernorm_bwd(const void* x, const void* dy, const void* gamma, const void* dres, void* dx, float* dgamma,
                            float* dbeta, int32_t n_tokens, int32_t hidden, int64_t ldx, int64_t lddy, int64_t ldr,
                            int64_t lddx, float eps, void* stream);
int32_t mpipe_colsum_accumulate(const void* a, float* out, int32_t n_tokens, int32_t n_cols, int64_t lda, void* stream);
/*
 * Bwd(enc, r, m) of the same layer -- exists only when the encoder is trainable (Lemma 1): with mode FROZEN the call
 * returns MPIPE_OK at once and touches nothing.  TRAINED: given dy = dL/dy it writes
 * dx = dL/dx (bf16 [n_tokens, hidden]) and ADDS the parameter gradients, in fp32, to the twelve buffers of `grads`
 * (same shapes as the weights; the caller zeroes them at the start of a step, every microbatch accumulates).
 * fwd_workspace is the workspace of the matching mpipe_encoder_layer_fwd call (TRAINED mode, same x, weights, plan and
 * rope tables), untouched since: it holds the rotated q | k | v, the attention output, x1, GELU(u) and (TRAINED forward
 * only) the MLP pre-activation u; its LN slot is overwritten here.  lse is that call's LSE.  The two LayerNorm outputs
 * are recomputed instead of being stored by the forward.  workspace: device, 256-byte aligned,
 * >= mpipe_encoder_layer_bwd_workspace_bytes.  About twenty launches on `stream`, nothing allocated.  bwd_items_dev /
 * n_bwd_items are the plan's backward list.  Sums over tokens use fp32 atomics and TMA reductions: parameter gradients
 * are reproducible to rounding order only.
 */
typedef struct {
    float *ln1_gamma, *ln1_beta, *w_qkv, *b_qkv, *w_o, *b_o, *ln2_gamma, *ln2_beta, *w_fc1, *b_fc1, *w_fc2, *b_fc2;
} mpipe_layer_grads_t;
size_t mpipe_encoder_layer_bwd_workspace_bytes(int32_t n_tokens, int32_t hidden, int32_t n_heads, int32_t ffn);
int32_t mpipe_encoder_layer_bwd(const void* dy, const void* x, void* dx, const mpipe_layer_weights_t* w,
                                const mpipe_layer_grads_t* grads, int32_t n_tokens, int32_t hidden, int32_t n_heads,
                                int32_t ffn, const int32_t* cu_seqlens_dev, int32_t n_seg, int32_t max_seqlen,
                                const mpipe_work_item_t* bwd_items_dev, int32_t n_bwd_items, float softmax_scale,
                                float ln_eps, const float* rope_cos, const float* rope_sin, int32_t mode,
                                const float* lse, void* fwd_workspace, void* workspace, size_t workspace_bytes,
                                int32_t* status_buf, void* stream);
/*
 * The whole encoder: n_layers blocks of the same shape applied in turn -- what one Fwd(enc, r, m) / Bwd(enc, r, m)
 * event executes.  layers / grads: host arrays of n_layers structs.  lse: fp32 [n_layers, n_heads, n_tokens] when
 * TRAINED.  mpipe_encoder_fwd's workspace (mpipe_encoder_workspace_bytes): FROZEN, one layer's workspace and two
 * activation buffers, reused; TRAINED, every layer's workspace and input, kept for mpipe_encoder_bwd, which takes
 * it as fwd_workspace (untouched) plus a workspace of its own (mpipe_encoder_bwd_workspace_bytes).  The rope tables
 * and the plan are shared by all layers.  FROZEN: mpipe_encoder_bwd returns MPIPE_OK at once.
 */
size_t mpipe_encoder_workspace_bytes(int32_t n_layers, int32_t n_tokens, int32_t hidden, int32_t ffn, int32_t mode);
size_t mpipe_encoder_bwd_workspace_bytes(int32_t n_tokens, int32_t hidden, int32_t n_heads, int32_t ffn);
int32_t mpipe_encoder_fwd(const void* x, void* y, const mpipe_layer_weights_t* layers, int32_t n_layers, int32_t n_tokens,
                          int32_t hidden, int32_t n_heads, int32_t ffn, const int32_t* cu_seqlens_dev, int32_t n_seg,
                          int32_t max_seqlen, const mpipe_work_item_t* fwd_items_dev, int32_t n_fwd_items,
                          float softmax_scale, float ln_eps, const float* rope_cos, const float* rope_sin, int32_t mode,
                          float* lse, void* workspace, size_t workspace_bytes, int32_t* status_buf, void* stream);
int32_t mpipe_encoder_bwd(const void* dy, const void* x, void* dx, const mpipe_layer_weights_t* layers,
                          const mpipe_layer_grads_t* grads, int32_t n_layers, int32_t n_tokens, int32_t hidden,
                          int32_t n_heads, int32_t ffn, const int32_t* cu_seqlens_dev, int32_t n_seg, int32_t max_seqlen,
                          const mpipe_work_item_t* bwd_items_dev, int32_t n_bwd_items, float softmax_scale, float ln_eps,
                          const float* rope_cos, const float* rope_sin, int32_t mode, const float* lse,
                          void* fwd_workspace, void* workspace, size_t workspace_bytes, int32_t* status_buf,
                          void* stream);
size_t mpipe_encoder_layer_workspace_bytes(int32_t n_tokens, int32_t hidden, int32_t ffn);
int32_t mpipe_encoder_layer_fwd(const void* x, void* y, const mpipe_layer_weights_t* w, int32_t n_tokens,
                                int32_t hidden, int32_t n_heads, int32_t ffn, const int32_t* cu_seqlens_dev,
                                int32_t n_seg, int32_t max_seqlen, const mpipe_work_item_t* fwd_items_dev,
                                int32_t n_fwd_items, float softmax_scale, float ln_eps, const float* rope_cos,
                                const float* rope_sin, int32_t mode, float* lse, void* workspace,
                                size_t workspace_bytes, int32_t* status_buf, void* stream);

/*
 * The Replicated -> Sharded seam across ranks (Table 2: Gather forward, Scatter backward).  The encoder output of
 * microbatch m is produced on ByMicrobatch(m); the LLM input sequence lives on the first pipeline stage.  The seam is
 * run as ONE kernel: mpipe_merge_tokens on the owner with `llm_embeds` pointing into the first stage's buffer through
 * a peer mapping (plain stores over NVLink), and mpipe_merge_tokens_bwd reading the gradient rows the same way.
 * These three host calls provide the mapping (CUDA IPC; the exporting allocation must come from cudaMalloc and stay
 * alive while mapped).  handle buffers are mpipe_ipc_handle_bytes() bytes of host memory.  An opened pointer is valid
 * in the opening process only and must be closed there.  Ordering between ranks (the first stage may read the rows
 * only after the owner's kernel has completed) is the caller's: a stream synchronisation on the owner followed by any
 * host-level message.  MPIPE_ERR_CUDA when the runtime refuses (e.g. same process as the exporter).
 */
int32_t mpipe_ipc_handle_bytes(void);
int32_t mpipe_ipc_export(const void* dev_ptr, void* handle_out);
int32_t mpipe_ipc_open(const void* handle, void** dev_ptr_out);
int32_t mpipe_ipc_close(void* dev_ptr);

/*
 * derive : cut x schedule x model -> placement x collectives x order  (Section 4.1, "Schedule Algebra") -- host only.
 *
 * A model of n_layers layers is cut into k contiguous regions by k-1 interior boundaries cut[0] < ... < cut[k-2]
 * in (0, n_layers); skeletons[j] in {1f1b, gpipe, transpose} is region j+1's skeleton and trainable[j] its
 * trainable bit.  layout(transpose) = Replicated, layout(1f1b) = layout(gpipe) = Sharded.  Regions, microbatches
 * and events' `mb` are 1-based as in the paper; ranks are 0-based.
 *
 *   mpipe_schedule_valid      MPIPE_OK iff the cut tiles the model and no two adjacent regions are Replicated
 *                             (normal form), MPIPE_ERR_INVALID_ARG otherwise.
 *   mpipe_schedule_normalize  collapses runs of adjacent transpose regions into one (their seam is the identity):
 *                             <transpose, transpose> -> <transpose>.  out_skeletons[k], out_cut[k-1], *out_k.
 *   mpipe_stage_index         rank + (region - 1) * n_ranks.
 *   mpipe_derive              for a VALID schedule:
 *     regions[k]      layout, first layer, layer count, skeleton of each region (placement);
 *     slabs[k][P][2]  the owner's table: Sharded = ByLayer, contiguous slabs (first layer, count), the remainder of
 *                     count / P going to the first ranks; Replicated = the whole region on every rank, with
 *                     ByMicrobatch given by owner[mb-1] (NULL: (mb-1) mod P);
 *     seams[k-1]      Table 2: forward comm of (j, j+1) from the layout pair, backward comm present (else
 *                     MPIPE_COMM_NONE) iff some region <= j is trainable (Lemma 1 (ii) at j = (i) at j+1);
 *     reduces         (region, group) of every trainable region: ReplicaGroup if Replicated, DataGroup if Sharded;
 *     events / edges  the order graph.  Per microbatch: Fwd(j, r, m) on every rank of a Sharded region (r = 0..P-1 in
 *                     turn) or on owner(m) for a Replicated one; Coll(fwd comm, seam j, m) between regions, placed
 *                     on the receiving rank; Loss(m) on the last rank of the last region; Bwd(j, r, m) for every
 *                     region with some trainable region <= j, in reverse; Coll(bwd comm, seam j-1, m) iff some region
 *                     < j is trainable.  Then one DpReduce per entry of `reduces` and one StepBarrier (rank -1).
 *                     Edges: Activation along the forward chain and from each Fwd to its own Bwd (the saved
 *                     activation), Turnaround Loss -> first Bwd, Gradient along the backward chain, Accumulate
 *                     Bwd -> DpReduce, Sequence DpReduce -> StepBarrier (Loss -> StepBarrier when nothing is
 *                     trainable), Sequence for the skeleton's order inside a stage (1f1b: as many forwards as there are
 *                     stages downstream -- P-1-r in the region, P per later Sharded and 1 per later Replicated
 *                     region --, then forward/backward pairs, then backwards; gpipe: forwards then backwards in reverse; transpose:
 *                     forwards then backwards by microbatch) and between neighbours of nodes(r);
 *     node_order / node_offsets[P+1]   nodes(r): rank r's events in execution order, from unit-cost list scheduling
 *                     in which a rank prefers (0) forwards of a Replicated region ahead of the first Sharded region
 *                     (the warm-up bubble), (1) Sharded-region events, collectives and losses, (2) other
 *                     Replicated-region events (cool-down); ties by event index.  The paper's figure for this is
 *                     missing; this is the reading taken.
 *     Capacities: events_cap / edges_cap entries; when too small the counts are still written and
 *     MPIPE_ERR_WORKSPACE is returned.  MPIPE_ERR_INVALID_ARG for an invalid schedule or a Sharded region with
 *     fewer layers than ranks; MPIPE_ERR_INDEX for an owner outside [0, P).
 *   mpipe_order_makespan      Section 4.3: with cost[e] >= 0 per event, T = longest path of the graph (each rank's
 *                             events follow nodes(r) through the Sequence edges), start[e] the earliest start times,
 *                             bubble[r] = T - sum of the costs of rank r's events.  start and bubble may be NULL.
 */
enum { MPIPE_SK_1F1B = 0, MPIPE_SK_GPIPE = 1, MPIPE_SK_TRANSPOSE = 2 };
enum { MPIPE_LAYOUT_SHARDED = 0, MPIPE_LAYOUT_REPLICATED = 1 };
enum { MPIPE_COMM_NONE = 0, MPIPE_COMM_GATHER = 1, MPIPE_COMM_SCATTER = 2, MPIPE_COMM_SEND = 3, MPIPE_COMM_RECVGRAD = 4 };
enum { MPIPE_GROUP_REPLICA = 0, MPIPE_GROUP_DATA = 1 };
enum { MPIPE_EV_FWD = 0, MPIPE_EV_BWD = 1, MPIPE_EV_COLL = 2, MPIPE_EV_DPREDUCE = 3, MPIPE_EV_LOSS = 4, MPIPE_EV_STEPBARRIER = 5 };
enum { MPIPE_EDGE_ACTIVATION = 0, MPIPE_EDGE_GRADIENT = 1, MPIPE_EDGE_TURNAROUND = 2, MPIPE_EDGE_ACCUMULATE = 3, MPIPE_EDGE_SEQUENCE = 4 };

typedef struct { int32_t layout, first_layer, n_layers, skeleton; } mpipe_region_t;
typedef struct { int32_t left_region, fwd_comm, bwd_comm; } mpipe_seam_t;          /* seam (left_region, left_region + 1) */
typedef struct { int32_t region, group; } mpipe_reduce_t;
/* kind; region (Coll: the seam's left region; StepBarrier: 0); rank (-1: all ranks); mb (0: none); comm (Coll only); group (DpReduce only, else -1) */
typedef struct { int32_t kind, region, rank, mb, comm, group; } mpipe_event_t;
typedef struct { int32_t src, dst, type; } mpipe_edge_t;

int32_t mpipe_stage_index(int32_t rank, int32_t region, int32_t n_ranks);
int32_t mpipe_schedule_valid(const int32_t* skeletons, const int32_t* cut, int32_t k, int32_t n_layers);
int32_t mpipe_schedule_normalize(const int32_t* skeletons, const int32_t* cut, int32_t k, int32_t n_layers,
                                 int32_t* out_skeletons, int32_t* out_cut, int32_t* out_k);
int32_t mpipe_derive(const int32_t* skeletons, const int32_t* cut, int32_t k, int32_t n_layers, const int32_t* trainable,
                     int32_t n_ranks, int32_t n_microbatches, const int32_t* owner, mpipe_region_t* regions,
                     int32_t* slabs, mpipe_seam_t* seams, mpipe_reduce_t* reduces, int32_t* n_reduces,
                     mpipe_event_t* events, int32_t events_cap, int32_t* n_events, mpipe_edge_t* edges,
                     int32_t edges_cap, int32_t* n_edges, int32_t* node_order, int32_t* node_offsets);
int32_t mpipe_order_makespan(const mpipe_event_t* events, int32_t n_events, const mpipe_edge_t* edges, int32_t n_edges,
                             const double* cost, int32_t n_ranks, double* makespan, double* start, double* bubble);

/*
 * Measurement aid (no counterpart in the paper; its cost model weights each compute event with one
 * duration, Section 4.3, and this is how a benchmark reads that duration for one kernel): while set,
 * the launch of kernel `which` (0 = attention forward, 1 = attention backward main kernel, 2 = merge
 * / merge_bwd, 3 = mpipe_linear_fwd, 4 = mpipe_layernorm_fwd) records the two cudaEvent_t handles on the call's stream directly before and after
 * it.  NULL handles switch it off.  The setting is per host thread (thread-local): it affects only the
 * launches the setting thread makes afterwards, so the library keeps no state shared between callers.
 * Returns MPIPE_ERR_INVALID_ARG for an unknown `which`.
 */
int32_t mpipe_set_profile_events(int32_t which, void* start_event, void* stop_event);

/*
 * Cost model of the transpose schedule (Section 4.3) -- host, double arithmetic, nothing on the device.
 *
 *   mpipe_event_cost         cost(Fwd) = cost(Bwd) = max(W / F, D / B): W FLOPs at peak rate F, D bytes of
 *                            HBM traffic at bandwidth B (the roofline of one compute event).
 *   mpipe_coll_cost          cost(Coll) = cost(DpReduce) = alpha + beta * n for an n-byte payload.
 *   mpipe_encoder_attn_work  W and D of this library's attention events for one encoder microbatch:
 *                            forward 4*H*D*sum n_i^2 FLOPs and sum n_i * H * (8*D [+4 LSE if trained]) bytes;
 *                            backward (trained only, else 0) 10*H*D*sum n_i^2 FLOPs and
 *                            sum n_i * H * (16*D + 16) bytes.
 *   mpipe_warmup_slack_1f1b  w_r, the idle time of pipeline rank r before its first LLM forward under
 *                            1F1B: r * (stage_fwd_cost + seam_cost).  (The paper's figure is missing; this
 *                            is the reading "rank r waits for r upstream stage forwards and their sends".)
 *   mpipe_owner_map          the ByMicrobatch owner: microbatches in order of decreasing encoder cost (ties:
 *                            lower index first), each to the rank with the most warm-up slack left,
 *                            w_r - E_r (ties: lower rank) -- "heavier encodes to longer warm-up slots".
 *                            Outputs owner[m], E_r = sum of the costs a rank received,
 *                            spill_r = max(0, E_r - w_r) and max_r spill_r, the time the encoder adds to
 *                            the step.
 * All pointers are HOST pointers.  Negative or NaN inputs, non-positive peaks or rank counts and NULL
 * outputs give MPIPE_ERR_INVALID_ARG.
 */
int32_t mpipe_event_cost(double flops, double bytes, double peak_flops, double peak_bw, double* cost);
int32_t mpipe_coll_cost(double alpha, double beta, double payload_bytes, double* cost);
int32_t mpipe_encoder_attn_work(const int32_t* patch_counts, int32_t n_seg, int32_t n_heads, int32_t head_dim,
                                int32_t mode, double* fwd_flops, double* fwd_bytes, double* bwd_flops,
                                double* bwd_bytes);
int32_t mpipe_warmup_slack_1f1b(int32_t n_ranks, double stage_fwd_cost, double seam_cost, double* slack);
int32_t mpipe_owner_map(const double* enc_cost, int32_t n_microbatches, const double* warmup_slack, int32_t n_ranks,
                        int32_t* owner, double* enc_work, double* spill, double* max_spill);

/*
 * Self-test of the bounded waits (the kernel-level counterpart of the paper's argument that an acyclic
 * order graph cannot dead-lock, Section 4.2: here a wait that would never be satisfied must end by
 * itself).  Launches one small CTA that waits on a barrier nobody signals, with a budget of
 * `budget_cycles` SM clock ticks (1 .. 4e9); when the budget runs out the kernel writes
 * MPIPE_ERR_TIMEOUT to status_buf[0] (device int32[4], required, zeroed by the caller) and returns
 * normally.  Nothing traps or faults and the CUDA context stays usable.  Enqueues on `stream`.
 */
int32_t mpipe_selftest_wait_timeout(int64_t budget_cycles, int32_t* status_buf, void* stream);

const char* mpipe_status_str(int32_t status);
int32_t mpipe_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MPIPE_ENC_H_ */
