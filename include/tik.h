/* tik: bitwise-consistent causal GQA attention and token log-probability for B200 (sm_100a).
 *
 * C ABI.  Unless stated otherwise every data pointer is a DEVICE pointer owned by the
 * caller; the library borrows it until the work queued on `stream` (a cudaStream_t
 * passed as void*) has completed.  Calls are asynchronous, never synchronise and never
 * read device memory on the host.  After tik_create the library allocates no device
 * memory: scratch comes from the caller (`ws`, sized by tik_workspace_bytes).
 *
 * Layouts (bf16 unless noted, all contiguous):
 *   packed tokens    [tokens][heads][d]
 *   KV cache         [num_pages][Hkv][page_size][d], separate K and V pools.  Rows of a
 *                    page that lie beyond a sequence's context must hold finite values
 *                    (zero-initialise the pool): they are multiplied by weight 0.
 *   block table      int32 [S][max_blocks]: physical page of each logical page.
 *   cu_seqlens       int32 [S+1] exclusive prefix sums of per-sequence token counts.
 *
 * The promise (paper Sec. 4.1, Eq. 1; Sec. 3.2 "same query data and causal KV prefix"):
 * for a fixed tik_contract_id(), the output bits of an attention row depend only on that
 * row's query, the values of its causal K/V prefix, softmax_scale and d -- not on the
 * entry point (train forward, prefill, decode), batch size or slot, packing order, page
 * size or placement, grid size or stream.  Likewise a log-probability depends only on
 * its hidden row, lm_head, target and inv_temperature, not on T or the row's index.
 *
 * Supported domain: d in {64,128}; page_size in {16,32,64,128}; Hq % Hkv == 0 and
 * Hq/Hkv <= 32; H % 64 == 0; all base pointers 16-byte aligned.  Anything else returns
 * TIK_ERR_UNSUPPORTED.  Nothing traps or aborts.
 */
#ifndef TIK_H
#define TIK_H
#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tik_ctx tik_ctx;   /* opaque, per device */
typedef int tik_status;

#define TIK_OK 0
#define TIK_ERR_INVALID_ARG (-1)   /* null pointer, negative size, Hq % Hkv != 0, bad scale */
#define TIK_ERR_UNSUPPORTED (-2)   /* outside the supported domain above */
#define TIK_ERR_WORKSPACE (-3)     /* ws_bytes smaller than tik_workspace_bytes(...) */
#define TIK_ERR_CUDA (-4)          /* a CUDA call failed; text via tik_last_error */

/* device-side flags reported by tik_device_status */
#define TIK_DEV_BAD_BLOCK 1        /* block-table entry outside [0,num_pages): page read as zeros */
#define TIK_DEV_BAD_TARGET 2       /* target id outside [0,V): logprob = NaN */
#define TIK_DEV_WAIT_EXPIRED 4     /* an in-kernel bounded wait ran out (outputs invalid) */
#define TIK_DEV_BAD_POSITION 8     /* token position outside the cos/sin table: token left untouched */
#define TIK_DEV_BAD_CONTEXT 16     /* decode: ctx_lens[b] > max_ctx_len: that slot attends keys 0..max_ctx_len-1 only */

#define TIK_OP_ATTN_TRAIN_FWD 0
#define TIK_OP_ATTN_PREFILL 1
#define TIK_OP_ATTN_DECODE 2
#define TIK_OP_TOKEN_LOGPROB 3
#define TIK_OP_ATTN_TRAIN_BWD 4

/* Create / destroy the per-device context (host memory plus one small device status
 * word).  `device` is a CUDA ordinal.  tik_create is the only call that allocates. */
tik_status tik_create(tik_ctx** out, int device);
tik_status tik_destroy(tik_ctx* ctx);

const char* tik_status_str(tik_status s);
/* Text of the last TIK_ERR_CUDA / argument error of this context (host string). */
const char* tik_last_error(const tik_ctx* ctx);
/* Identifies the numerical contract (tile sizes, MMA shape, exp variant, sum shape).
 * Outputs are bit-comparable only between builds with the same id. */
const char* tik_contract_id(void);

/* Host-only self-check of the library's per-device launch bookkeeping (no paper counterpart):
 * kernels that use more than 48 KiB of shared memory are opted in once per (kernel, device), and
 * this exercises that table with stand-in ordinals.  Needs no GPU.  Returns 0 when it holds. */
int tik_selftest_host(void);

/* Number of kernels the library has launched in this process so far (all contexts, all streams;
 * every launch site counts itself when it enqueues a kernel).  No paper counterpart: it lets a
 * benchmark state how many kernels a timed region launched.  Host only, never fails. */
unsigned long long tik_kernel_launches(void);

/* Scratch bytes an operator needs.  rows_or_batch: decode batch B, log-prob rows T, or the number
 * of sequences S for train forward / prefill.  max_ctx: the host's bound on a context length
 * (decode, prefill) or sequence length (train forward).  H, V only for the log-prob op.  Returns 0
 * when no scratch is needed or usable (train forward / prefill outside the range that the
 * persistent schedule handles: they then run without scratch). */
size_t tik_workspace_bytes(int op, int64_t rows_or_batch, int Hq, int Hkv, int d,
                           int64_t max_ctx, int H, int V);

/* Synchronises `stream`, then reads and clears the device flags (TIK_DEV_*). */
tik_status tik_device_status(tik_ctx* ctx, void* stream, int* out_flags);

/* Policy-update forward attention over packed variable-length sequences (paper Sec. 4.1:
 * the full-sequence entry point applied to prompt||response).  Token t of a sequence
 * attends keys 0..t of the same sequence; query head h uses KV head h / (Hq/Hkv).
 *   q [total_tokens][Hq][d], k, v [total_tokens][Hkv][d]  -> o [total_tokens][Hq][d]
 *   lse: optional fp32 [total_tokens][Hq] (natural-log log-sum-exp of the scaled scores)
 *   cu_seqlens: device int32 [S+1]; max_seqlen: host upper bound on any sequence length
 *   (sizes the grid; may be larger than the true maximum).
 *   ws, ws_bytes: optional device scratch of tik_workspace_bytes(TIK_OP_ATTN_TRAIN_FWD, S, ...,
 *   max_seqlen, ...) bytes, 16-byte aligned.  With it the call runs as a persistent kernel (one
 *   CTA per SM walks a device-built list of work items; the list lives in ws); with NULL, or a
 *   buffer that is too small, as one CTA per work item.  The output bits are the same: the
 *   schedule differs, not a row's arithmetic (paper Sec. 5.3: a schedule change must preserve
 *   bits).  ws is borrowed until the stream-ordered work completes; concurrent calls need
 *   buffers of their own. */
tik_status tik_attn_train_fwd(tik_ctx* ctx, const void* q, const void* k, const void* v, void* o,
                              float* lse, const int32_t* cu_seqlens, int S,
                              int64_t total_tokens, int max_seqlen, int Hq, int Hkv, int d,
                              float softmax_scale, void* ws, size_t ws_bytes, void* stream);

/* Backward of tik_attn_train_fwd (the paper measures the policy-update backward in its layer
 * timings, Sec. 6 Q2, and does not put it under Eq. 1: there is no rollout counterpart).  Given
 * dO = dL/dO it returns dQ, dK, dV of the same shapes as q, k, v (bf16, one rounding of fp32
 * accumulators).  With s_ij = scale q_i.k_j, p_ij = exp(s_ij - lse_i), delta_i = dO_i.o_i:
 *   dS_ij = p_ij (dO_i.v_j - delta_i),  dQ_i = scale sum_j dS_ij k_j,
 *   dK_j = scale sum_i dS_ij q_i,  dV_j = sum_i p_ij dO_i      (sums over the query heads of a KV head too)
 * o and lse are the forward's outputs for the same q, k, v, scale (lse: fp32 [total_tokens][Hq]).
 * Deterministic: every output element is accumulated in one fixed order (no atomics); the same
 * inputs give the same bits on every call.  ws: tik_workspace_bytes(TIK_OP_ATTN_TRAIN_BWD,
 * total_tokens, Hq, ...) bytes of device scratch.  Three kernels on `stream`. */
tik_status tik_attn_train_bwd(tik_ctx* ctx, const void* q, const void* k, const void* v, const void* o,
                              const void* d_o, const float* lse, void* dq, void* dk, void* dv,
                              const int32_t* cu_seqlens, int S, int64_t total_tokens, int max_seqlen,
                              int Hq, int Hkv, int d, float softmax_scale, void* ws, size_t ws_bytes,
                              void* stream);

/* Indexed KV-cache write (paper Sec. 4.1: a rollout-only operator; exact copy).  The new
 * tokens of sequence s are rows cu_seqlens_new[s] .. cu_seqlens_new[s+1]-1 of k_new/v_new
 * ([total_new][Hkv][d]) and land at positions ctx_lens[s]-n_s .. ctx_lens[s]-1, where
 * ctx_lens[s] is the context length AFTER the write.  Position p goes to page
 * block_table[s][p / page_size], row p % page_size. */
tik_status tik_kv_cache_write(tik_ctx* ctx, const void* k_new, const void* v_new,
                              const int32_t* cu_seqlens_new, const int32_t* ctx_lens,
                              void* k_cache, void* v_cache, const int32_t* block_table,
                              int max_blocks, int S, int64_t total_new, int Hkv, int d,
                              int page_size, int num_pages, void* stream);

/* Pre-attention step in one pass: per-head RMSNorm of Q and K, NeoX rotary embedding of Q and K,
 * indexed write of K and V into the paged cache.  The paper's operator table (Sec. 6, operator
 * correctness) lists Q RMSNorm, K RMSNorm, NeoX RoPE (Q, K) and the indexed KV-cache write as
 * unified operators verified bitwise between full-sequence and token-wise use; it gives no
 * formulas, so the textbook definitions apply, and the fusion and the order norm -> rotation ->
 * write (the Qwen3 layer order) are this library's choice.  Per (token, head) vector x of length d:
 *   y_i = x_i * rsqrt(mean_j x_j^2 + eps) * w_i                     (skipped when the weight is NULL)
 *   z_i = y_i cos_i - y_{i+d/2} sin_i,  z_{i+d/2} = y_{i+d/2} cos_i + y_i sin_i   for i < d/2
 * with (cos_i, sin_i) = cos_sin[pos][i], cos_sin[pos][d/2 + i]: a caller-built fp32 table
 * [max_pos][d] of cos(p theta_i) | sin(p theta_i) (device memory).  Arithmetic is fp32 with one
 * rounding to bf16 at the end; a vector's result depends on that vector, the weight, eps and its
 * table row only, never on the other tokens of the call.
 *   q [total_new][Hq][d], k [total_new][Hkv][d]: bf16, device, overwritten in place
 *   v [total_new][Hkv][d]: read only; may be NULL when there is no cache
 *   q_weight, k_weight: bf16 [d], device, each may be NULL
 *   token i of sequence s (rows cu_seqlens_new[s]..) has position ctx_lens[s] - n_s + i, where
 *   ctx_lens[s] is the context length AFTER this step; ctx_lens == NULL means positions start at 0
 *   (whole sequences, the policy-update forward)
 *   k_cache, v_cache [num_pages][Hkv][page_size][d]: both NULL = no cache write (then block_table
 *   is ignored); otherwise rotated K and V go to page block_table[s][pos / page_size], row
 *   pos % page_size, exactly the bf16 values written back to k / read from v
 * Device flags: TIK_DEV_BAD_POSITION (position outside [0, max_pos): the token's q, k and cache
 * rows are left untouched), TIK_DEV_BAD_BLOCK (bad table entry: q and k are still transformed, the
 * cache is not written).  Needs no workspace; launches one kernel on `stream`. */
tik_status tik_qk_norm_rope_kv_write(tik_ctx* ctx, void* q, void* k, const void* v,
                                     const void* q_weight, const void* k_weight, float eps,
                                     const float* cos_sin, int max_pos,
                                     const int32_t* cu_seqlens_new, const int32_t* ctx_lens,
                                     void* k_cache, void* v_cache, const int32_t* block_table,
                                     int max_blocks, int S, int64_t total_new, int Hq, int Hkv,
                                     int d, int page_size, int num_pages, void* stream);

/* Rollout prefill attention (paper Sec. 4.1: the full-sequence entry point applied to a
 * prompt) against the paged cache, which must already hold the keys/values of positions
 * 0 .. ctx_lens[s]-1 (tik_kv_cache_write first).  Query i of sequence s sits at absolute
 * position ctx_lens[s] - q_len[s] + i and attends keys 0..position, so a cached prefix
 * (chunked prefill) is supported.  max_q_len / max_ctx_len: host upper bounds.
 * ws, ws_bytes: optional scratch as for tik_attn_train_fwd, sized by
 * tik_workspace_bytes(TIK_OP_ATTN_PREFILL, S, ..., max_ctx_len, ...); same bits with or without. */
tik_status tik_attn_prefill(tik_ctx* ctx, const void* q, void* o, float* lse,
                            const int32_t* cu_seqlens_q, const int32_t* ctx_lens,
                            const void* k_cache, const void* v_cache,
                            const int32_t* block_table, int max_blocks, int S, int64_t total_q,
                            int max_q_len, int max_ctx_len, int Hq, int Hkv, int d,
                            int page_size, int num_pages, float softmax_scale, void* ws,
                            size_t ws_bytes, void* stream);

/* Cache write and prefill in one call (paper Sec. 4.1: prefill both fills the KV cache and scores
 * the prompt): tik_kv_cache_write of the new tokens' keys and values followed by tik_attn_prefill
 * of their queries, on the same stream.  The new tokens are the query tokens: row i of k_new / v_new
 * ([total_q][Hkv][d]) belongs to the same token as row i of q, sequence s owns rows
 * cu_seqlens_q[s] .. cu_seqlens_q[s+1]-1 at positions ctx_lens[s]-q_len[s] .. ctx_lens[s]-1.
 * Output bits are those of the two separate calls. */
tik_status tik_attn_prefill_kv(tik_ctx* ctx, const void* q, const void* k_new, const void* v_new, void* o,
                               float* lse, const int32_t* cu_seqlens_q, const int32_t* ctx_lens,
                               void* k_cache, void* v_cache, const int32_t* block_table,
                               int max_blocks, int S, int64_t total_q, int max_q_len, int max_ctx_len,
                               int Hq, int Hkv, int d, int page_size, int num_pages,
                               float softmax_scale, void* ws, size_t ws_bytes, void* stream);

/* Token-wise decode attention (paper Sec. 4.1: the decode entry point): one query token
 * per sequence at position ctx_lens[b]-1 (its own key/value already written) against keys
 * 0..ctx_lens[b]-1.  q, o [B][Hq][d]; lse optional fp32 [B][Hq].  A slot with
 * ctx_lens[b] <= 0 is skipped and its output rows are left untouched.  The KV range is
 * split into fixed 2048-key chunks whose partial results go through `ws` and are folded in
 * ascending order by a second kernel on the same stream (fixed-order split-KV combine).
 * With max_ctx_len <= 2048 every slot has one chunk, whose state is the result: the decode
 * kernel then normalises and stores the rows itself (same operations, same bits), `ws` is
 * not touched and no second kernel runs.
 * max_ctx_len is a host upper bound on ctx_lens[]: it sizes the grid and the scratch.  A slot
 * whose ctx_lens[b] exceeds it is computed over keys 0..max_ctx_len-1 only and raises
 * TIK_DEV_BAD_CONTEXT; nothing is written outside that slot's own scratch and output rows. */
tik_status tik_attn_decode(tik_ctx* ctx, const void* q, void* o, float* lse,
                           const int32_t* ctx_lens, const void* k_cache, const void* v_cache,
                           const int32_t* block_table, int max_blocks, int B, int max_ctx_len,
                           int Hq, int Hkv, int d, int page_size, int num_pages,
                           float softmax_scale, void* ws, size_t ws_bytes, void* stream);

/* Token log-probabilities (paper Sec. 3.1): z = inv_temperature * hidden[t] . lm_head[v]
 * for all v in fp32 (never rounded to bf16), logprob[t] = z[target[t]] - logsumexp_v z.
 *   hidden [T][H], lm_head [V][H] (row v = class v), target_ids int32 [T]
 *   -> logprob fp32 [T]; lse optional fp32 [T].
 * The logits are never materialised: the GEMM runs on tensor cores with a fixed
 * ascending-K accumulation and is fused with a chunked log-sum-exp whose partial results
 * (per 1024-column super-chunk) go through `ws` and are folded in ascending order. */
tik_status tik_token_logprob(tik_ctx* ctx, const void* hidden, const void* lm_head,
                             const int32_t* target_ids, float* logprob, float* lse, int64_t T,
                             int H, int V, float inv_temperature, void* ws, size_t ws_bytes,
                             void* stream);

/* Hidden RMSNorm, optionally fused with the residual add (the paper's operator table, Sec. 6:
 * "Hidden RMSNorm", "Fused residual + RMSNorm"; no formulas are given, the textbook ones apply).
 *   residual == NULL:  y[t] = x[t] * rsqrt(mean_j x[t][j]^2 + eps) * weight
 *   residual != NULL:  s = bf16(x + residual) (fp32 sum rounded to bf16) is stored back to
 *                      residual and normalised: y[t] = s * rsqrt(mean s^2 + eps) * weight,
 *                      exactly what a bf16 add followed by the plain form gives.
 * x, residual, y: bf16 [T][H], device; weight bf16 [H]; y may alias x.  fp32 arithmetic, one
 * rounding of y.  A row's result depends on that row only (fixed reduction shape), not on T.
 * H must be a multiple of 8 and <= 8192. */
tik_status tik_rmsnorm(tik_ctx* ctx, const void* x, void* residual, const void* weight, void* y,
                       float eps, int64_t T, int H, void* stream);

/* SwiGLU on a fused gate/up projection (operator table: "Standalone SwiGLU"): row t of gate_up
 * [T][2I] holds gate (first I columns) then up (last I); out[t][i] = silu(gate) * up with
 * silu(g) = g / (1 + exp(-g)); bf16 in and out, fp32 arithmetic.  I must be a multiple of 8. */
tik_status tik_swiglu(tik_ctx* ctx, const void* gate_up, void* out, int64_t T, int I, void* stream);

/* Dense linear layer without bias (operator table: "Generic dense FFN"): y = x W^T with
 * x bf16 [T][K], weight bf16 [N][K] (the nn.Linear layout), y bf16 [T][N]; fp32 accumulation over
 * K in one fixed ascending order, one rounding to bf16.  Row t of y depends on row t of x and on
 * weight only, so it has the same bits at T = 1 and inside any batch.  K must be a multiple of
 * 64, N a multiple of 8.  No workspace. */
tik_status tik_linear(tik_ctx* ctx, const void* x, const void* weight, void* y, int64_t T, int K,
                      int N, void* stream);

/* Decode attention without any allocation (the paper has no counterpart; this variant
 * exists for deployments of this library).  Same arguments, kernels and output bits as
 * tik_attn_decode, but it takes no tik_ctx and no workspace: the split-KV scratch is a
 * fixed __device__ array of TIK_STATIC_SCRATCH_BYTES inside the library, resident on every
 * GPU that loads the library until the process exits.  Meant for callers that cannot call
 * cudaMalloc: a server whose KV-cache pool already owns all free device memory, or a decode
 * loop that must avoid the device-wide synchronisation of cudaMalloc/cudaFree.
 *   - Needs B * Hq * ceil(max_ctx_len/2048) * (d+4) * 4 <= TIK_STATIC_SCRATCH_BYTES,
 *     otherwise returns TIK_ERR_WORKSPACE and launches nothing.
 *   - Works on the current CUDA device.  The first call on each device resolves the
 *     scratch's device address and the driver's tensor-map encoder (host-side set-up, no
 *     allocation); make that first call before any stream capture.
 *   - All calls on a device share the one scratch array: two calls whose kernels may overlap
 *     on the GPU (different streams) race on it.  Issue them on one stream or order them.
 *   - dev_flags: optional device int that receives TIK_DEV_* flags (OR-ed in; the caller
 *     zeroes it before the call and reads it afterwards: a word that still holds
 *     TIK_DEV_WAIT_EXPIRED makes the kernels return at once).  With NULL the flags go to a
 *     word inside the library that is cleared at the start of every call and that no entry
 *     point reads: they are DISCARDED, so a bad block-table entry (page read as zeros) or an
 *     expired wait (outputs invalid) goes unreported.  Pass a word to observe them.
 *   - No error text is kept (there is no context): only the status code is returned. */
#define TIK_STATIC_SCRATCH_BYTES (8u << 20)
tik_status tik_attn_decode_static(const void* q, void* o, float* lse, const int32_t* ctx_lens,
                                  const void* k_cache, const void* v_cache,
                                  const int32_t* block_table, int max_blocks, int B,
                                  int max_ctx_len, int Hq, int Hkv, int d, int page_size,
                                  int num_pages, float softmax_scale, int* dev_flags,
                                  void* stream);

#ifdef __cplusplus
}
#endif
#endif /* TIK_H */
