/*
 * diffqkv.h -- C ABI of libdiffqkv: DiffQKV attention over a KV cache on NVIDIA B200 (sm_100a).
 *
 * DiffQKV attention (paper Section 2, "Formulation of DiffQKV Attention") is softmax
 * attention in which Q, K and V have their own head counts n_q, n_k, n_v.  Query head h
 * reads K head  hk = floor(h * n_k / n_q)  and V head  hv = floor(h * n_v / n_q)
 * (Section 3.2, Eq. (idx); n_k and n_v must divide n_q, so hk = h / (n_q/n_k)).  For one
 * query vector q_h and the visible cached tokens j:
 *
 *     s_j = scale * <q_h, K[j, hk]>          m = max_j s_j
 *     p_j = exp(s_j - m)                     l = sum_j p_j
 *     out_h = (sum_j p_j * V[j, hv]) / l     lse_h = m + log(l)
 *
 * K and V live in two separate pools (Section 3.1: the key cache and the value cache have
 * different shapes), streamed once per call; that traffic, b*s*(n_k*d_k + n_v*d_v) elements
 * (Eq. (cache_0)), is what bounds decoding.
 *
 * General rules for every call
 *   - Every pointer in the argument lists and structs is a DEVICE pointer unless it is marked
 *     "host".  The structs themselves (diffqkv_cache, diffqkv_shape) are read on the host.
 *   - The library borrows all buffers, owns nothing and, unless an entry point says otherwise,
 *     allocates nothing: scratch memory is a caller-provided workspace.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*) and return without
 *     synchronising.  Buffers must stay valid until the stream has run the work.
 *   - Errors the host can see (null pointers, head counts that do not divide, unsupported head
 *     dimensions, misaligned pointers, a workspace that is too small, a failed launch) return a
 *     status and launch nothing.  Conditions only the device can see (a page id outside the
 *     pool, a bounded wait that ran out) OR the bit (1 << diffqkv_status value) into *dev_status
 *     (when given) and the affected block skips that work; nothing traps.
 *   - Tensors are dense in their last (channel) dimension.  bf16 tensors must be 16-byte
 *     aligned with strides that are multiples of 8 elements; fp32 tensors 16-byte aligned with
 *     strides that are multiples of 4 elements.
 */
#ifndef DIFFQKV_H_
#define DIFFQKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DIFFQKV_OK = 0,
  DIFFQKV_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, n_k or n_v not dividing n_q ... */
  DIFFQKV_ERR_UNSUPPORTED = 2, /* a shape or dtype no kernel covers                                */
  DIFFQKV_ERR_ALIGNMENT = 3,   /* a pointer or stride violates the alignment rules above           */
  DIFFQKV_ERR_WORKSPACE = 4,   /* workspace missing or smaller than the *_workspace_bytes answer   */
  DIFFQKV_ERR_CUDA = 5,        /* a CUDA runtime or driver call failed                             */
  DIFFQKV_ERR_TIMEOUT = 6,     /* device: a bounded wait on a copy ran out                         */
  DIFFQKV_ERR_INDEX = 7        /* device: page id outside [0, num_blocks)                          */
} diffqkv_status;

typedef enum { DIFFQKV_BF16 = 0, DIFFQKV_F32 = 1 } diffqkv_dtype;

/*
 * The KV cache: two pools addressed through the same rule.  Token j of sequence b, head hd,
 * channel c of the K pool sits at element offset
 *     blk * k_stride_blk + hd * k_stride_head + slot * k_stride_tok + c
 * with (blk, slot) = (b, j) for a contiguous cache (page_table == NULL) and
 * (blk, slot) = (page_table[b * max_pages_per_seq + j / page_size], j % page_size) for a paged
 * one; likewise for V.  One page table serves both pools.  The paper fixes only the logical
 * shapes (b, s, n_h, d_h) (Section 3.1); strides make head-major and token-major storage
 * both expressible, and the page format is this library's own.
 */
typedef struct {
  void *k_cache;             /* K pool, element type = shape.dtype                                  */
  void *v_cache;             /* V pool                                                              */
  int64_t k_stride_blk, k_stride_head, k_stride_tok; /* in elements                                 */
  int64_t v_stride_blk, v_stride_head, v_stride_tok;
  const int32_t *seqlens;    /* [batch] visible tokens per sequence (decode: includes the new one)  */
  const int32_t *page_table; /* [batch, max_pages_per_seq] physical page ids, or NULL = contiguous  */
  int32_t page_size;         /* tokens per page (paged only; a multiple of 16 for the TMA kernels)  */
  int32_t max_pages_per_seq; /* row length of page_table                                            */
  int32_t num_blocks;        /* extent of the blk dimension: pages in the pool, or batch            */
  int32_t max_seqlen;        /* host-known upper bound of seqlens[]; contiguous: also the token     */
                             /* extent of each (blk, head) slab, so reads never pass it             */
} diffqkv_cache;

typedef struct {
  int32_t batch, n_q, n_k, n_v; /* n_q % n_k == 0 and n_q % n_v == 0                                */
  int32_t d_qk, d_v;            /* channels per head of Q/K and of V                                */
  diffqkv_dtype dtype;          /* storage type of q, K and V; accumulation is always fp32          */
  diffqkv_dtype out_dtype;      /* storage type of `out`                                            */
  float scale;                  /* multiplies the inner product; the paper uses 1/sqrt(d_k)         */
} diffqkv_shape;

/*
 * Split planning for decode (Section 3.2: the split kernel divides K and V into chunks along
 * the sequence).  The sequence axis is cut into chunks of one fixed length; sequence b uses
 * ceil(seqlens[b] / chunk) of the at most S splits.
 *   diffqkv_decode_num_splits: S the library would choose for num_splits = 0 (always >= 1).
 *   diffqkv_decode_workspace_bytes: bytes of workspace diffqkv_decode / gqa_decode need for
 *   this shape, max_seqlen and num_splits (0 = the automatic choice).  Returns 0 on bad input.
 */
int32_t diffqkv_decode_num_splits(const diffqkv_shape *shape, int32_t max_seqlen);
size_t diffqkv_decode_workspace_bytes(const diffqkv_shape *shape, int32_t max_seqlen, int32_t num_splits);

/*
 * diffqkv_decode -- one query token per sequence against the cache (Section 2 formulation with
 * the head map of Eq. (idx); split-sequence execution per Section 3.2).
 *   q          [batch, n_q, d_qk]  shape.dtype, contiguous
 *   cache      see diffqkv_cache; seqlens[b] == 0 gives out = 0 and lse = -inf for that sequence
 *   num_splits 0 = automatic (recommended): bf16 caches that a TMA tensor map can describe use the
 *              persistent TMA kernel, which divides all (sequence, head group, 64-token tile) work
 *              evenly over one block per SM and cuts sequences wherever a block's share ends; other
 *              inputs use fixed chunks.  > 0 = fixed chunks, at most that many per sequence (generic kernel);
 *              more than 8192 returns DIFFQKV_ERR_UNSUPPORTED
 *   workspace  at least diffqkv_decode_workspace_bytes(...) bytes, 256-byte aligned; holds the
 *              per-split partial outputs (fp32 [batch, n_q, S, d_v]) and log-sum-exps
 *              (fp32 [batch, n_q, S]); contents on entry are ignored
 *   out        [batch, n_q, d_v]   shape.out_dtype
 *   lse        [batch, n_q] fp32 natural-log log-sum-exp of the scaled scores, or NULL
 *   dev_status one int32 the kernels OR (1 << diffqkv_status) bits into, or NULL; the caller zeroes it
 * Runs the split kernel and then the combine kernel on `stream`.  With few, short rows (the blocks that share a
 * (sequence, head group) row fill at least 0.85 of the SMs as clusters of 2 to 8 and the cache's capacity for them is
 * small enough that the idle SMs cost less than a second launch) the TMA kernel's blocks of a row form a thread-block
 * cluster and merge on chip instead: one launch, the workspace is not used.
 */
diffqkv_status diffqkv_decode(const void *q, const diffqkv_cache *cache, const diffqkv_shape *shape,
                              int32_t num_splits, void *workspace, size_t workspace_bytes, void *out,
                              float *lse, int32_t *dev_status, void *stream);

/*
 * diffqkv_decode_host -- diffqkv_decode for a query that sits in host memory and a result that is wanted there (the
 * paper has no counterpart; the KV cache is decode state and stays on the device).  On `stream`, in order: copy
 * q_host -> q_dev, diffqkv_decode(q_dev ... out_dev), copy out_dev -> out_host.  Nothing is synchronised: the result
 * is in out_host once the stream has run the last copy.
 *   q_host, out_host  HOST pointers ([batch, n_q, d_qk] shape.dtype and [batch, n_q, d_v] shape.out_dtype);
 *                     page-locked memory keeps the copies asynchronous
 *   q_dev, out_dev    device staging buffers of the same sizes, provided by the caller (the library allocates nothing)
 *   everything else as in diffqkv_decode
 */
diffqkv_status diffqkv_decode_host(const void *q_host, void *q_dev, const diffqkv_cache *cache,
                                   const diffqkv_shape *shape, int32_t num_splits, void *workspace,
                                   size_t workspace_bytes, void *out_dev, void *out_host, float *lse,
                                   int32_t *dev_status, void *stream);

/*
 * diffqkv_decode_static -- diffqkv_decode for callers that cannot provide or allocate a workspace.
 * (The paper has no counterpart; this is a deployment convenience of this library.)
 * Some hosts cannot call cudaMalloc when they decode: all device memory already belongs to their own
 * pool, or they sit behind an interface with no workspace argument, or an allocation would stall a
 * latency-critical loop.  For them the split kernel's partial results go to a fixed 8 MiB array built
 * into the library (each GPU that loads the library carries those 8 MiB until the process exits).
 * Arguments and results are those of diffqkv_decode without `workspace` / `workspace_bytes`.
 *   - Returns DIFFQKV_ERR_WORKSPACE, launching nothing, when
 *     diffqkv_decode_workspace_bytes(shape, cache->max_seqlen, num_splits) exceeds 8 MiB (8388608 bytes);
 *     choose fewer splits or a smaller batch, or use diffqkv_decode with your own buffer.
 *   - Calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - The first call on each device resolves the array's device address (the device of `stream` must be
 *     the current device); make that first call outside any stream capture.
 *   - All calls on one device share the one array: two calls whose kernels may overlap on the GPU
 *     (different streams without ordering, or several host threads) race on it.  Calls on one stream
 *     are safe.  The array keeps the previous call's partials; nothing in it needs clearing because a
 *     call reads only what it has itself written.
 */
diffqkv_status diffqkv_decode_static(const void *q, const diffqkv_cache *cache, const diffqkv_shape *shape,
                                     int32_t num_splits, void *out, float *lse, int32_t *dev_status,
                                     void *stream);

/*
 * gqa_decode -- grouped-query attention, the comparison point of the paper (Appendix B.1: GQA is
 * the special case n_k == n_v).  Same arguments and the same kernels as diffqkv_decode; returns
 * DIFFQKV_ERR_INVALID_ARG when shape.n_k != shape.n_v.
 */
diffqkv_status gqa_decode(const void *q, const diffqkv_cache *cache, const diffqkv_shape *shape,
                          int32_t num_splits, void *workspace, size_t workspace_bytes, void *out,
                          float *lse, int32_t *dev_status, void *stream);

/*
 * diffqkv_combine -- merge per-split partial results (Section 3.2: the combine kernel assembles
 * the output chunks).  With o_s the NORMALISED output of split s and lse_s its log-sum-exp:
 *     lse = log sum_s exp(lse_s),   out = sum_s exp(lse_s - lse) * o_s,
 * splits with lse_s == -inf are skipped; if all are, out = 0 and lse = -inf.
 *   o_partial   [rows, S, d_v] fp32     lse_partial [rows, S] fp32     (rows = batch * n_q)
 *   out         [rows, d_v] out_dtype   lse [rows] fp32 or NULL
 */
diffqkv_status diffqkv_combine(const float *o_partial, const float *lse_partial, int32_t batch, int32_t n_q,
                               int32_t d_v, int32_t num_splits, diffqkv_dtype out_dtype, void *out,
                               float *lse, void *stream);

/*
 * diffqkv_prefill -- causal attention for q_len new tokens per sequence, writing their K and V
 * rows into the cache first (appendix attention listing: cache update, then the causal
 * flash-attention call; head map of Eq. (idx)).
 *   q      [batch, q_len, n_q, d_qk]   k_new [batch, q_len, n_k, d_qk]   v_new [batch, q_len, n_v, d_v]
 *   cache  seqlens[b] = tokens already cached (past_b) on entry; rows past_b .. past_b + q_len - 1 of
 *          both pools are overwritten; seqlens itself is not modified (the caller adds q_len)
 *   out    [batch, q_len, n_q, d_v] out_dtype; query row i sees tokens 0 .. past_b + i
 *   lse    [batch, q_len, n_q] fp32 or NULL
 * bf16 with (d_qk, d_v) = (128, 128), (64, 64) or (64, 128), a positive scale and pages of at least 8 tokens that
 * divide or are multiples of 128 runs on the tensor cores; every other shape diffqkv_decode accepts (fp32, other head
 * dimensions, scale <= 0) runs the same two steps on a plain fp32-FMA kernel, one block per query row, which is a
 * correctness path, not a fast one.
 */
diffqkv_status diffqkv_prefill(const void *q, const void *k_new, const void *v_new, int32_t q_len,
                               const diffqkv_cache *cache, const diffqkv_shape *shape, void *out, float *lse,
                               int32_t *dev_status, void *stream);

/*
 * diffqkv_augq -- the augmented-Q projection that produces the queries (Section 2, Observation 3;
 * appendix attention listing: q_proj followed by q_down_proj(act(q_gate_proj(x)) * q_up_proj(x))).
 * act is read as SiLU, there are no biases, and weights use the nn.Linear layout [out, in]:
 *     x = h W_Q^T,   a = silu(x W_gate^T) * (x W_up^T),   q = a W_down^T
 *   h [T, d_model]   W_Q [d_q0, d_model]   W_gate, W_up [d_aug, d_q0]   W_down [d_out, d_aug]   all bf16
 *   workspace  diffqkv_augq_workspace_bytes(T, d_q0, d_aug) bytes, 256-byte aligned, for x and a
 *   q_out [T, d_out] bf16
 *   dev_status as in diffqkv_decode, or NULL
 * Products accumulate in fp32 on the tensor cores; x and a are rounded to bf16 once each (they are the next
 * product's bf16 operands).  All dimensions must be multiples of 128 except T; T == 0 does nothing.
 */
size_t diffqkv_augq_workspace_bytes(int64_t T, int32_t d_q0, int32_t d_aug);
diffqkv_status diffqkv_augq(const void *h, const void *W_Q, const void *W_gate, const void *W_up,
                            const void *W_down, int64_t T, int32_t d_model, int32_t d_q0, int32_t d_aug,
                            int32_t d_out, void *workspace, size_t workspace_bytes, void *q_out,
                            int32_t *dev_status, void *stream);

/*
 * diffqkv_augq_rope -- diffqkv_augq followed by the rotary position embedding of the appendix attention listing
 * (apply_rotary_pos_emb on the query), fused into the last product's epilogue: the rotation acts on the fp32
 * result before it is rounded to bf16.  The listing only names the call; it is read as the rotate-half pairing:
 * within a head of width head_dim, channel i < head_dim/2 pairs with channel i + head_dim/2,
 *     y_i = x_i cos[t, i] - x_{i+head_dim/2} sin[t, i],   y_{i+head_dim/2} = x_{i+head_dim/2} cos[t, i] + x_i sin[t, i].
 *   cos, sin  [T, head_dim / 2] fp32 tables of the caller (angle of pair i at position pos: pos * theta^(-2 i / head_dim));
 *             both NULL = no rotation
 *   head_dim  64 or 128; d_out must be a multiple of it
 * Everything else as diffqkv_augq.
 */
diffqkv_status diffqkv_augq_rope(const void *h, const void *W_Q, const void *W_gate, const void *W_up,
                                 const void *W_down, int64_t T, int32_t d_model, int32_t d_q0, int32_t d_aug,
                                 int32_t d_out, int32_t head_dim, const float *cos, const float *sin, void *workspace,
                                 size_t workspace_bytes, void *q_out, int32_t *dev_status, void *stream);

/*
 * diffqkv_project -- a plain projection of the attention listing (k_proj, v_proj): y = x W^T with W in the
 * nn.Linear layout [d_out, d_in], no bias, on the tensor cores with fp32 accumulation; with cos / sin given, the
 * rotary embedding above is applied per head before rounding (the key projection), without them it is a plain
 * product (the value projection).
 *   x [T, d_in] bf16   W [d_out, d_in] bf16   y [T, d_out] bf16   d_in and d_out multiples of 128
 * The result [T, n_heads, head_dim] is the k_new / v_new layout of diffqkv_prefill and diffqkv_cache_append.
 */
diffqkv_status diffqkv_project(const void *x, const void *W, int64_t T, int32_t d_in, int32_t d_out, int32_t head_dim,
                               const float *cos, const float *sin, void *y, int32_t *dev_status, void *stream);

/*
 * diffqkv_cache_append -- the cache update of the attention listing on its own (diffqkv_prefill does the same
 * before it attends): k_new [batch, q_len, n_k, d_qk] and v_new [batch, q_len, n_v, d_v] are written to token
 * positions seqlens[b] .. seqlens[b] + q_len - 1 of the pools (any strides, paged or contiguous, bf16 or fp32).
 * seqlens itself is not modified.  Positions at or past max_seqlen, and page ids outside the pool, are skipped
 * and reported as DIFFQKV_ERR_INDEX in *dev_status.  A decode step is: append the new token's rows, add 1 to
 * seqlens, call diffqkv_decode.
 */
diffqkv_status diffqkv_cache_append(const void *k_new, const void *v_new, int32_t q_len, const diffqkv_cache *cache,
                                    const diffqkv_shape *shape, int32_t *dev_status, void *stream);

/*
 * diffqkv_decode_frontend -- everything one decode step computes from the hidden states before it attends
 * (appendix attention listing: q_proj and the augmented-Q chain, k_proj, v_proj, rotary embedding, cache update), for
 * one new token per sequence:
 *     q_out[b] = rope(aug-Q(h[b]))                      as diffqkv_augq_rope with T = batch rows
 *     K cache row at position seqlens[b]  = rope(h[b] W_K^T)     V cache row at seqlens[b] = h[b] W_V^T
 *   h [batch, d_model] bf16; W_Q [n_q d_qk, d_model], W_gate, W_up [d_aug, n_q d_qk], W_down [n_q d_qk, d_aug],
 *   W_K [n_k d_qk, d_model], W_V [n_v d_v, d_model], all bf16 in the nn.Linear layout
 *   cos, sin   [batch, d_qk / 2] fp32 tables of the new tokens' positions, or both NULL for no rotation
 *   cache      bf16 pools; seqlens[b] = tokens already cached; seqlens is not modified (the caller adds 1 and calls
 *              diffqkv_decode with q_out); positions at or past max_seqlen and page ids outside the pool are
 *              reported as DIFFQKV_ERR_INDEX in *dev_status and skipped
 *   workspace  diffqkv_decode_frontend_workspace_bytes(shape, d_aug) bytes, 256-byte aligned
 *   q_out      [batch, n_q, d_qk] bf16
 * With at most 64 sequences this is three launches (the products of h share one, which writes k and v straight into
 * the cache); with more it is the separate steps of diffqkv_augq_rope, diffqkv_project and diffqkv_cache_append.
 * d_model, d_aug and n_q d_qk must be multiples of 128, n_k d_qk and n_v d_v multiples of 16 (of 128 beyond 64
 * sequences), d_qk 64 or 128 when rotating.
 */
size_t diffqkv_decode_frontend_workspace_bytes(const diffqkv_shape *shape, int32_t d_aug);
diffqkv_status diffqkv_decode_frontend(const void *h, const void *W_Q, const void *W_gate, const void *W_up,
                                       const void *W_down, const void *W_K, const void *W_V, int32_t d_model,
                                       int32_t d_aug, const float *cos, const float *sin, const diffqkv_cache *cache,
                                       const diffqkv_shape *shape, void *workspace, size_t workspace_bytes,
                                       void *q_out, int32_t *dev_status, void *stream);

/*
 * diffqkv_fold_k_up -- queries for a K cache that is stored at a smaller head width than the queries (Section 2:
 * when the Q and K head dimensions differ, Attend first transforms K to the query width through another feed-forward
 * layer; Observation 2 and its table: d_k = d_v / 2).  The layer is read as linear, without bias, one matrix per K
 * head.  Since <q_h, W[hk] k_j> = <W[hk]^T q_h, k_j>, widening every cached key is replaced by folding the layer
 * into the query once:
 *     q_out[t, h, :] = W_kup[hk]^T q[t, h, :],   hk = floor(h * n_k / n_q)
 *   q      [T, n_q, d_q] bf16      W_kup [n_k, d_q, d_k] bf16      q_out [T, n_q, d_k] bf16 (fp32 accumulation)
 * Call sequence for the half-width cache: diffqkv_fold_k_up, then diffqkv_decode / diffqkv_prefill /
 * diffqkv_decode_topk with shape.d_qk = d_k (64 with d_v = 128 runs on the TMA and tensor-core kernels) and the
 * same scale the full-width scores would use.  Runs on the tensor cores when d_q is a multiple of 16 up to 256, d_k
 * is 32, 64 or 128 and not above d_q, and the three pointers are 16-byte aligned; every other shape takes a plain
 * kernel, for which (n_q / n_k) * d_q may not exceed 3072 and d_q must be a multiple of 4 (DIFFQKV_ERR_UNSUPPORTED
 * otherwise).
 */
diffqkv_status diffqkv_fold_k_up(const void *q, const void *W_kup, int64_t T, int32_t n_q, int32_t n_k, int32_t d_q,
                                 int32_t d_k, void *q_out, void *stream);

/*
 * diffqkv_decode_topk -- decode with selective V cache fetching (paper Section "Selective V Cache Fetching"; its
 * table uses the 100 highest scores): every query head scores all cached tokens of its K head, keeps the `topk`
 * highest scores (equal scores: the earlier token), takes the softmax over the kept scores only (the paper does
 * not say whether the weights are renormalised; read as renormalised) and sums the kept V rows.  The K cache is
 * streamed once, of the V cache only topk rows per query head are read.  A sequence with at most topk tokens gives
 * exactly the full attention of diffqkv_decode.
 *   q, cache, out, lse, dev_status as in diffqkv_decode; bf16 only, d_qk 64 or 128, at most 32 query heads per
 *   K head, 1 <= topk <= 1024, d_v a multiple of 8 with 16-byte aligned V rows, pages of 16, 32, 64 or a multiple
 *   of 128 tokens; topk times the number of 32768-token pieces of max_seqlen may not exceed 8192
 *   (DIFFQKV_ERR_UNSUPPORTED otherwise)
 *   workspace  diffqkv_decode_topk_workspace_bytes(shape, cache->max_seqlen, topk) bytes, 256-byte aligned: the fp32
 *              scores [batch, n_q, max_seqlen rounded up to 128] and the largest score of every 16 consecutive tokens
 */
size_t diffqkv_decode_topk_workspace_bytes(const diffqkv_shape *shape, int32_t max_seqlen, int32_t topk);
diffqkv_status diffqkv_decode_topk(const void *q, const diffqkv_cache *cache, const diffqkv_shape *shape, int32_t topk,
                                   void *workspace, size_t workspace_bytes, void *out, float *lse,
                                   int32_t *dev_status, void *stream);
/*
 * diffqkv_decode_topk_ids -- the same, and also says which tokens were kept (for callers that audit the selection or
 * reuse it for a later step):
 *   kept_ids  int32 [batch, n_q, topk]: the cached positions of the tokens whose V rows entered the output of each
 *             query head, in no particular order, padded with -1 when the sequence has fewer than topk tokens; NULL
 *             makes the call identical to diffqkv_decode_topk
 */
diffqkv_status diffqkv_decode_topk_ids(const void *q, const diffqkv_cache *cache, const diffqkv_shape *shape,
                                       int32_t topk, void *workspace, size_t workspace_bytes, void *out, float *lse,
                                       int32_t *kept_ids, int32_t *dev_status, void *stream);

/* Static, never-null description of a status value. */
const char *diffqkv_status_string(diffqkv_status status);

/*
 * Tuning hook (process-wide host state) for the TMA decode kernel's tail balance.  Every persistent block holds the
 * last few 64-token tiles of its share in a reserve that it and the other blocks working on the same (sequence, head
 * group) draw from one tile at a time, so that a block that runs ahead takes over tiles of one that runs behind.
 * Which block ends up with which tile depends on timing, so results can differ between runs in the last bits
 * (fp32 summation order); everything stays within the stated tolerances.
 *   tiles < 0  automatic (default): up to 8 tiles per block, at most a sixth of a block's share
 *   tiles = 0  no reserve: every tile has a fixed owner and results are bitwise reproducible from run to run
 *   tiles > 0  exactly that many (always leaving each segment one tile of its own); for tests
 * Workspace sizes do not depend on it.
 */
void diffqkv_set_tail_reserve(int32_t tiles);

#ifdef __cplusplus
}
#endif
#endif /* DIFFQKV_H_ */
