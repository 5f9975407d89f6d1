// C-ABI entry points of libdiffqkv: argument checks, split planning, kernel selection.
#include <atomic>

#include "common.cuh"
#include "diffqkv_debug.h"

namespace diffqkv {

static std::atomic<long long> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

DecodePlan plan_decode(const diffqkv_shape& shape, int max_seqlen, int num_splits) {
  if (max_seqlen < 1) max_seqlen = 1;
  int want = num_splits;
  if (want <= 0) {  // automatic: chunks of about 512 tokens, shorter when that leaves most SMs idle; at most 64 splits
    want = (max_seqlen + 511) / 512;
    const long long rows = (long long)shape.batch * shape.n_q;
    const long long fill = rows > 0 ? (592 + rows - 1) / rows : 1;  // about four blocks per SM
    if (want < fill) want = (int)fill;
    if (want > 64) want = 64;
  }
  if (want < 1) want = 1;
  int chunk = (max_seqlen + want - 1) / want;
  chunk = (chunk + kChunkQuantum - 1) / kChunkQuantum * kChunkQuantum;
  DecodePlan pl;
  pl.chunk = chunk;
  pl.splits = (max_seqlen + chunk - 1) / chunk;
  return pl;
}

constexpr int kMaxSplits = 8192;  // combine_kernel keeps one weight per split in shared memory
// Hook state: process-wide, written and read from any calling thread, hence atomics.
static std::atomic<cudaEvent_t> g_ev_before{nullptr}, g_ev_after{nullptr};
static std::atomic<int> g_last_kernel{0};  // 0 none, 1 generic, 2 TMA

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static diffqkv_status check_shape(const diffqkv_shape* s) {
  if (!s) return DIFFQKV_ERR_INVALID_ARG;
  if (s->batch < 0 || s->n_q <= 0 || s->n_k <= 0 || s->n_v <= 0 || s->d_qk <= 0 || s->d_v <= 0)
    return DIFFQKV_ERR_INVALID_ARG;
  if (s->n_q % s->n_k != 0 || s->n_q % s->n_v != 0) return DIFFQKV_ERR_INVALID_ARG;
  if (s->dtype != DIFFQKV_BF16 && s->dtype != DIFFQKV_F32) return DIFFQKV_ERR_INVALID_ARG;
  if (s->out_dtype != DIFFQKV_BF16 && s->out_dtype != DIFFQKV_F32) return DIFFQKV_ERR_INVALID_ARG;
  if (!(s->scale == s->scale)) return DIFFQKV_ERR_INVALID_ARG;
  if (s->batch > 65535 || s->n_q > 65535) return DIFFQKV_ERR_UNSUPPORTED;
  const int vec = s->dtype == DIFFQKV_BF16 ? 8 : 4;
  if (s->d_qk % vec != 0 || s->d_v % vec != 0) return DIFFQKV_ERR_UNSUPPORTED;
  if (s->d_v > 512 || s->d_qk > 8192) return DIFFQKV_ERR_UNSUPPORTED;
  return DIFFQKV_OK;
}

static diffqkv_status check_cache(const diffqkv_cache* c, const diffqkv_shape* s) {
  if (!c || !c->k_cache || !c->v_cache || !c->seqlens) return DIFFQKV_ERR_INVALID_ARG;
  if (c->max_seqlen < 0 || c->num_blocks < 0) return DIFFQKV_ERR_INVALID_ARG;
  if (c->page_table) {
    if (c->page_size <= 0 || c->max_pages_per_seq <= 0) return DIFFQKV_ERR_INVALID_ARG;
    if ((long long)c->max_pages_per_seq * c->page_size < c->max_seqlen) return DIFFQKV_ERR_INVALID_ARG;
  } else if (c->num_blocks < s->batch) {
    return DIFFQKV_ERR_INVALID_ARG;
  }
  const int vec = s->dtype == DIFFQKV_BF16 ? 8 : 4;
  const long long strides[6] = {c->k_stride_blk, c->k_stride_head, c->k_stride_tok,
                                c->v_stride_blk, c->v_stride_head, c->v_stride_tok};
  for (long long st : strides)
    if (st < 0 || st % vec != 0) return DIFFQKV_ERR_ALIGNMENT;
  if (c->k_stride_tok < s->d_qk || c->v_stride_tok < s->d_v) return DIFFQKV_ERR_INVALID_ARG;
  if (!aligned16(c->k_cache) || !aligned16(c->v_cache)) return DIFFQKV_ERR_ALIGNMENT;
  return DIFFQKV_OK;
}

static CacheView view_of(const diffqkv_cache* c) {
  CacheView v;
  v.k = c->k_cache;
  v.v = c->v_cache;
  v.k_sb = c->k_stride_blk; v.k_sh = c->k_stride_head; v.k_st = c->k_stride_tok;
  v.v_sb = c->v_stride_blk; v.v_sh = c->v_stride_head; v.v_st = c->v_stride_tok;
  v.seqlens = c->seqlens;
  v.page_table = c->page_table;
  v.page_size = c->page_size;
  v.max_pages_per_seq = c->max_pages_per_seq;
  v.num_blocks = c->num_blocks;
  v.max_seqlen = c->max_seqlen;
  return v;
}

static size_t decode_workspace_bytes(const diffqkv_shape& s, const DecodePlan& pl) {
  const size_t rows = (size_t)s.batch * s.n_q;
  return align_up(rows * pl.splits * s.d_v * sizeof(float), 256) + align_up(rows * pl.splits * sizeof(float), 256);
}

// Workspace for either schedule.  The TMA path needs little, but whether a given cache layout can be
// described by a tensor map is only known at the call, so the answer covers the generic kernel too.
static size_t workspace_need(const diffqkv_shape& s, int max_seqlen, int num_splits) {
  size_t need = decode_workspace_bytes(s, plan_decode(s, max_seqlen, num_splits));
  if (num_splits == 0) {
    diffqkv_cache fake = {};
    fake.max_seqlen = max_seqlen;
    TmaPlan tp;
    if (tma_decode_supported(s, fake, &tp)) {
      const size_t t = tma_decode_workspace_bytes(s, tp);
      if (t > need) need = t;
    }
  }
  return need;
}

void profile_after_split(cudaStream_t stream) {
  const cudaEvent_t before = g_ev_before.load(), after = g_ev_after.load();
  if (before && after) cudaEventRecord(after, stream);
}

static diffqkv_status decode_impl(const void* q, const diffqkv_cache* cache, const diffqkv_shape* shape,
                                  int32_t num_splits, void* workspace, size_t workspace_bytes, void* out,
                                  float* lse, int32_t* dev_status, cudaStream_t stream) {
  diffqkv_status st = check_shape(shape);
  if (st != DIFFQKV_OK) return st;
  if (!q || !out) return DIFFQKV_ERR_INVALID_ARG;
  st = check_cache(cache, shape);
  if (st != DIFFQKV_OK) return st;
  if (!aligned16(q) || !aligned16(out)) return DIFFQKV_ERR_ALIGNMENT;
  if (num_splits < 0) return DIFFQKV_ERR_INVALID_ARG;
  if (num_splits > kMaxSplits) return DIFFQKV_ERR_UNSUPPORTED;  // the combine kernel's limit, as in diffqkv_combine
  if (shape->batch == 0) return DIFFQKV_OK;
  const DecodePlan pl = plan_decode(*shape, cache->max_seqlen, num_splits);
  const size_t need = workspace_need(*shape, cache->max_seqlen, num_splits);
  if (!workspace || workspace_bytes < need) return DIFFQKV_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return DIFFQKV_ERR_ALIGNMENT;
  const cudaEvent_t ev_before = g_ev_before.load();
  const bool timed = ev_before && g_ev_after.load();

  // bf16 caches a tensor map can describe go to the TMA kernel (automatic schedule only)
  TmaPlan tp;
  if (num_splits == 0 && tma_decode_supported(*shape, *cache, &tp)) {
    if (timed) cudaEventRecord(ev_before, stream);
    const cudaError_t terr = launch_decode_tma(q, *cache, *shape, tp, workspace, out, lse, dev_status, stream);
    if (terr == cudaSuccess) {
      g_last_kernel = 2;
      return DIFFQKV_OK;
    }
    if (terr != cudaErrorNotSupported) return DIFFQKV_ERR_CUDA;
  }

  const size_t rows = (size_t)shape->batch * shape->n_q;
  DecodeParams p;
  p.q = q;
  p.cache = view_of(cache);
  p.batch = shape->batch; p.n_q = shape->n_q; p.n_k = shape->n_k; p.n_v = shape->n_v;
  p.d_qk = shape->d_qk; p.d_v = shape->d_v;
  p.scale_log2 = shape->scale * kLog2e;
  p.chunk = pl.chunk;
  p.splits = pl.splits;
  p.o_partial = reinterpret_cast<float*>(workspace);
  p.lse_partial = reinterpret_cast<float*>(reinterpret_cast<char*>(workspace) +
                                           align_up(rows * pl.splits * shape->d_v * sizeof(float), 256));
  p.dev_status = dev_status;

  if (timed) cudaEventRecord(ev_before, stream);
  cudaError_t err = launch_decode_generic(p, shape->dtype, stream);
  g_last_kernel = 1;
  profile_after_split(stream);
  if (err != cudaSuccess) return DIFFQKV_ERR_CUDA;
  err = launch_combine(p.o_partial, p.lse_partial, (int)rows, shape->d_v, pl.splits, shape->out_dtype, out, lse,
                       stream);
  return err == cudaSuccess ? DIFFQKV_OK : DIFFQKV_ERR_CUDA;
}

}  // namespace diffqkv

using namespace diffqkv;

extern "C" {

int32_t diffqkv_decode_num_splits(const diffqkv_shape* shape, int32_t max_seqlen) {
  if (check_shape(shape) != DIFFQKV_OK) return 1;
  return plan_decode(*shape, max_seqlen, 0).splits;
}

size_t diffqkv_decode_workspace_bytes(const diffqkv_shape* shape, int32_t max_seqlen, int32_t num_splits) {
  if (check_shape(shape) != DIFFQKV_OK || max_seqlen < 0 || num_splits < 0) return 0;
  return workspace_need(*shape, max_seqlen, num_splits);
}

void diffqkv_set_max_blocks(int32_t max_blocks) { set_tma_max_blocks(max_blocks); }

void diffqkv_set_tail_reserve(int32_t tiles) { set_tma_tail_reserve(tiles); }

void diffqkv_debug_decode_per_head_only(int32_t on) { set_decode_per_head_only(on); }
void diffqkv_debug_decode_cluster(int32_t mode) { set_tma_cluster_mode(mode); }

void diffqkv_debug_decode_timeout(int64_t wait_limit_ns, int64_t skip_tile) {
  set_tma_debug_timeout(wait_limit_ns, skip_tile);
}

void diffqkv_topk_general_only(int32_t on) { set_topk_general_only(on); }

void diffqkv_force_tensor_gemm(int32_t on) { set_force_tensor_gemm(on); }

int32_t diffqkv_last_decode_kernel(void) { return g_last_kernel; }

diffqkv_status diffqkv_decode(const void* q, const diffqkv_cache* cache, const diffqkv_shape* shape,
                              int32_t num_splits, void* workspace, size_t workspace_bytes, void* out, float* lse,
                              int32_t* dev_status, void* stream) {
  return decode_impl(q, cache, shape, num_splits, workspace, workspace_bytes, out, lse, dev_status,
                     static_cast<cudaStream_t>(stream));
}

diffqkv_status diffqkv_decode_host(const void* q_host, void* q_dev, const diffqkv_cache* cache,
                                   const diffqkv_shape* shape, int32_t num_splits, void* workspace,
                                   size_t workspace_bytes, void* out_dev, void* out_host, float* lse,
                                   int32_t* dev_status, void* stream) {
  const diffqkv_status st = check_shape(shape);
  if (st != DIFFQKV_OK) return st;
  if (!q_host || !q_dev || !out_dev || !out_host) return DIFFQKV_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t rows = (size_t)shape->batch * shape->n_q;
  const size_t q_bytes = rows * shape->d_qk * (shape->dtype == DIFFQKV_BF16 ? 2 : 4);
  const size_t out_bytes = rows * shape->d_v * (shape->out_dtype == DIFFQKV_BF16 ? 2 : 4);
  if (q_bytes && cudaMemcpyAsync(q_dev, q_host, q_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return DIFFQKV_ERR_CUDA;
  const diffqkv_status ds =
      decode_impl(q_dev, cache, shape, num_splits, workspace, workspace_bytes, out_dev, lse, dev_status, s);
  if (ds != DIFFQKV_OK) return ds;
  if (out_bytes && cudaMemcpyAsync(out_host, out_dev, out_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return DIFFQKV_ERR_CUDA;
  return DIFFQKV_OK;
}

diffqkv_status gqa_decode(const void* q, const diffqkv_cache* cache, const diffqkv_shape* shape, int32_t num_splits,
                          void* workspace, size_t workspace_bytes, void* out, float* lse, int32_t* dev_status,
                          void* stream) {
  if (shape && shape->n_k != shape->n_v) return DIFFQKV_ERR_INVALID_ARG;
  return decode_impl(q, cache, shape, num_splits, workspace, workspace_bytes, out, lse, dev_status,
                     static_cast<cudaStream_t>(stream));
}

diffqkv_status diffqkv_combine(const float* o_partial, const float* lse_partial, int32_t batch, int32_t n_q,
                               int32_t d_v, int32_t num_splits, diffqkv_dtype out_dtype, void* out, float* lse,
                               void* stream) {
  if (!o_partial || !lse_partial || !out) return DIFFQKV_ERR_INVALID_ARG;
  if (batch < 0 || n_q <= 0 || d_v <= 0 || num_splits <= 0) return DIFFQKV_ERR_INVALID_ARG;
  if (out_dtype != DIFFQKV_BF16 && out_dtype != DIFFQKV_F32) return DIFFQKV_ERR_INVALID_ARG;
  if (num_splits > kMaxSplits) return DIFFQKV_ERR_UNSUPPORTED;
  if ((long long)batch * n_q > 0x7fffffffLL) return DIFFQKV_ERR_UNSUPPORTED;
  cudaError_t err = launch_combine(o_partial, lse_partial, batch * n_q, d_v, num_splits, out_dtype, out, lse,
                                   static_cast<cudaStream_t>(stream));
  return err == cudaSuccess ? DIFFQKV_OK : DIFFQKV_ERR_CUDA;
}

static std::atomic<int> g_last_prefill_kernel{0};  // 0 none yet, 1 generic, 2 tensor-core (for tests)

diffqkv_status diffqkv_prefill(const void* q, const void* k_new, const void* v_new, int32_t q_len,
                               const diffqkv_cache* cache, const diffqkv_shape* shape, void* out, float* lse,
                               int32_t* dev_status, void* stream) {
  diffqkv_status st = check_shape(shape);
  if (st != DIFFQKV_OK) return st;
  if (!q || !k_new || !v_new || !out || q_len < 0) return DIFFQKV_ERR_INVALID_ARG;
  st = check_cache(cache, shape);
  if (st != DIFFQKV_OK) return st;
  if (!aligned16(q) || !aligned16(k_new) || !aligned16(v_new) || !aligned16(out)) return DIFFQKV_ERR_ALIGNMENT;
  if (q_len > cache->max_seqlen) return DIFFQKV_ERR_INVALID_ARG;
  if (shape->batch == 0 || q_len == 0) return DIFFQKV_OK;
  cudaStream_t st_ = static_cast<cudaStream_t>(stream);
  int box_tok = 0;
  cudaError_t err = cudaErrorNotSupported;
  if (prefill_supported(*shape, *cache, &box_tok))  // bf16, d 128: cache update + tensor-core attention
    err = launch_prefill(q, k_new, v_new, q_len, *cache, *shape, box_tok, out, lse, dev_status, st_);
  if (err == cudaErrorNotSupported) {  // everything else: the same two steps on the generic kernels
    err = launch_cache_append(k_new, v_new, q_len, *cache, *shape, dev_status, st_);
    if (err != cudaSuccess) return DIFFQKV_ERR_CUDA;
    DecodeParams p;
    p.q = q;
    p.cache = view_of(cache);
    p.batch = shape->batch; p.n_q = shape->n_q; p.n_k = shape->n_k; p.n_v = shape->n_v;
    p.d_qk = shape->d_qk; p.d_v = shape->d_v;
    p.scale_log2 = shape->scale * kLog2e;
    p.chunk = 0; p.splits = 1;
    p.o_partial = nullptr; p.lse_partial = nullptr;
    p.dev_status = dev_status;
    err = launch_prefill_generic(p, shape->dtype, q_len, out, shape->out_dtype == DIFFQKV_F32, lse, st_);
    g_last_prefill_kernel = 1;
  } else {
    g_last_prefill_kernel = 2;
  }
  if (err == cudaErrorNotSupported) return DIFFQKV_ERR_UNSUPPORTED;
  return err == cudaSuccess ? DIFFQKV_OK : DIFFQKV_ERR_CUDA;
}

int32_t diffqkv_last_prefill_kernel(void) { return g_last_prefill_kernel; }

size_t diffqkv_augq_workspace_bytes(int64_t T, int32_t d_q0, int32_t d_aug) {
  if (T < 0 || d_q0 <= 0 || d_aug <= 0) return 0;
  return augq_workspace_bytes(T, d_q0, d_aug);
}

static diffqkv_status check_rope(const float* cos, const float* sin, int32_t head_dim, int32_t d_out) {
  if (!cos && !sin) return DIFFQKV_OK;
  if (!cos || !sin) return DIFFQKV_ERR_INVALID_ARG;
  if (head_dim != 64 && head_dim != 128) return DIFFQKV_ERR_UNSUPPORTED;
  if (d_out % head_dim != 0) return DIFFQKV_ERR_INVALID_ARG;
  if (!aligned16(cos) || !aligned16(sin)) return DIFFQKV_ERR_ALIGNMENT;
  return DIFFQKV_OK;
}

diffqkv_status diffqkv_augq_rope(const void* h, const void* W_Q, const void* W_gate, const void* W_up,
                                 const void* W_down, int64_t T, int32_t d_model, int32_t d_q0, int32_t d_aug,
                                 int32_t d_out, int32_t head_dim, const float* cos, const float* sin, void* workspace,
                                 size_t workspace_bytes, void* q_out, int32_t* dev_status, void* stream) {
  if (!h || !W_Q || !W_gate || !W_up || !W_down || !q_out) return DIFFQKV_ERR_INVALID_ARG;
  if (T < 0 || d_model <= 0 || d_q0 <= 0 || d_aug <= 0 || d_out <= 0) return DIFFQKV_ERR_INVALID_ARG;
  if (T > 0x7fffff00LL) return DIFFQKV_ERR_UNSUPPORTED;
  if (d_model % 128 != 0 || d_q0 % 128 != 0 || d_aug % 128 != 0 || d_out % 128 != 0) return DIFFQKV_ERR_UNSUPPORTED;
  const diffqkv_status rs = check_rope(cos, sin, head_dim, d_out);
  if (rs != DIFFQKV_OK) return rs;
  const void* ptrs[6] = {h, W_Q, W_gate, W_up, W_down, q_out};
  for (const void* ptr : ptrs)
    if (!aligned16(ptr)) return DIFFQKV_ERR_ALIGNMENT;
  if (T == 0) return DIFFQKV_OK;
  if (!workspace || workspace_bytes < augq_workspace_bytes(T, d_q0, d_aug)) return DIFFQKV_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return DIFFQKV_ERR_ALIGNMENT;
  const cudaError_t err = launch_augq(h, W_Q, W_gate, W_up, W_down, T, d_model, d_q0, d_aug, d_out, workspace, q_out,
                                      dev_status, static_cast<cudaStream_t>(stream), cos, sin, head_dim);
  if (err == cudaErrorNotSupported) return DIFFQKV_ERR_UNSUPPORTED;
  return err == cudaSuccess ? DIFFQKV_OK : DIFFQKV_ERR_CUDA;
}

size_t diffqkv_decode_frontend_workspace_bytes(const diffqkv_shape* shape, int32_t d_aug) {
  if (!shape || check_shape(shape) != DIFFQKV_OK || d_aug <= 0) return 0;
  return decode_frontend_workspace_bytes(*shape, d_aug);
}

diffqkv_status diffqkv_decode_frontend(const void* h, const void* W_Q, const void* W_gate, const void* W_up,
                                       const void* W_down, const void* W_K, const void* W_V, int32_t d_model,
                                       int32_t d_aug, const float* cos, const float* sin, const diffqkv_cache* cache,
                                       const diffqkv_shape* shape, void* workspace, size_t workspace_bytes, void* q_out,
                                       int32_t* dev_status, void* stream) {
  diffqkv_status st = check_shape(shape);
  if (st != DIFFQKV_OK) return st;
  if (!h || !W_Q || !W_gate || !W_up || !W_down || !W_K || !W_V || !q_out) return DIFFQKV_ERR_INVALID_ARG;
  if (d_model <= 0 || d_aug <= 0) return DIFFQKV_ERR_INVALID_ARG;
  if (shape->dtype != DIFFQKV_BF16) return DIFFQKV_ERR_UNSUPPORTED;
  st = check_cache(cache, shape);
  if (st != DIFFQKV_OK) return st;
  const int d_q0 = shape->n_q * shape->d_qk;
  if (d_model % 128 != 0 || d_aug % 128 != 0 || d_q0 % 128 != 0) return DIFFQKV_ERR_UNSUPPORTED;
  if ((shape->n_k * shape->d_qk) % 16 != 0 || (shape->n_v * shape->d_v) % 16 != 0) return DIFFQKV_ERR_UNSUPPORTED;
  const diffqkv_status rs = check_rope(cos, sin, shape->d_qk, d_q0);
  if (rs != DIFFQKV_OK) return rs;
  const void* ptrs[8] = {h, W_Q, W_gate, W_up, W_down, W_K, W_V, q_out};
  for (const void* ptr : ptrs)
    if (!aligned16(ptr)) return DIFFQKV_ERR_ALIGNMENT;
  if (shape->batch == 0) return DIFFQKV_OK;
  if (!workspace || workspace_bytes < decode_frontend_workspace_bytes(*shape, d_aug)) return DIFFQKV_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return DIFFQKV_ERR_ALIGNMENT;
  const cudaError_t err = launch_decode_frontend(h, W_Q, W_gate, W_up, W_down, W_K, W_V, d_model, d_aug, cos, sin,
                                                 *cache, view_of(cache), *shape, workspace, q_out, dev_status,
                                                 static_cast<cudaStream_t>(stream));
  if (err == cudaErrorNotSupported) return DIFFQKV_ERR_UNSUPPORTED;
  return err == cudaSuccess ? DIFFQKV_OK : DIFFQKV_ERR_CUDA;
}

diffqkv_status diffqkv_augq(const void* h, const void* W_Q, const void* W_gate, const void* W_up, const void* W_down,
                            int64_t T, int32_t d_model, int32_t d_q0, int32_t d_aug, int32_t d_out, void* workspace,
                            size_t workspace_bytes, void* q_out, int32_t* dev_status, void* stream) {
  return diffqkv_augq_rope(h, W_Q, W_gate, W_up, W_down, T, d_model, d_q0, d_aug, d_out, 0, nullptr, nullptr,
                           workspace, workspace_bytes, q_out, dev_status, stream);
}

diffqkv_status diffqkv_project(const void* x, const void* W, int64_t T, int32_t d_in, int32_t d_out, int32_t head_dim,
                               const float* cos, const float* sin, void* y, int32_t* dev_status, void* stream) {
  if (!x || !W || !y) return DIFFQKV_ERR_INVALID_ARG;
  if (T < 0 || d_in <= 0 || d_out <= 0) return DIFFQKV_ERR_INVALID_ARG;
  if (T > 0x7fffff00LL) return DIFFQKV_ERR_UNSUPPORTED;
  if (d_in % 128 != 0 || d_out % 128 != 0) return DIFFQKV_ERR_UNSUPPORTED;
  const diffqkv_status rs = check_rope(cos, sin, head_dim, d_out);
  if (rs != DIFFQKV_OK) return rs;
  if (!aligned16(x) || !aligned16(W) || !aligned16(y)) return DIFFQKV_ERR_ALIGNMENT;
  if (T == 0) return DIFFQKV_OK;
  const cudaError_t err = launch_project(x, W, T, d_in, d_out, y, dev_status, static_cast<cudaStream_t>(stream), cos,
                                         sin, head_dim);
  if (err == cudaErrorNotSupported) return DIFFQKV_ERR_UNSUPPORTED;
  return err == cudaSuccess ? DIFFQKV_OK : DIFFQKV_ERR_CUDA;
}

diffqkv_status diffqkv_cache_append(const void* k_new, const void* v_new, int32_t q_len, const diffqkv_cache* cache,
                                    const diffqkv_shape* shape, int32_t* dev_status, void* stream) {
  diffqkv_status st = check_shape(shape);
  if (st != DIFFQKV_OK) return st;
  if (!k_new || !v_new || q_len < 0) return DIFFQKV_ERR_INVALID_ARG;
  st = check_cache(cache, shape);
  if (st != DIFFQKV_OK) return st;
  if (!aligned16(k_new) || !aligned16(v_new)) return DIFFQKV_ERR_ALIGNMENT;
  if (q_len > cache->max_seqlen) return DIFFQKV_ERR_INVALID_ARG;
  if (shape->batch == 0 || q_len == 0) return DIFFQKV_OK;
  const cudaError_t err = launch_cache_append(k_new, v_new, q_len, *cache, *shape, dev_status,
                                              static_cast<cudaStream_t>(stream));
  return err == cudaSuccess ? DIFFQKV_OK : DIFFQKV_ERR_CUDA;
}

diffqkv_status diffqkv_fold_k_up(const void* q, const void* W_kup, int64_t T, int32_t n_q, int32_t n_k, int32_t d_q,
                                 int32_t d_k, void* q_out, void* stream) {
  if (!q || !W_kup || !q_out) return DIFFQKV_ERR_INVALID_ARG;
  if (T < 0 || n_q <= 0 || n_k <= 0 || d_q <= 0 || d_k <= 0 || n_q % n_k != 0) return DIFFQKV_ERR_INVALID_ARG;
  if (T > 0x7fffffffLL) return DIFFQKV_ERR_UNSUPPORTED;
  if (T == 0) return DIFFQKV_OK;
  const cudaError_t err = launch_fold_kup(q, W_kup, T, n_q, n_k, d_q, d_k, q_out, static_cast<cudaStream_t>(stream));
  if (err == cudaErrorNotSupported) return DIFFQKV_ERR_UNSUPPORTED;
  return err == cudaSuccess ? DIFFQKV_OK : DIFFQKV_ERR_CUDA;
}

size_t diffqkv_decode_topk_workspace_bytes(const diffqkv_shape* shape, int32_t max_seqlen, int32_t topk) {
  if (check_shape(shape) != DIFFQKV_OK || max_seqlen < 0 || topk < 1) return 0;
  return topk_decode_workspace_bytes(*shape, max_seqlen, topk);
}

diffqkv_status diffqkv_decode_topk_ids(const void* q, const diffqkv_cache* cache, const diffqkv_shape* shape,
                                       int32_t topk, void* workspace, size_t workspace_bytes, void* out, float* lse,
                                       int32_t* kept_ids, int32_t* dev_status, void* stream) {
  diffqkv_status st = check_shape(shape);
  if (st != DIFFQKV_OK) return st;
  if (!q || !out || topk < 1) return DIFFQKV_ERR_INVALID_ARG;
  st = check_cache(cache, shape);
  if (st != DIFFQKV_OK) return st;
  if (!aligned16(q) || !aligned16(out)) return DIFFQKV_ERR_ALIGNMENT;
  if (shape->batch == 0) return DIFFQKV_OK;
  int box_tok = 0;
  if (!topk_decode_supported(*shape, *cache, topk, &box_tok)) return DIFFQKV_ERR_UNSUPPORTED;
  if (!workspace || workspace_bytes < topk_decode_workspace_bytes(*shape, cache->max_seqlen, topk)) return DIFFQKV_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return DIFFQKV_ERR_ALIGNMENT;
  const cudaError_t err = launch_decode_topk(q, *cache, *shape, topk, box_tok, workspace, out, lse, dev_status,
                                             static_cast<cudaStream_t>(stream), kept_ids);
  if (err == cudaErrorNotSupported) return DIFFQKV_ERR_UNSUPPORTED;
  return err == cudaSuccess ? DIFFQKV_OK : DIFFQKV_ERR_CUDA;
}

diffqkv_status diffqkv_decode_topk(const void* q, const diffqkv_cache* cache, const diffqkv_shape* shape, int32_t topk,
                                   void* workspace, size_t workspace_bytes, void* out, float* lse, int32_t* dev_status,
                                   void* stream) {
  return diffqkv_decode_topk_ids(q, cache, shape, topk, workspace, workspace_bytes, out, lse, nullptr, dev_status, stream);
}

const char* diffqkv_status_string(diffqkv_status status) {
  switch (status) {
    case DIFFQKV_OK: return "ok";
    case DIFFQKV_ERR_INVALID_ARG: return "invalid argument";
    case DIFFQKV_ERR_UNSUPPORTED: return "unsupported shape or dtype";
    case DIFFQKV_ERR_ALIGNMENT: return "pointer or stride alignment";
    case DIFFQKV_ERR_WORKSPACE: return "workspace missing or too small";
    case DIFFQKV_ERR_CUDA: return "CUDA call failed";
    case DIFFQKV_ERR_TIMEOUT: return "device wait ran out";
    case DIFFQKV_ERR_INDEX: return "page id out of range";
  }
  return "unknown status";
}

void diffqkv_profile_split_events(void* before_split, void* after_split) {
  g_ev_before.store(static_cast<cudaEvent_t>(before_split));
  g_ev_after.store(static_cast<cudaEvent_t>(after_split));
}

int64_t diffqkv_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
