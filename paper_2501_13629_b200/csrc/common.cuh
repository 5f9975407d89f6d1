// Shared device/host helpers of libdiffqkv (CUDA side only; the CPU oracle shares nothing with this).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "diffqkv.h"

namespace diffqkv {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Host-side decode plan: the sequence axis is cut into chunks of `chunk` tokens (a multiple of
// kChunkQuantum); sequence b uses ceil(len_b / chunk) of the `splits` partial slots.
constexpr int kChunkQuantum = 64;
struct DecodePlan {
  int chunk;
  int splits;
};
DecodePlan plan_decode(const diffqkv_shape& shape, int max_seqlen, int num_splits);

struct CacheView {  // device copy of the addressing part of diffqkv_cache
  const void* k;
  const void* v;
  long long k_sb, k_sh, k_st;
  long long v_sb, v_sh, v_st;
  const int* seqlens;
  const int* page_table;
  int page_size, max_pages_per_seq, num_blocks, max_seqlen;
};

struct DecodeParams {
  const void* q;
  CacheView cache;
  int batch, n_q, n_k, n_v, d_qk, d_v;
  float scale_log2;  // scale * log2(e): scores are kept in the base-2 domain
  int chunk, splits;
  float* o_partial;    // [batch, n_q, splits, d_v]
  float* lse_partial;  // [batch, n_q, splits]   natural log
  int* dev_status;
};

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ void store_out(float* p, float x) { *p = x; }
__device__ __forceinline__ void store_out(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

// Device-side conditions are reported as bit (1 << diffqkv_status) so that several can coexist.
__device__ __forceinline__ void report(int* dev_status, int code) {
  if (dev_status) atomicOr(dev_status, 1 << code);
}

// Launchers (defined next to their kernels).
cudaError_t launch_decode_generic(const DecodeParams& p, diffqkv_dtype dtype, cudaStream_t stream);
cudaError_t launch_prefill_generic(const DecodeParams& p, diffqkv_dtype dtype, int q_len, void* out, int out_is_f32,
                                   float* lse, cudaStream_t stream);
cudaError_t launch_combine(const float* o_partial, const float* lse_partial, int rows, int d_v, int splits,
                           diffqkv_dtype out_dtype, void* out, float* lse, cudaStream_t stream);
void count_launch(int n = 1);
void set_decode_per_head_only(int on);  // test hook: the generic decode never takes the unit kernel

// Linear layers for at most kSkinnyMaxRows rows of x (weight-streaming kernel, linear_skinny.cu); same operands as the
// tensor-core GEMM of augq.cu: C[M, N] = A[M, K] . B0[N, K]^T, with B1 silu(A.B0^T) * (A.B1^T), with rope_cos/rope_sin
// the rotate-half rotary embedding per head of head_dim channels.
constexpr int kSkinnyMaxRows = 64;
void set_force_tensor_gemm(int on);
cudaError_t launch_qkv_skinny(const void* h, const void* W_Q, void* x, int d_q0, const void* W_K, const void* W_V,
                              long long M, int K, const float* rope_cos, const float* rope_sin, const CacheView& cache,
                              int n_k, int n_v, int d_qk, int d_v, int* dev_status, cudaStream_t stream);
// Everything a decode step computes from the hidden states h [batch, d_model]: q_out = rope(aug-Q(h)), and the new
// token's k = rope(h W_K^T), v = h W_V^T written into the cache at position seqlens[b] (augq.cu).
size_t decode_frontend_workspace_bytes(const diffqkv_shape& s, int d_aug);
cudaError_t launch_decode_frontend(const void* h, const void* W_Q, const void* W_gate, const void* W_up,
                                   const void* W_down, const void* W_K, const void* W_V, int d_model, int d_aug,
                                   const float* rope_cos, const float* rope_sin, const diffqkv_cache& c,
                                   const CacheView& view, const diffqkv_shape& s, void* workspace, void* q_out,
                                   int* dev_status, cudaStream_t stream);
bool linear_skinny_supported(long long M, int N, int K, bool dual, int head_dim, bool rotary);
cudaError_t launch_linear_skinny(const void* A, const void* B0, const void* B1, void* C, long long M, int N, int K,
                                 int* dev_status, cudaStream_t stream, const float* rope_cos, const float* rope_sin,
                                 int head_dim);
void profile_after_split(cudaStream_t stream);  // records the benchmark hook's second event, if armed

// TMA decode path (decode_tma.cu): persistent blocks over a flat (sequence, unit, tile) list.
struct TmaPlan {
  int U, kpu, vpu;   // query heads, K heads and V heads per unit
  int k_shift, v_shift;  // 2^shift neighbouring units read the same K (V) head (more than 8 query heads per head)
  int box_tok;       // tokens per TMA box
  int stages, grid, smem;
  long long slots;   // partial-result slots: grid + batch * units
  int reserve, reserve_auto;  // tail reserve per block in tiles (0 = none); auto: also at most a sixth of a block's share
  int cluster;       // 0, or the blocks per (sequence, unit) row that merge through each other's shared memory
};
bool tma_decode_supported(const diffqkv_shape& s, const diffqkv_cache& c, TmaPlan* plan);
size_t tma_decode_workspace_bytes(const diffqkv_shape& s, const TmaPlan& plan);
cudaError_t launch_decode_tma(const void* q, const diffqkv_cache& c, const diffqkv_shape& s, const TmaPlan& plan,
                              void* workspace, void* out, float* lse, int* dev_status, cudaStream_t stream);
void set_tma_max_blocks(int n);
void set_tma_tail_reserve(int n);
void set_tma_cluster_mode(int mode);  // -1 automatic, 0 never, 1 whenever the shape allows
void set_tma_debug_timeout(long long wait_limit_ns, long long skip_tile);

// Augmented-Q projection (augq.cu): three tcgen05 GEMMs, the gate/up pair fused with its silu-gate epilogue.
size_t augq_workspace_bytes(long long T, int d_q0, int d_aug);
cudaError_t launch_augq(const void* h, const void* W_Q, const void* W_gate, const void* W_up, const void* W_down,
                        long long T, int d_model, int d_q0, int d_aug, int d_out, void* workspace, void* q_out,
                        int* dev_status, cudaStream_t stream, const float* rope_cos = nullptr,
                        const float* rope_sin = nullptr, int head_dim = 0);
cudaError_t launch_project(const void* x, const void* W, long long T, int d_in, int d_out, void* y, int* dev_status,
                           cudaStream_t stream, const float* rope_cos, const float* rope_sin, int head_dim);


// Causal prefill (prefill.cu): cache update kernel, then tcgen05 attention over the cache.
bool prefill_supported(const diffqkv_shape& s, const diffqkv_cache& c, int* box_tok);
cudaError_t launch_cache_append(const void* k_new, const void* v_new, int q_len, const diffqkv_cache& c,
                                const diffqkv_shape& s, int* dev_status, cudaStream_t stream);
cudaError_t launch_prefill(const void* q, const void* k_new, const void* v_new, int q_len, const diffqkv_cache& c,
                           const diffqkv_shape& s, int box_tok, void* out, float* lse, int* dev_status,
                           cudaStream_t stream);


// Queries folded through the K feed-forward layer (kup.cu): q' = W_kup[hk]^T q per query head.
cudaError_t launch_fold_kup(const void* q, const void* W_kup, long long T, int n_q, int n_k, int d_q, int d_k,
                            void* q_out, cudaStream_t stream);

// Selective V fetching (decode_topk.cu): K-only score pass, then top-k selection and V gather per query head.
bool topk_decode_supported(const diffqkv_shape& s, const diffqkv_cache& c, int topk, int* box_tok);
size_t topk_decode_workspace_bytes(const diffqkv_shape& s, int max_seqlen, int topk);
void set_topk_general_only(int on);
cudaError_t launch_decode_topk(const void* q, const diffqkv_cache& c, const diffqkv_shape& s, int topk, int box_tok,
                               void* workspace, void* out, float* lse, int* dev_status, cudaStream_t stream,
                               int* kept_ids = nullptr);

}  // namespace diffqkv
