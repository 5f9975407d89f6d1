// Generic DiffQKV attention kernels: plain fp32 FMAs, any head counts, any strides, fp32 or bf16 storage.  They are
// the path for the fp32 mode and for shapes the TMA / tensor-core kernels do not take.  Decode: one block per (split,
// query head, sequence); causal prefill: one block per (query row, query head, sequence).  The head map is Eq. (idx)
// of the paper.
#include "common.cuh"

namespace diffqkv {
namespace {

constexpr int kThreads = 128;
constexpr int kMaxAccPerThread = 4;  // d_v <= kThreads * kMaxAccPerThread

template <typename T>
struct Vec;  // 16-byte vector of T
template <>
struct Vec<float> {
  static constexpr int N = 4;
  __device__ static void load(const float* p, float (&x)[4]) {
    float4 v = *reinterpret_cast<const float4*>(p);
    x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
  }
};
template <>
struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void load(const __nv_bfloat16* p, float (&x)[8]) {
    uint4 v = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[2 * i] = __uint_as_float(w[i] << 16);
      x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
};

__device__ __forceinline__ float block_reduce(float v, bool is_max, float* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    float w = __shfl_xor_sync(0xffffffffu, v, o);
    v = is_max ? fmaxf(v, w) : v + w;
  }
  __syncthreads();  // protects `red` against the previous use
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = red[0];
#pragma unroll
  for (int i = 1; i < kThreads / 32; ++i) r = is_max ? fmaxf(r, red[i]) : r + red[i];
  return r;
}

// Shared memory of one block.
struct GenericSmem {
  float p_s[kThreads];
  long long vrow_s[kThreads];
  float red[kThreads / 32];
};

// Attention of query head h of sequence b over cached tokens [t0, t1), t0 < t1: running maximum and sum (base-2
// domain) and the un-normalised output channels tid, tid + kThreads, ... of this thread.  q_s holds the query times
// scale * log2(e).  All threads of the block call it.
template <typename T>
__device__ void attend_range(const DecodeParams& p, int b, int h, int t0, int t1, const float* q_s, GenericSmem& sm,
                             float& m_run, float& l_run, float (&acc)[kMaxAccPerThread]) {
  const int tid = threadIdx.x;
  const CacheView& c = p.cache;
  const int hk = (int)(((long long)h * p.n_k) / p.n_q);  // Eq. (idx)
  const int hv = (int)(((long long)h * p.n_v) / p.n_q);
  const T* kbase = reinterpret_cast<const T*>(c.k);
  const T* vbase = reinterpret_cast<const T*>(c.v);
  m_run = -INFINITY;
  l_run = 0.f;
#pragma unroll
  for (int i = 0; i < kMaxAccPerThread; ++i) acc[i] = 0.f;

  for (int base = t0; base < t1; base += kThreads) {
    const int j = base + tid;
    float sc = -INFINITY;
    long long vrow = -1;
    if (j < t1) {
      long long blk = b, slot = j;
      bool ok = true;
      if (c.page_table) {
        const int page = c.page_table[(long long)b * c.max_pages_per_seq + j / c.page_size];
        slot = j % c.page_size;
        blk = page;
        if (page < 0 || page >= c.num_blocks) {
          ok = false;
          report(p.dev_status, DIFFQKV_ERR_INDEX);
        }
      }
      if (ok) {
        const T* krow = kbase + blk * c.k_sb + (long long)hk * c.k_sh + slot * c.k_st;
        vrow = blk * c.v_sb + (long long)hv * c.v_sh + slot * c.v_st;
        float dot = 0.f;
        for (int ch = 0; ch < p.d_qk; ch += Vec<T>::N) {
          float x[Vec<T>::N];
          Vec<T>::load(krow + ch, x);
#pragma unroll
          for (int e = 0; e < Vec<T>::N; ++e) dot = fmaf(q_s[ch + e], x[e], dot);
        }
        sc = dot;
      }
    }
    const float m_tile = block_reduce(sc, true, sm.red);
    const float m_new = fmaxf(m_run, m_tile);
    float alpha = 0.f, pj = 0.f;
    if (m_new != -INFINITY) {  // all tokens of the tile may have been rejected
      alpha = exp2f(m_run - m_new);
      pj = exp2f(sc - m_new);
    }
    sm.p_s[tid] = pj;
    sm.vrow_s[tid] = vrow;
    const float l_tile = block_reduce(pj, false, sm.red);  // also publishes p_s / vrow_s
    l_run = l_run * alpha + l_tile;
    m_run = m_new;
    const int nt = min(kThreads, t1 - base);
#pragma unroll
    for (int i = 0; i < kMaxAccPerThread; ++i) {
      const int ch = tid + i * kThreads;
      if (ch < p.d_v) {
        float a = acc[i] * alpha;
        for (int jj = 0; jj < nt; ++jj) {
          const long long r = sm.vrow_s[jj];
          if (r >= 0) a = fmaf(sm.p_s[jj], to_float(vbase[r + ch]), a);
        }
        acc[i] = a;
      }
    }
    __syncthreads();
  }
}

template <typename T>
__global__ void __launch_bounds__(kThreads) decode_generic_kernel(DecodeParams p) {
  extern __shared__ float q_s[];  // [d_qk]
  __shared__ GenericSmem sm;

  const int s = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x;
  const CacheView& c = p.cache;
  const int len = min(c.seqlens[b], c.max_seqlen);
  const int t0 = s * p.chunk;
  const int t1 = min(len, t0 + p.chunk);
  const long long row_id = ((long long)b * p.n_q + h) * p.splits + s;
  float* o_out = p.o_partial + row_id * p.d_v;
  if (t0 >= t1) {  // empty split: the combine step skips -inf entries
    if (tid == 0) p.lse_partial[row_id] = -INFINITY;
    return;
  }
  const T* q = reinterpret_cast<const T*>(p.q) + ((long long)b * p.n_q + h) * p.d_qk;
  for (int i = tid; i < p.d_qk; i += kThreads) q_s[i] = to_float(q[i]) * p.scale_log2;
  __syncthreads();

  float m_run, l_run, acc[kMaxAccPerThread];
  attend_range<T>(p, b, h, t0, t1, q_s, sm, m_run, l_run, acc);
  const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
#pragma unroll
  for (int i = 0; i < kMaxAccPerThread; ++i) {
    const int ch = tid + i * kThreads;
    if (ch < p.d_v) o_out[ch] = acc[i] * inv;
  }
  if (tid == 0) p.lse_partial[row_id] = l_run > 0.f ? (m_run + log2f(l_run)) * kLn2 : -INFINITY;
}

// Causal prefill on the same arithmetic: one block per (query row i, query head, sequence); row i of sequence b
// attends cached tokens 0 .. past_b + i (the new rows are in the cache already) and writes its normalised output.
// The path for fp32 storage and for head dimensions the tensor-core prefill kernel does not take.
template <typename T>
__global__ void __launch_bounds__(kThreads) prefill_generic_kernel(DecodeParams p, int q_len, void* out, int out_is_f32,
                                                                  float* lse) {
  extern __shared__ float q_s[];  // [d_qk]
  __shared__ GenericSmem sm;

  const int i = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x;
  const CacheView& c = p.cache;
  const int past = min(max(c.seqlens[b], 0), c.max_seqlen);
  const int t1 = min(past + i + 1, c.max_seqlen);  // rows past the cache's end see what fits
  const long long row = ((long long)b * q_len + i) * p.n_q + h;
  const T* q = reinterpret_cast<const T*>(p.q) + row * p.d_qk;
  for (int e = tid; e < p.d_qk; e += kThreads) q_s[e] = to_float(q[e]) * p.scale_log2;
  __syncthreads();

  float m_run = -INFINITY, l_run = 0.f, acc[kMaxAccPerThread];
#pragma unroll
  for (int e = 0; e < kMaxAccPerThread; ++e) acc[e] = 0.f;
  if (t1 > 0) attend_range<T>(p, b, h, 0, t1, q_s, sm, m_run, l_run, acc);
  const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
#pragma unroll
  for (int e = 0; e < kMaxAccPerThread; ++e) {
    const int ch = tid + e * kThreads;
    if (ch < p.d_v) {
      if (out_is_f32) reinterpret_cast<float*>(out)[row * p.d_v + ch] = acc[e] * inv;
      else reinterpret_cast<__nv_bfloat16*>(out)[row * p.d_v + ch] = __float2bfloat16_rn(acc[e] * inv);
    }
  }
  if (lse && tid == 0) lse[row] = l_run > 0.f ? (m_run + log2f(l_run)) * kLn2 : -INFINITY;
}

}  // namespace

cudaError_t launch_decode_generic(const DecodeParams& p, diffqkv_dtype dtype, cudaStream_t stream) {
  dim3 grid(p.splits, p.n_q, p.batch);
  const size_t smem = sizeof(float) * p.d_qk;
  if (dtype == DIFFQKV_F32)
    decode_generic_kernel<float><<<grid, kThreads, smem, stream>>>(p);
  else
    decode_generic_kernel<__nv_bfloat16><<<grid, kThreads, smem, stream>>>(p);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_prefill_generic(const DecodeParams& p, diffqkv_dtype dtype, int q_len, void* out, int out_is_f32,
                                   float* lse, cudaStream_t stream) {
  if (q_len > 0x7fffffff || p.n_q > 65535 || p.batch > 65535) return cudaErrorNotSupported;
  dim3 grid(q_len, p.n_q, p.batch);
  const size_t smem = sizeof(float) * p.d_qk;
  if (dtype == DIFFQKV_F32)
    prefill_generic_kernel<float><<<grid, kThreads, smem, stream>>>(p, q_len, out, out_is_f32, lse);
  else
    prefill_generic_kernel<__nv_bfloat16><<<grid, kThreads, smem, stream>>>(p, q_len, out, out_is_f32, lse);
  count_launch();
  return cudaGetLastError();
}

}  // namespace diffqkv
