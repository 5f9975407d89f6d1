// Generic split-sequence DiffQKV decode kernel: plain fp32 FMAs, any head counts, any strides,
// fp32 or bf16 storage.  It is the path for the fp32 mode and for shapes the TMA kernel does not
// take.  One block per (split, query head, sequence); the head map is Eq. (idx) of the paper.
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

template <typename T>
__global__ void __launch_bounds__(kThreads) decode_generic_kernel(DecodeParams p) {
  extern __shared__ float q_s[];  // [d_qk]
  __shared__ float p_s[kThreads];
  __shared__ long long vrow_s[kThreads];
  __shared__ float red[kThreads / 32];

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
  const int hk = (int)(((long long)h * p.n_k) / p.n_q);  // Eq. (idx)
  const int hv = (int)(((long long)h * p.n_v) / p.n_q);
  const T* q = reinterpret_cast<const T*>(p.q) + ((long long)b * p.n_q + h) * p.d_qk;
  for (int i = tid; i < p.d_qk; i += kThreads) q_s[i] = to_float(q[i]) * p.scale_log2;
  __syncthreads();

  const T* kbase = reinterpret_cast<const T*>(c.k);
  const T* vbase = reinterpret_cast<const T*>(c.v);
  float m_run = -INFINITY, l_run = 0.f;
  float acc[kMaxAccPerThread];
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
    const float m_tile = block_reduce(sc, true, red);
    const float m_new = fmaxf(m_run, m_tile);
    float alpha = 0.f, pj = 0.f;
    if (m_new != -INFINITY) {  // all tokens of the tile may have been rejected
      alpha = exp2f(m_run - m_new);
      pj = exp2f(sc - m_new);
    }
    p_s[tid] = pj;
    vrow_s[tid] = vrow;
    const float l_tile = block_reduce(pj, false, red);  // also publishes p_s / vrow_s
    l_run = l_run * alpha + l_tile;
    m_run = m_new;
    const int nt = min(kThreads, t1 - base);
#pragma unroll
    for (int i = 0; i < kMaxAccPerThread; ++i) {
      const int ch = tid + i * kThreads;
      if (ch < p.d_v) {
        float a = acc[i] * alpha;
        for (int jj = 0; jj < nt; ++jj) {
          const long long r = vrow_s[jj];
          if (r >= 0) a = fmaf(p_s[jj], to_float(vbase[r + ch]), a);
        }
        acc[i] = a;
      }
    }
    __syncthreads();
  }
  const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
#pragma unroll
  for (int i = 0; i < kMaxAccPerThread; ++i) {
    const int ch = tid + i * kThreads;
    if (ch < p.d_v) o_out[ch] = acc[i] * inv;
  }
  if (tid == 0) p.lse_partial[row_id] = l_run > 0.f ? (m_run + log2f(l_run)) * kLn2 : -INFINITY;
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

}  // namespace diffqkv
