// Combine kernel: log-sum-exp merge of the per-split partial results of the decode kernels
// (paper Section 3.2: the combine kernel assembles the output chunks).
#include "common.cuh"

namespace diffqkv {
namespace {

constexpr int kCombineThreads = 128;

// One block per output row (sequence, query head).  Every thread first scans the row's S
// log-sum-exps (a broadcast read), then threads own channels and accumulate the weighted partials.
template <typename OutT>
__global__ void __launch_bounds__(kCombineThreads)
combine_kernel(const float* __restrict__ o_partial, const float* __restrict__ lse_partial, int d_v, int splits,
               OutT* __restrict__ out, float* __restrict__ lse) {
  extern __shared__ float w_s[];  // [splits] weights exp(lse_s - lse)
  const long long row = blockIdx.x;
  const float* lp = lse_partial + row * splits;
  float m = -INFINITY;
  for (int s = threadIdx.x; s < splits; s += kCombineThreads) m = fmaxf(m, lp[s]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  __shared__ float red[kCombineThreads / 32];
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
  __syncthreads();
  m = red[0];
#pragma unroll
  for (int i = 1; i < kCombineThreads / 32; ++i) m = fmaxf(m, red[i]);
  OutT* orow = out + row * d_v;
  if (m == -INFINITY) {  // every split empty
    for (int ch = threadIdx.x; ch < d_v; ch += kCombineThreads) store_out(orow + ch, 0.f);
    if (lse && threadIdx.x == 0) lse[row] = -INFINITY;
    return;
  }
  float sum = 0.f;
  for (int s = threadIdx.x; s < splits; s += kCombineThreads) {
    const float e = lp[s] == -INFINITY ? 0.f : exp2f((lp[s] - m) * kLog2e);
    w_s[s] = e;
    sum += e;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  __syncthreads();  // red[] reads above are done
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sum;
  __syncthreads();  // publishes red[] and w_s[]
  sum = red[0];
#pragma unroll
  for (int i = 1; i < kCombineThreads / 32; ++i) sum += red[i];
  const float inv = 1.f / sum;
  const float* op = o_partial + row * (long long)splits * d_v;
  for (int ch = threadIdx.x; ch < d_v; ch += kCombineThreads) {
    float a = 0.f;
    for (int s = 0; s < splits; ++s) {
      const float w = w_s[s];
      if (w != 0.f) a = fmaf(w, op[(long long)s * d_v + ch], a);
    }
    store_out(orow + ch, a * inv);
  }
  if (lse && threadIdx.x == 0) lse[row] = m + logf(sum);
}

}  // namespace

cudaError_t launch_combine(const float* o_partial, const float* lse_partial, int rows, int d_v, int splits,
                           diffqkv_dtype out_dtype, void* out, float* lse, cudaStream_t stream) {
  if (rows == 0) return cudaSuccess;
  const size_t smem = sizeof(float) * splits;
  if (out_dtype == DIFFQKV_F32)
    combine_kernel<float><<<rows, kCombineThreads, smem, stream>>>(o_partial, lse_partial, d_v, splits,
                                                                   reinterpret_cast<float*>(out), lse);
  else
    combine_kernel<__nv_bfloat16><<<rows, kCombineThreads, smem, stream>>>(
        o_partial, lse_partial, d_v, splits, reinterpret_cast<__nv_bfloat16*>(out), lse);
  count_launch();
  return cudaGetLastError();
}

}  // namespace diffqkv
