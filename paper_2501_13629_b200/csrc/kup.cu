// Folding the K feed-forward layer into the queries (paper Section 2: when the Q and K head dimensions differ,
// "Attend" first widens K to the query width through another feed-forward layer; Observation 2: d_k = d_v / 2).
// With that layer read as linear and bias-free, W_kup[hk] of shape [d_q, d_k] per K head,
//     <q_h, W_kup[hk] k_j> = <W_kup[hk]^T q_h, k_j>,
// so the half-width cache can be scored directly by q'_h = W_kup[hk]^T q_h (width d_k) and the cached keys never
// have to be widened: one small product per query row instead of one per cached token.
#include "common.cuh"

namespace diffqkv {
namespace {

// One block per (row t, K head hk): the g = n_q / n_k query heads of the group against the same matrix.
// q [T, n_q, d_q] bf16, W [n_k, d_q, d_k] bf16, out [T, n_q, d_k] bf16; fp32 accumulation, one rounding.
__global__ void __launch_bounds__(256)
fold_kup_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ W,
                __nv_bfloat16* __restrict__ out, int n_q, int n_k, int d_q, int d_k) {
  extern __shared__ float qs[];  // [g][d_q]
  const int g = n_q / n_k;
  const long long t = blockIdx.x / n_k;
  const int hk = blockIdx.x % n_k;
  const __nv_bfloat16* qrow = q + (t * n_q + (long long)hk * g) * d_q;
  for (int i = threadIdx.x; i < g * d_q; i += blockDim.x) qs[i] = __bfloat162float(qrow[i]);
  __syncthreads();
  const __nv_bfloat16* w = W + (long long)hk * d_q * d_k;
  __nv_bfloat16* orow = out + (t * n_q + (long long)hk * g) * d_k;
  for (int o = threadIdx.x; o < g * d_k; o += blockDim.x) {
    const int hh = o / d_k, i = o % d_k;
    float acc = 0.f;
    for (int c = 0; c < d_q; ++c) acc = fmaf(qs[hh * d_q + c], __bfloat162float(w[(long long)c * d_k + i]), acc);
    orow[o] = __float2bfloat16_rn(acc);
  }
}

}  // namespace

cudaError_t launch_fold_kup(const void* q, const void* W_kup, long long T, int n_q, int n_k, int d_q, int d_k,
                            void* q_out, cudaStream_t stream) {
  const size_t smem = (size_t)(n_q / n_k) * d_q * sizeof(float);
  if (smem > 48 * 1024) return cudaErrorNotSupported;
  fold_kup_kernel<<<(unsigned)(T * n_k), 256, smem, stream>>>(reinterpret_cast<const __nv_bfloat16*>(q),
                                                               reinterpret_cast<const __nv_bfloat16*>(W_kup),
                                                               reinterpret_cast<__nv_bfloat16*>(q_out), n_q, n_k, d_q,
                                                               d_k);
  count_launch();
  return cudaGetLastError();
}

}  // namespace diffqkv
