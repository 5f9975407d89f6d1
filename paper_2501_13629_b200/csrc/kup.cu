// Folding the K feed-forward layer into the queries (paper Section 2: when the Q and K head dimensions differ,
// "Attend" first widens K to the query width through another feed-forward layer; Observation 2: d_k = d_v / 2).
// With that layer read as linear and bias-free, W_kup[hk] of shape [d_q, d_k] per K head,
//     <q_h, W_kup[hk] k_j> = <W_kup[hk]^T q_h, k_j>,
// so the half-width cache can be scored directly by q'_h = W_kup[hk]^T q_h (width d_k) and the cached keys never
// have to be widened: one small product per query row instead of one per cached token.
#include "common.cuh"

namespace diffqkv {
namespace {

// One block per (four rows, K head hk): a thread owns an output column of one row for eight query heads of the group
// at a time, so that every weight it loads serves eight products and the queries come out of shared memory four
// channels at a time.  q [T, n_q, d_q] bf16, W [n_k, d_q, d_k] bf16, out [T, n_q, d_k] bf16; fp32 accumulation, one
// rounding.  d_q is a multiple of 4.
constexpr int kFoldRows = 4, kFoldCols = 64, kFoldHeads = 8;
__global__ void __launch_bounds__(kFoldRows * kFoldCols)
fold_kup_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ W,
                __nv_bfloat16* __restrict__ out, long long T, int n_q, int n_k, int d_q, int d_k) {
  extern __shared__ __align__(16) float qs[];  // [rows][g][d_q]
  const int g = n_q / n_k;
  const long long t0 = (long long)blockIdx.x * kFoldRows;
  const int hk = blockIdx.y;
  const int per_row = g * d_q;
  for (int i = threadIdx.x; i < kFoldRows * per_row; i += blockDim.x) {
    const long long t = t0 + i / per_row;
    qs[i] = t < T ? __bfloat162float(q[(t * n_q + (long long)hk * g) * d_q + i % per_row]) : 0.f;
  }
  __syncthreads();
  const int r = threadIdx.x / kFoldCols, cl = threadIdx.x % kFoldCols;
  const long long t = t0 + r;
  if (t >= T) return;
  const __nv_bfloat16* w = W + (long long)hk * d_q * d_k;
  for (int i = cl; i < d_k; i += kFoldCols) {
    for (int h0 = 0; h0 < g; h0 += kFoldHeads) {
      float acc[kFoldHeads];
#pragma unroll
      for (int j = 0; j < kFoldHeads; ++j) acc[j] = 0.f;
      for (int c = 0; c < d_q; c += 4) {
        float wv[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) wv[e] = __bfloat162float(w[(long long)(c + e) * d_k + i]);
#pragma unroll
        for (int j = 0; j < kFoldHeads; ++j) {
          if (h0 + j < g) {
            const float4 x = *reinterpret_cast<const float4*>(qs + (r * g + h0 + j) * d_q + c);
            acc[j] = fmaf(x.x, wv[0], fmaf(x.y, wv[1], fmaf(x.z, wv[2], fmaf(x.w, wv[3], acc[j]))));
          }
        }
      }
#pragma unroll
      for (int j = 0; j < kFoldHeads; ++j)
        if (h0 + j < g) out[(t * n_q + (long long)hk * g + h0 + j) * d_k + i] = __float2bfloat16_rn(acc[j]);
    }
  }
}

}  // namespace

cudaError_t launch_fold_kup(const void* q, const void* W_kup, long long T, int n_q, int n_k, int d_q, int d_k,
                            void* q_out, cudaStream_t stream) {
  const size_t smem = (size_t)kFoldRows * (n_q / n_k) * d_q * sizeof(float);
  if (smem > 48 * 1024 || d_q % 4 != 0 || n_k > 65535) return cudaErrorNotSupported;
  const dim3 grid((unsigned)((T + kFoldRows - 1) / kFoldRows), (unsigned)n_k);
  fold_kup_kernel<<<grid, kFoldRows * kFoldCols, smem, stream>>>(reinterpret_cast<const __nv_bfloat16*>(q),
                                                                reinterpret_cast<const __nv_bfloat16*>(W_kup),
                                                                reinterpret_cast<__nv_bfloat16*>(q_out), T, n_q, n_k,
                                                                d_q, d_k);
  count_launch();
  return cudaGetLastError();
}

}  // namespace diffqkv
