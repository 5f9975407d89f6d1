// Folding the K feed-forward layer into the queries (paper Section 2: when the Q and K head dimensions differ,
// "Attend" first widens K to the query width through another feed-forward layer; Observation 2: d_k = d_v / 2).
// With that layer read as linear and bias-free, W_kup[hk] of shape [d_q, d_k] per K head,
//     <q_h, W_kup[hk] k_j> = <W_kup[hk]^T q_h, k_j>,
// so the half-width cache can be scored directly by q'_h = W_kup[hk]^T q_h (width d_k) and the cached keys never
// have to be widened: one small product per query row instead of one per cached token.
#include <algorithm>
#include <atomic>

#include "common.cuh"
#include "ptx.cuh"

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


// The same product on the tensor cores, for the shapes a long prefill brings (bf16, d_q a multiple of 16 up to 256,
// d_k 32 / 64 / 128 and not above d_q).  For K head hk the query rows (t, u), u over the g heads of its group, form a
// [T g, d_q] matrix whose row t g + u starts at q + ((t n_q + hk g + u) d_q); the block keeps W_kup[hk] in shared
// memory and walks 128-row tiles of that matrix, one 16-row slab per warp: 16-byte loads into a padded slab, ldmatrix
// + mma.sync m16n8k16 with fp32 accumulators, one rounding, and the slab is reused to turn the accumulator fragments
// into 16-byte stores.  A slab belongs to one warp from load to store, so the tile loop needs no block barrier.
constexpr int kMmaThreads = 256, kMmaRows = 16 * (kMmaThreads / 32);
template <int DK>
__global__ void __launch_bounds__(kMmaThreads)
fold_kup_mma_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ W,
                    __nv_bfloat16* __restrict__ out, long long R, int n_q, int g, int d_q) {
  extern __shared__ __align__(16) unsigned char fold_smem[];
  const int lda = d_q + 8, ldw = DK + 8;  // +16 bytes per row keeps the eight rows of an ldmatrix on distinct banks
  __nv_bfloat16* Ws = reinterpret_cast<__nv_bfloat16*>(fold_smem);  // [d_q][ldw]
  __nv_bfloat16* As = Ws + d_q * ldw;                                // [warp][2][16][lda]
  const int hk = blockIdx.y, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const __nv_bfloat16* w = W + (long long)hk * d_q * DK;
  for (int i = threadIdx.x; i < d_q * (DK / 8); i += kMmaThreads) {
    const int r = i / (DK / 8), c = i % (DK / 8);
    *reinterpret_cast<uint4*>(Ws + r * ldw + c * 8) = __ldg(reinterpret_cast<const uint4*>(w + r * DK + c * 8));
  }
  __syncthreads();
  // Two slabs per warp: while one is multiplied and stored, cp.async fills the other with the warp's next 16 rows.
  __nv_bfloat16* slab0 = As + 2 * warp * 16 * lda;
  const int cq = d_q / 8;
  const long long tiles = (R + kMmaRows - 1) / kMmaRows;
  // Lane r < 16 works out where row r of a slab lives (one 32-bit division per slab) and the copy loops fetch that
  // by shuffle; rows past the end repeat the last one and are never stored.  The (row, chunk) a lane copies advances
  // by additions only.
  const int dr = 32 / cq, dc = 32 % cq;
  auto row_index = [&](long long r0) {
    const unsigned rr = (unsigned)min(r0 + (lane & 15), R - 1);
    const unsigned t = rr / (unsigned)g;
    return t * (unsigned)n_q + (unsigned)(hk * g) + (rr - t * (unsigned)g);
  };
  auto fetch = [&](long long tile, __nv_bfloat16* dst) {
    if (tile < tiles) {
      const unsigned mine = row_index(tile * kMmaRows + warp * 16);
      int r = lane / cq, c = lane % cq;
      for (int i = lane; i < 16 * cq; i += 32) {
        const unsigned row = __shfl_sync(0xffffffffu, mine, r);
        ptx::cp_async_16(ptx::smem_u32(dst + r * lda + c * 8), q + (long long)row * d_q + c * 8);
        r += dr, c += dc;
        if (c >= cq) c -= cq, ++r;
      }
    }
    ptx::cp_async_commit();
  };
  fetch(blockIdx.x, slab0);
  int cur = 0;
  for (long long tile = blockIdx.x; tile < tiles; tile += gridDim.x, cur ^= 1) {
    const long long r0 = tile * kMmaRows + warp * 16;
    __nv_bfloat16* Aw = slab0 + cur * 16 * lda;
    fetch(tile + gridDim.x, slab0 + (cur ^ 1) * 16 * lda);
    ptx::cp_async_wait<1>();
    __syncwarp();
    if (r0 >= R) continue;
    float acc[DK / 8][4];
#pragma unroll
    for (int n = 0; n < DK / 8; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
    for (int k0 = 0; k0 < d_q; k0 += 16) {
      uint32_t a[4];
      ptx::ldmatrix_x4(ptx::smem_u32(Aw + (lane & 15) * lda + k0 + (lane >> 4) * 8), a);
#pragma unroll
      for (int n0 = 0; n0 < DK; n0 += 16) {
        uint32_t b[4];
        ptx::ldmatrix_x4_trans(
            ptx::smem_u32(Ws + (k0 + (lane & 7) + ((lane >> 3) & 1) * 8) * ldw + n0 + (lane >> 4) * 8), b);
        ptx::mma_bf16_16816(acc[n0 / 8], a, b[0], b[1]);
        ptx::mma_bf16_16816(acc[n0 / 8 + 1], a, b[2], b[3]);
      }
    }
    __syncwarp();
#pragma unroll
    for (int n = 0; n < DK / 8; ++n) {
      const int col = n * 8 + (lane & 3) * 2;
      *reinterpret_cast<__nv_bfloat162*>(Aw + (lane >> 2) * lda + col) = __floats2bfloat162_rn(acc[n][0], acc[n][1]);
      *reinterpret_cast<__nv_bfloat162*>(Aw + ((lane >> 2) + 8) * lda + col) =
          __floats2bfloat162_rn(acc[n][2], acc[n][3]);
    }
    __syncwarp();
    const unsigned mine = row_index(r0);
#pragma unroll
    for (int i = lane; i < 16 * (DK / 8); i += 32) {
      const int r = i / (DK / 8), c = i % (DK / 8);
      const unsigned row = __shfl_sync(0xffffffffu, mine, r);
      if (r0 + r < R)
        *reinterpret_cast<uint4*>(out + (long long)row * DK + c * 8) =
            *reinterpret_cast<const uint4*>(Aw + r * lda + c * 8);
    }
    __syncwarp();
  }
}

template <int DK>
cudaError_t launch_fold_mma(const __nv_bfloat16* q, const __nv_bfloat16* W, __nv_bfloat16* out, long long T, int n_q,
                            int n_k, int d_q, cudaStream_t stream) {
  const int g = n_q / n_k;
  const size_t smem = ((size_t)d_q * (DK + 8) + 2 * (size_t)kMmaRows * (d_q + 8)) * sizeof(__nv_bfloat16);
  static std::atomic<int> configured{0};
  if (!configured.load(std::memory_order_acquire)) {
    const cudaError_t e = cudaFuncSetAttribute(fold_kup_mma_kernel<DK>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               210 * 1024);  // d_q 256, d_k 128 takes 205 KB
    if (e != cudaSuccess) return e;
    configured.store(1, std::memory_order_release);
  }
  const long long R = T * g, tiles = (R + kMmaRows - 1) / kMmaRows;
  // two blocks per SM and K head are enough to keep the loads in flight; each then amortises W over its tiles
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
    return cudaErrorUnknown;
  const long long per_head = std::max(1LL, (long long)(2 * sms + n_k - 1) / n_k);
  const dim3 grid((unsigned)std::min(tiles, per_head), (unsigned)n_k);
  fold_kup_mma_kernel<DK><<<grid, kMmaThreads, smem, stream>>>(q, W, out, R, n_q, g, d_q);
  count_launch();
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_fold_kup(const void* q, const void* W_kup, long long T, int n_q, int n_k, int d_q, int d_k,
                            void* q_out, cudaStream_t stream) {
  const auto aligned = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; };
  if (d_q % 16 == 0 && d_q <= 256 && d_k <= d_q && n_k <= 65535 && T * n_q <= 0x7fffffffLL && aligned(q) && aligned(W_kup) && aligned(q_out)) {
    const auto* qp = reinterpret_cast<const __nv_bfloat16*>(q);
    const auto* wp = reinterpret_cast<const __nv_bfloat16*>(W_kup);
    auto* op = reinterpret_cast<__nv_bfloat16*>(q_out);
    if (d_k == 32) return launch_fold_mma<32>(qp, wp, op, T, n_q, n_k, d_q, stream);
    if (d_k == 64) return launch_fold_mma<64>(qp, wp, op, T, n_q, n_k, d_q, stream);
    if (d_k == 128) return launch_fold_mma<128>(qp, wp, op, T, n_q, n_k, d_q, stream);
  }
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
