// Augmented-Q projection (paper Section 2, Observation 3; appendix attention listing):
//     x = h W_Q^T,   a = silu(x W_gate^T) * (x W_up^T),   q = a W_down^T
// as three bf16 GEMMs C[M,N] = A[M,K] . B[N,K]^T on the sm_100a tensor cores (tcgen05.mma, fp32 accumulators in
// tensor memory), the gate and up products fused into one kernel whose epilogue applies silu(g) * u.
//
// One persistent block per SM walks output tiles of 128 rows x 256 accumulator columns:
//   warp 0      TMA producer: A tile (128 x 64) and B tile (256 x 64; in the fused kernel 128 gate rows followed by
//               128 up rows) per K block into a 4-stage ring, 128-byte swizzle, one mbarrier per stage
//   warp 1      MMA issuer: four 128x256x16 tcgen05.mma per K block, tcgen05.commit frees the stage; the two
//               256-column accumulators in TMEM alternate so the epilogue of a tile overlaps the next main loop
//   warps 2-5   epilogue: tcgen05.ld of the warp's 32 TMEM lanes (= 32 output rows), silu-gate when fused,
//               bf16 conversion, 16-byte global stores
// Every wait is bounded; on expiry the block reports DIFFQKV_ERR_TIMEOUT, drains and frees its TMEM.
#include <atomic>

#include "common.cuh"
#include "ptx.cuh"
#include "tcgen05.cuh"
#include "tmap.cuh"

namespace diffqkv {
namespace {

constexpr int kBM = 128, kBN = 256, kBK = 64;
constexpr int kStages = 4;
constexpr int kABytes = kBM * kBK * 2;  // 16 KB
constexpr int kBBytes = kBN * kBK * 2;  // 32 KB
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kGemmThreads = 192;
constexpr int kTmemCols = 512;
constexpr int kGemmSmem = 1024 + kStages * kStageBytes + 256;

struct GemmParams {
  __nv_bfloat16* C;
  long long ldc;
  int M, N;
  int m_tiles, n_tiles, k_blocks;
  int dual;  // 0: C tile 128x256 = A.B0^T;  1: C tile 128x128 = silu(A.B0^T) * (A.B1^T)
  // rotary embedding applied to the fp32 result before it is rounded (plain mode only): tables [M, head_dim / 2],
  // channel i < head_dim / 2 of a head pairs with channel i + head_dim / 2; NULL = none
  const float* rope_cos;
  const float* rope_sin;
  int head_dim;
  int* dev_status;
};

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_nt_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b0,
               const __grid_constant__ CUtensorMap tmap_b1, const GemmParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
  // full[kStages], empty[kStages], tfull[2], tempty[2], drain
  const uint32_t full0 = ptx::smem_u32(bars), empty0 = full0 + 8 * kStages;
  const uint32_t tfull0 = empty0 + 8 * kStages, tempty0 = tfull0 + 16, drain = tempty0 + 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kStages + 5);
  volatile int* abort_flag = reinterpret_cast<int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    *abort_flag = 0;
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(full0 + 8 * s, 1);
      ptx::mbar_init(empty0 + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(tfull0 + 8 * a, 1);
      ptx::mbar_init(tempty0 + 8 * a, 4);
    }
    ptx::mbar_init(drain, 1);
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmap_a);
    ptx::prefetch_tmap(&tmap_b0);
    if (p.dual) ptx::prefetch_tmap(&tmap_b1);
  }
  if (warp == 1) {
    tc::tmem_alloc(ptx::smem_u32(tmem_slot), kTmemCols);
    tc::tmem_relinquish();
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  const int num_tiles = p.m_tiles * p.n_tiles;
  const uint32_t smem0 = ptx::smem_u32(smem);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    int stage = 0, issued = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x) {
      const int m0 = (t / p.n_tiles) * kBM;
      const int nt = t % p.n_tiles;
      for (int kb = 0; kb < p.k_blocks; ++kb) {
        if (!ptx::mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag)) { ok = false; break; }
        if (lane == 0) {
          const uint32_t bar = full0 + 8 * stage;
          const uint32_t dst = smem0 + stage * kStageBytes;
          ptx::mbar_arrive_expect_tx(bar, kStageBytes);
          ptx::tma_load_2d(dst, &tmap_a, bar, kb * kBK, m0);
          if (p.dual) {
            ptx::tma_load_2d(dst + kABytes, &tmap_b0, bar, kb * kBK, nt * 128);
            ptx::tma_load_2d(dst + kABytes + kBBytes / 2, &tmap_b1, bar, kb * kBK, nt * 128);
          } else {
            ptx::tma_load_2d(dst + kABytes, &tmap_b0, bar, kb * kBK, nt * kBN);
            ptx::tma_load_2d(dst + kABytes + kBBytes / 2, &tmap_b0, bar, kb * kBK, nt * kBN + 128);
          }
        }
        __syncwarp();
        ++issued;
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
    }
    if (!ok) {
      report(p.dev_status, DIFFQKV_ERR_TIMEOUT);
      // give copies in flight a bounded chance to land before the block's shared memory is released
      for (int s = 0; s < min(issued, kStages); ++s) {
        const int uses = (issued - s + kStages - 1) / kStages;
        ptx::mbar_wait(full0 + 8 * s, (uint32_t)(uses - 1) & 1u, nullptr);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    constexpr uint32_t idesc = tc::idesc_bf16_f32(kBM, kBN, 0, 0);
    int stage = 0, local = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++local) {
      const int acc = local & 1;
      const uint32_t acc_phase = (local >> 1) & 1;
      if (!ptx::mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1, abort_flag)) { ok = false; break; }
      tc::fence_after_sync();
      const uint32_t d_tmem = tmem_base + acc * kBN;
      for (int kb = 0; kb < p.k_blocks; ++kb) {
        if (!ptx::mbar_wait(full0 + 8 * stage, phase, abort_flag)) { ok = false; break; }
        tc::fence_after_sync();
        if (lane == 0) {
          const uint32_t a_addr = smem0 + stage * kStageBytes, b_addr = a_addr + kABytes;
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) {
            const uint64_t da = tc::smem_desc_sw128(a_addr + k * 32, 16, 1024);
            const uint64_t db = tc::smem_desc_sw128(b_addr + k * 32, 16, 1024);
            tc::mma_ss(d_tmem, da, db, idesc, (kb > 0 || k > 0) ? 1u : 0u);
          }
          tc::commit(empty0 + 8 * stage);
        }
        __syncwarp();
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
      if (ok && lane == 0) tc::commit(tfull0 + 8 * acc);
      __syncwarp();
    }
    if (!ok) report(p.dev_status, DIFFQKV_ERR_TIMEOUT);
    if (lane == 0) tc::commit(drain);
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int quarter = warp & 3;  // TMEM lanes this warp may touch
    int local = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < num_tiles && ok; t += gridDim.x, ++local) {
      const int acc = local & 1;
      const uint32_t acc_phase = (local >> 1) & 1;
      if (!ptx::mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag)) { ok = false; break; }
      tc::fence_after_sync();
      const int row = (t / p.n_tiles) * kBM + quarter * 32 + lane;
      const int nt = t % p.n_tiles;
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + acc * kBN;
      if (p.dual) {
        __nv_bfloat16* crow = p.C + (long long)row * p.ldc + (long long)nt * 128;
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          if (nt * 128 + c * 32 >= p.N) break;  // warp-uniform: partial last column tile
          uint32_t g[32], u[32];
          tc::ld_32x32b_x32(taddr + c * 32, g);
          tc::ld_32x32b_x32(taddr + 128 + c * 32, u);
          tc::wait_ld();
          if (row < p.M) {
            uint32_t o[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              const float g0 = __uint_as_float(g[2 * e]), g1 = __uint_as_float(g[2 * e + 1]);
              const float a0 = g0 / (1.f + __expf(-g0)) * __uint_as_float(u[2 * e]);
              const float a1 = g1 / (1.f + __expf(-g1)) * __uint_as_float(u[2 * e + 1]);
              o[e] = pack2(a0, a1);
            }
#pragma unroll
            for (int v = 0; v < 4; ++v)
              *reinterpret_cast<uint4*>(crow + c * 32 + v * 8) = make_uint4(o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3]);
          }
        }
      } else if (p.rope_cos) {
        __nv_bfloat16* crow = p.C + (long long)row * p.ldc + (long long)nt * kBN;
        const int half = p.head_dim >> 1;
        const long long trow = (long long)(row < p.M ? row : 0) * half;
#pragma unroll 1
        for (int hd = 0; hd < kBN; hd += p.head_dim) {  // heads of this column tile
          if (nt * kBN + hd >= p.N) break;              // warp-uniform: partial last column tile
#pragma unroll 1
          for (int c = 0; c < half; c += 32) {
            uint32_t x1[32], x2[32];
            tc::ld_32x32b_x32(taddr + hd + c, x1);
            tc::ld_32x32b_x32(taddr + hd + half + c, x2);
            tc::wait_ld();
            if (row < p.M) {
              uint32_t o1[16], o2[16];
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const float4 cs = *reinterpret_cast<const float4*>(p.rope_cos + trow + c + 4 * e);
                const float4 sn = *reinterpret_cast<const float4*>(p.rope_sin + trow + c + 4 * e);
                const float cv[4] = {cs.x, cs.y, cs.z, cs.w}, sv[4] = {sn.x, sn.y, sn.z, sn.w};
                float y1[4], y2[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  const float a = __uint_as_float(x1[4 * e + i]), b = __uint_as_float(x2[4 * e + i]);
                  y1[i] = a * cv[i] - b * sv[i];
                  y2[i] = b * cv[i] + a * sv[i];
                }
                o1[2 * e] = pack2(y1[0], y1[1]); o1[2 * e + 1] = pack2(y1[2], y1[3]);
                o2[2 * e] = pack2(y2[0], y2[1]); o2[2 * e + 1] = pack2(y2[2], y2[3]);
              }
#pragma unroll
              for (int v = 0; v < 4; ++v) {
                *reinterpret_cast<uint4*>(crow + hd + c + v * 8) = make_uint4(o1[4 * v], o1[4 * v + 1], o1[4 * v + 2], o1[4 * v + 3]);
                *reinterpret_cast<uint4*>(crow + hd + half + c + v * 8) = make_uint4(o2[4 * v], o2[4 * v + 1], o2[4 * v + 2], o2[4 * v + 3]);
              }
            }
          }
        }
      } else {
        __nv_bfloat16* crow = p.C + (long long)row * p.ldc + (long long)nt * kBN;
#pragma unroll 1
        for (int c = 0; c < kBN / 32; ++c) {
          if (nt * kBN + c * 32 >= p.N) break;  // warp-uniform: partial last column tile
          uint32_t r[32];
          tc::ld_32x32b_x32(taddr + c * 32, r);
          tc::wait_ld();
          if (row < p.M) {
            uint32_t o[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) o[e] = pack2(__uint_as_float(r[2 * e]), __uint_as_float(r[2 * e + 1]));
#pragma unroll
            for (int v = 0; v < 4; ++v)
              *reinterpret_cast<uint4*>(crow + c * 32 + v * 8) = make_uint4(o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3]);
          }
        }
      }
      tc::fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(tempty0 + 8 * acc);
    }
    if (!ok) report(p.dev_status, DIFFQKV_ERR_TIMEOUT);
  }

  // ---- teardown: all MMAs this block issued must be done before its tensor memory is released
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::mbar_wait(drain, 0, nullptr);
    tc::fence_after_sync();
    tc::tmem_dealloc(tmem_base, kTmemCols);
  }
}

bool make_operand_map(CUtensorMap* map, const void* base, long long rows, long long cols) {
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  const cuuint32_t box[2] = {kBK, 128};
  return make_tmap_bf16_sw128(map, base, 2, dims, strides, box);
}

int sm_count() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  return sms;
}

std::atomic<int> g_force_tensor_gemm{0};  // test hook: 1 = never take the weight-streaming kernel for few rows

// C[M, N] = A[M, K] . B0[N, K]^T, or with B1: C[M, N] = silu(A.B0^T) * (A.B1^T).
cudaError_t launch_gemm(const void* A, const void* B0, const void* B1, void* C, long long M, int N, int K,
                        int* dev_status, cudaStream_t stream, const float* rope_cos = nullptr,
                        const float* rope_sin = nullptr, int head_dim = 0) {
  // a handful of rows (decode): the weight-streaming kernel; its tiles would leave most SMs of this one idle
  if (!g_force_tensor_gemm && linear_skinny_supported(M, N, K, B1 != nullptr, head_dim, rope_cos != nullptr))
    return launch_linear_skinny(A, B0, B1, C, M, N, K, dev_status, stream, rope_cos, rope_sin, head_dim);
  CUtensorMap ma, mb0, mb1;
  if (!make_operand_map(&ma, A, M, K) || !make_operand_map(&mb0, B0, N, K) ||
      !make_operand_map(&mb1, B1 ? B1 : B0, N, K))
    return cudaErrorNotSupported;
  GemmParams p;
  p.C = reinterpret_cast<__nv_bfloat16*>(C);
  p.ldc = N;
  p.M = (int)M;
  p.N = N;
  p.m_tiles = (int)((M + kBM - 1) / kBM);
  p.dual = B1 ? 1 : 0;
  p.n_tiles = p.dual ? N / 128 : (N + kBN - 1) / kBN;
  p.k_blocks = K / kBK;
  p.dev_status = dev_status;
  p.rope_cos = p.dual ? nullptr : rope_cos;
  p.rope_sin = rope_sin;
  p.head_dim = head_dim;
  const int sms = sm_count();
  if (sms <= 0) return cudaErrorUnknown;
  const long long tiles = (long long)p.m_tiles * p.n_tiles;
  const int grid = (int)(tiles < sms ? tiles : sms);
  cudaError_t err = cudaFuncSetAttribute(gemm_nt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmem);
  if (err != cudaSuccess) return err;
  gemm_nt_kernel<<<grid, kGemmThreads, kGemmSmem, stream>>>(ma, mb0, mb1, p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace

void set_force_tensor_gemm(int on) { g_force_tensor_gemm = on != 0; }

size_t augq_workspace_bytes(long long T, int d_q0, int d_aug) {
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  return up((size_t)T * d_q0 * 2) + up((size_t)T * d_aug * 2);
}

cudaError_t launch_augq(const void* h, const void* W_Q, const void* W_gate, const void* W_up, const void* W_down,
                        long long T, int d_model, int d_q0, int d_aug, int d_out, void* workspace, void* q_out,
                        int* dev_status, cudaStream_t stream, const float* rope_cos, const float* rope_sin,
                        int head_dim) {
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  char* ws = reinterpret_cast<char*>(workspace);
  void* x = ws;
  void* a = ws + up((size_t)T * d_q0 * 2);
  cudaError_t err = launch_gemm(h, W_Q, nullptr, x, T, d_q0, d_model, dev_status, stream);
  if (err != cudaSuccess) return err;
  err = launch_gemm(x, W_gate, W_up, a, T, d_aug, d_q0, dev_status, stream);
  if (err != cudaSuccess) return err;
  return launch_gemm(a, W_down, nullptr, q_out, T, d_out, d_aug, dev_status, stream, rope_cos, rope_sin, head_dim);
}

size_t decode_frontend_workspace_bytes(const diffqkv_shape& s, int d_aug) {
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  return augq_workspace_bytes(s.batch, s.n_q * s.d_qk, d_aug) + up((size_t)s.batch * s.n_k * s.d_qk * 2) +
         up((size_t)s.batch * s.n_v * s.d_v * 2);
}

cudaError_t launch_decode_frontend(const void* h, const void* W_Q, const void* W_gate, const void* W_up,
                                   const void* W_down, const void* W_K, const void* W_V, int d_model, int d_aug,
                                   const float* rope_cos, const float* rope_sin, const diffqkv_cache& c,
                                   const CacheView& view, const diffqkv_shape& s, void* workspace, void* q_out,
                                   int* dev_status, cudaStream_t stream) {
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  const long long T = s.batch;
  const int d_q0 = s.n_q * s.d_qk, kw = s.n_k * s.d_qk, vw = s.n_v * s.d_v;
  char* ws = reinterpret_cast<char*>(workspace);
  void* x = ws;
  void* a = ws + up((size_t)T * d_q0 * 2);
  if (!g_force_tensor_gemm && T <= kSkinnyMaxRows) {
    // three launches: {x = h W_Q^T, k and v into the cache}, a = silu(x W_gate^T) * (x W_up^T), q = rope(a W_down^T)
    cudaError_t err = launch_qkv_skinny(h, W_Q, x, d_q0, W_K, W_V, T, d_model, rope_cos, rope_sin, view, s.n_k, s.n_v,
                                        s.d_qk, s.d_v, dev_status, stream);
    if (err != cudaSuccess) return err;
    err = launch_gemm(x, W_gate, W_up, a, T, d_aug, d_q0, dev_status, stream);
    if (err != cudaSuccess) return err;
    return launch_gemm(a, W_down, nullptr, q_out, T, d_q0, d_aug, dev_status, stream, rope_cos, rope_sin, s.d_qk);
  }
  // many rows: the separate steps (tensor-core products, then the cache update)
  if (kw % 128 != 0 || vw % 128 != 0) return cudaErrorNotSupported;
  char* k_new = ws + augq_workspace_bytes(T, d_q0, d_aug);
  char* v_new = k_new + up((size_t)T * kw * 2);
  cudaError_t err = launch_augq(h, W_Q, W_gate, W_up, W_down, T, d_model, d_q0, d_aug, d_q0, workspace, q_out,
                                dev_status, stream, rope_cos, rope_sin, s.d_qk);
  if (err != cudaSuccess) return err;
  err = launch_gemm(h, W_K, nullptr, k_new, T, kw, d_model, dev_status, stream, rope_cos, rope_sin, s.d_qk);
  if (err != cudaSuccess) return err;
  err = launch_gemm(h, W_V, nullptr, v_new, T, vw, d_model, dev_status, stream);
  if (err != cudaSuccess) return err;
  return launch_cache_append(k_new, v_new, 1, c, s, dev_status, stream);
}

// y[T, d_out] = x[T, d_in] . W[d_out, d_in]^T, optionally rotated per head (the K and V projections).
cudaError_t launch_project(const void* x, const void* W, long long T, int d_in, int d_out, void* y, int* dev_status,
                           cudaStream_t stream, const float* rope_cos, const float* rope_sin, int head_dim) {
  return launch_gemm(x, W, nullptr, y, T, d_out, d_in, dev_status, stream, rope_cos, rope_sin, head_dim);
}

}  // namespace diffqkv
