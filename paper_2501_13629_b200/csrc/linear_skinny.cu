// Linear layers for a handful of rows (decode: one new token per sequence): y[M, N] = x[M, K] . W[N, K]^T with the
// epilogues of the projection chain (plain; silu(gate) * up over two weight matrices; rotate-half rotary embedding).
//
// With M <= 64 rows the tensor-core GEMM of augq.cu has 16 to 24 column tiles for 148 SMs and every tile streams its
// weight panel alone, so the step is bound by how few SMs pull on HBM (74 us for the aug-Q chain of config 4's widths
// where the weights, read once, take 14 us).  Here the weights are the streamed operand and the rows the stationary
// one, as in the decode kernels:
//   item       16 weight rows over the whole K: two groups of 8 rows that the epilogue needs side by side (plain: rows
//              16 i .. 16 i + 7 and 16 i + 8 .. 16 i + 15; gate/up: rows 8 i .. of W_gate and the same rows of W_up;
//              rotary: channels c .. c + 7 of a head and their partners c + d/2 ..), times a pass of 16 rows of x.
//              Items are dealt round-robin to one persistent block per SM, passes of an item back to back (the
//              second pass finds the weight rows in L2).
//   producer   one warp; a stage is 512 columns of K: two 8-row weight boxes (8 KB each) and a box of x (8 or 16 rows,
//              from L2), TMA with 128-byte swizzle into a ring of 4 or 3 stages, bounded waits.  The weights do not
//              depend on the grid before this one, so the first ring-full of weight boxes is requested before the
//              grid-dependency wait and only the x boxes after it.
//   consumers  8 warps; a stage has 32 steps of 16 columns, warp w takes steps w, w + 8, ...: ldmatrix of the weight
//              rows (A, 16 x 16) and of the x rows (B, 16 columns x 8 or 16 rows), mma.sync.m16n8k16 into fp32
//              accumulators; at the end of an item the eight partial sums go to shared memory
//   epilogue   one warp adds them and applies the epilogue (rows g and g + 8 of the accumulator tile, i.e. the two
//              groups, sit in the same thread) while the consumers are already in the next item.
// A block takes half an SM's shared memory: two blocks per SM stream side by side, and the blocks of the next grid in
// the stream (programmatic launch) move in and request their weights while this grid's last blocks finish.
// HBM-bound by design (2 flops per weight byte and row of x), hence mma.sync and not tcgen05.
#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"
#include "tmap.cuh"

namespace diffqkv {
namespace {

constexpr int kKC = 512;                  // columns of K per stage
constexpr int kChunks = kKC / 64;         // 64-column chunks (128 bytes) per stage
constexpr int kSkWarps = 8;               // consumer warps
constexpr int kSkThreads = (kSkWarps + 2) * 32;  // + producer warp + epilogue warp
constexpr int kWBox = kChunks * 8 * 128;  // one 8-row weight box
constexpr int kRingBytes = 96 * 1024;     // 4 stages with 8 rows of x, 3 with 16
constexpr int kRedBytes = kSkWarps * 32 * 8 * 4;
constexpr int kSkSmem = 1024 + kRingBytes + kRedBytes + 256;
constexpr int kBarThreads = (kSkWarps + 1) * 32;  // consumers + epilogue warp on the two named barriers

enum { kPlain = 0, kGateUp = 1, kRotary = 2 };

enum { kToMatrix = 0, kToKCache = 1, kToVCache = 2 };

// A launch covers up to three weight matrices that share x (and so K): a segment is a run of items on one of them.
struct Segment {
  int first_item, mode, head_dim;
  int map_a, map_b;  // which of the four weight maps the two 8-row boxes come from
  int dest;          // kToMatrix: row t of C; otherwise the cache row of sequence t at position seqlens[t]
  __nv_bfloat16* C;
  int ldc;
};

struct SkinnyParams {
  Segment seg[3];
  int n_seg;
  int M, K;
  int items, passes;  // items of 16 weight rows over all segments; passes of 8 or 16 rows of x
  const float* rope_cos;
  const float* rope_sin;
  CacheView cache;    // for the cache destinations
  int d_qk, d_v;
  int* dev_status;
};

// Segment of an item and the first weight rows of its two boxes.
__device__ __forceinline__ const Segment& item_rows(const SkinnyParams& p, int item, int& row_a, int& row_b) {
  int si = 0;
  if (p.n_seg > 1 && item >= p.seg[1].first_item) si = 1;
  if (p.n_seg > 2 && item >= p.seg[2].first_item) si = 2;
  const Segment& sg = p.seg[si];
  const int local = item - sg.first_item;
  if (sg.mode == kGateUp) {
    row_a = row_b = 8 * local;
  } else if (sg.mode == kRotary) {
    const int half = sg.head_dim >> 1, per_head = half >> 3;
    row_a = (local / per_head) * sg.head_dim + 8 * (local % per_head);
    row_b = row_a + half;
  } else {
    row_a = 16 * local;
    row_b = row_a + 8;
  }
  return sg;
}

// Where output channel `col` of row t goes: into C, or into the cache row of sequence t at position seqlens[t]
// (one new token per sequence; positions at or past max_seqlen and page ids outside the pool are reported and skipped).
__device__ __forceinline__ __nv_bfloat16* dest_of(const SkinnyParams& p, const Segment& sg, int t, int col) {
  if (sg.dest == kToMatrix) return sg.C + (long long)t * sg.ldc + col;
  const CacheView& c = p.cache;
  const int pos = c.seqlens[t];
  if (pos < 0 || pos >= c.max_seqlen) {
    report(p.dev_status, DIFFQKV_ERR_INDEX);
    return nullptr;
  }
  long long blk = t, slot = pos;
  if (c.page_table) {
    blk = c.page_table[(long long)t * c.max_pages_per_seq + pos / c.page_size];
    slot = pos % c.page_size;
    if (blk < 0 || blk >= c.num_blocks) {
      report(p.dev_status, DIFFQKV_ERR_INDEX);
      return nullptr;
    }
  }
  if (sg.dest == kToKCache)
    return reinterpret_cast<__nv_bfloat16*>(const_cast<void*>(c.k)) + blk * c.k_sb + (long long)(col / p.d_qk) * c.k_sh +
           slot * c.k_st + col % p.d_qk;
  return reinterpret_cast<__nv_bfloat16*>(const_cast<void*>(c.v)) + blk * c.v_sb + (long long)(col / p.d_v) * c.v_sh +
         slot * c.v_st + col % p.d_v;
}

template <int XROWS>  // rows of x per pass: 8 or 16
__global__ void __launch_bounds__(kSkThreads, 2)
linear_skinny_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w0,
                     const __grid_constant__ CUtensorMap tmap_w1, const __grid_constant__ CUtensorMap tmap_w2,
                     const __grid_constant__ CUtensorMap tmap_w3, const SkinnyParams p) {
  constexpr int kXBox = kChunks * XROWS * 128;
  constexpr int kStageBytes = 2 * kWBox + kXBox;
  constexpr int kStages = kRingBytes / kStageBytes;
  constexpr int NB = XROWS / 8;  // 8-row blocks of x = N blocks of the MMA
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  float* red = reinterpret_cast<float*>(smem + kRingBytes);  // [warp][lane][8]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kRingBytes + kRedBytes);  // full[s], empty[s]
  volatile int* abort_flag = reinterpret_cast<int*>(bars + 2 * kStages);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t full0 = ptx::smem_u32(bars), empty0 = ptx::smem_u32(bars + kStages);
  if (tid == 0) {
    *abort_flag = 0;
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(full0 + 8 * s, 1);
      ptx::mbar_init(empty0 + 8 * s, kSkWarps);
    }
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmap_x);
    ptx::prefetch_tmap(&tmap_w0);
    ptx::prefetch_tmap(&tmap_w1);
    ptx::prefetch_tmap(&tmap_w2);
    ptx::prefetch_tmap(&tmap_w3);
  }
  __syncthreads();
  ptx::grid_launch_dependents();

  const int total = p.items * p.passes;
  const int n_chunks = (p.K + kKC - 1) / kKC;  // stages per item (columns past K read as zero)
  const uint32_t smem_u32 = ptx::smem_u32(smem);

  if (warp == kSkWarps) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      int stage = 0, issued = 0;
      uint32_t phase = 0;
      bool ok = true;
      // the (item, chunk) sequence of this block, walked twice: `w` requests weight boxes, `x` the boxes of x
      struct Walk { int it, c; };
      Walk w = {(int)blockIdx.x, 0}, x = w;
      auto step = [&](Walk& k) { if (++k.c == n_chunks) { k.c = 0; k.it += gridDim.x; } };
      const CUtensorMap* wmaps[4] = {&tmap_w0, &tmap_w1, &tmap_w2, &tmap_w3};
      auto load_w = [&](const Walk& k, int st) {
        int row_a, row_b;
        const Segment& sg = item_rows(p, k.it / p.passes, row_a, row_b);
        const uint32_t bar = full0 + 8 * st, dst = smem_u32 + st * kStageBytes;
        ptx::mbar_arrive_expect_tx(bar, kStageBytes);
        ptx::tma_load_3d(dst, wmaps[sg.map_a], bar, 0, row_a, k.c * kChunks);
        ptx::tma_load_3d(dst + kWBox, wmaps[sg.map_b], bar, 0, row_b, k.c * kChunks);
      };
      auto load_x = [&](const Walk& k, int st) {
        ptx::tma_load_3d(smem_u32 + st * kStageBytes + 2 * kWBox, &tmap_x, full0 + 8 * st, 0, XROWS * (k.it % p.passes),
                         k.c * kChunks);
      };
      int ahead = 0;  // stages whose weights are requested but whose x is not
      for (; ahead < kStages && w.it < total; ++ahead, step(w)) load_w(w, ahead);
      ptx::grid_dependency_wait();  // x may be the output of the grid before this one
      for (int s = 0; s < ahead; ++s, step(x)) load_x(x, s);
      issued = ahead;
      stage = ahead % kStages;
      phase = ahead == kStages ? 1 : 0;
      for (; w.it < total; step(w), step(x)) {
        if (!ptx::mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag)) {
          report(p.dev_status, DIFFQKV_ERR_TIMEOUT);
          ok = false;
          break;
        }
        load_w(w, stage);
        load_x(x, stage);
        ++issued;
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
      if (!ok) {  // give copies in flight a bounded chance to land before the block's shared memory is released
        for (int s = 0; s < min(issued, kStages); ++s) {
          const int uses = (issued - s + kStages - 1) / kStages;
          ptx::mbar_wait(full0 + 8 * s, (uint32_t)(uses - 1) & 1u, nullptr);
        }
      }
    }
    return;
  }
  ptx::grid_dependency_wait();

  if (warp == kSkWarps + 1) {
    // ------------------------------------------------------------------ epilogue warp
    const int g8 = lane >> 2, t4 = lane & 3;
    for (int it = blockIdx.x; it < total; it += gridDim.x) {
      asm volatile("bar.sync 1, %0;" ::"n"(kBarThreads) : "memory");  // the item's partial sums are in place
      float v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = 0.f;
#pragma unroll
      for (int w = 0; w < kSkWarps; ++w) {
        const float4* src = reinterpret_cast<const float4*>(red + (w * 32 + lane) * 8);
        const float4 lo = src[0], hi = src[1];
        v[0] += lo.x; v[1] += lo.y; v[2] += lo.z; v[3] += lo.w;
        v[4] += hi.x; v[5] += hi.y; v[6] += hi.z; v[7] += hi.w;
      }
      asm volatile("bar.arrive 2, %0;" ::"n"(kBarThreads) : "memory");  // the buffer may be written again
      if (*abort_flag) continue;
      int row_a, row_b;
      const Segment& sg = item_rows(p, it / p.passes, row_a, row_b);
      // thread: weight rows g8 of either group, rows 2 t4 and 2 t4 + 1 of x in each 8-row block of the pass
#pragma unroll
      for (int nb = 0; nb < NB; ++nb)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const int t = XROWS * (it % p.passes) + 8 * nb + 2 * t4 + e;
          if (t >= p.M) continue;
          const float ca = v[4 * nb + e], cb = v[4 * nb + 2 + e];
          __nv_bfloat16* da = dest_of(p, sg, t, row_a + g8);
          if (!da) continue;
          if (sg.mode == kGateUp) {
            *da = __float2bfloat16_rn(ca / (1.f + __expf(-ca)) * cb);
            continue;
          }
          __nv_bfloat16* db = dest_of(p, sg, t, row_b + g8);
          if (sg.mode == kRotary) {
            const int half = sg.head_dim >> 1;
            const long long ti = (long long)t * half + (row_a % sg.head_dim) + g8;
            const float cs = p.rope_cos[ti], sn = p.rope_sin[ti];
            *da = __float2bfloat16_rn(ca * cs - cb * sn);
            *db = __float2bfloat16_rn(cb * cs + ca * sn);
          } else {
            *da = __float2bfloat16_rn(ca);
            *db = __float2bfloat16_rn(cb);
          }
        }
    }
    return;
  }

  // -------------------------------------------------------------------- consumers
  const int mi = lane >> 3, rr = lane & 7;
  // A (weights): matrices (rows 0-7, k 0-7), (rows 8-15, k 0-7), (rows 0-7, k 8-15), (rows 8-15, k 8-15); rows 8-15
  // are the second box.  B (x): matrices (rows 0-7, k 0-7), (rows 0-7, k 8-15), (rows 8-15, k 0-7), (rows 8-15, k 8-15);
  // with 8 rows of x the last two repeat the first two and are not used.
  const uint32_t a_base = (mi & 1) * kWBox + rr * 128, a_half = mi >> 1;
  const int xr = (NB == 2 ? (mi >> 1) * 8 : 0) + rr;
  const uint32_t b_base = 2 * kWBox + xr * 128, b_half = mi & 1;
  int stage = 0, n_item = 0;
  uint32_t phase = 0;
  bool dead = false;
  for (int it = blockIdx.x; it < total; it += gridDim.x, ++n_item) {
    float acc[2][4];
#pragma unroll
    for (int nb = 0; nb < 2; ++nb)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[nb][e] = 0.f;
    for (int c = 0; c < n_chunks; ++c) {
      if (!ptx::mbar_wait(full0 + 8 * stage, phase, abort_flag)) {
        if (!dead) report(p.dev_status, DIFFQKV_ERR_TIMEOUT);
        dead = true;  // keep walking the loops (no more waits succeed) so that the block's barriers still meet
      }
      if (!dead) {
        const uint32_t st = smem_u32 + stage * kStageBytes;
#pragma unroll
        for (int s4 = 0; s4 < 32 / kSkWarps; ++s4) {
          const int s = warp + s4 * kSkWarps;  // 16-column step of the stage
          const uint32_t chunk = s >> 2, unit = (s & 3) * 2;
          uint32_t a[4], b[4];
          ptx::ldmatrix_x4(st + a_base + chunk * 1024 + (((unit + a_half) ^ rr) << 4), a);
          ptx::ldmatrix_x4(st + b_base + chunk * (XROWS * 128) + (((unit + b_half) ^ rr) << 4), b);
          ptx::mma_bf16_16816(acc[0], a, b[0], b[1]);
          if (NB == 2) ptx::mma_bf16_16816(acc[1], a, b[2], b[3]);
        }
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(empty0 + 8 * stage);
      if (++stage == kStages) { stage = 0; phase ^= 1; }
    }
    // ---- the eight partial sums go to the epilogue warp
    if (n_item > 0) asm volatile("bar.sync 2, %0;" ::"n"(kBarThreads) : "memory");  // it has read the previous ones
    float4* mine = reinterpret_cast<float4*>(red + (warp * 32 + lane) * 8);
    mine[0] = make_float4(acc[0][0], acc[0][1], acc[0][2], acc[0][3]);
    mine[1] = make_float4(acc[1][0], acc[1][1], acc[1][2], acc[1][3]);
    asm volatile("bar.arrive 1, %0;" ::"n"(kBarThreads) : "memory");
  }
  if (n_item > 0) asm volatile("bar.sync 2, %0;" ::"n"(kBarThreads) : "memory");  // pairs with the last arrival
}

// dims (64 columns, rows, K / 64 chunks); a box is 64 columns x box_rows rows x kChunks chunks.
bool make_rows_map(CUtensorMap* map, const void* base, long long rows, int K, int box_rows) {
  const cuuint64_t dims[3] = {64, (cuuint64_t)rows, (cuuint64_t)(K / 64)};
  const cuuint64_t strides[2] = {(cuuint64_t)K * 2, 128};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, (cuuint32_t)kChunks};
  return make_tmap_bf16_sw128(map, base, 3, dims, strides, box);
}

}  // namespace

bool linear_skinny_supported(long long M, int N, int K, bool dual, int head_dim, bool rotary) {
  if (M < 1 || M > kSkinnyMaxRows || K % 64 != 0 || K < 64) return false;
  if (rotary) return !dual && head_dim % 16 == 0 && head_dim >= 16 && N % head_dim == 0;
  return dual ? N % 8 == 0 : N % 16 == 0;
}

namespace {

cudaError_t launch_segments(const CUtensorMap& mx, const CUtensorMap (&mw)[4], SkinnyParams& p, int xrows,
                            cudaStream_t stream) {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
    return cudaErrorUnknown;
  p.passes = (p.M + xrows - 1) / xrows;
  const long long total = (long long)p.items * p.passes;
  auto kernel = xrows == 8 ? linear_skinny_kernel<8> : linear_skinny_kernel<16>;
  cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSkSmem);
  if (err != cudaSuccess) return err;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cfg.gridDim = dim3((unsigned)(total < 2 * sms ? total : 2 * sms));  // two blocks per SM
  cfg.blockDim = dim3(kSkThreads);
  cfg.dynamicSmemBytes = kSkSmem;
  err = cudaLaunchKernelEx(&cfg, kernel, mx, mw[0], mw[1], mw[2], mw[3], p);
  if (err != cudaSuccess) return err;
  count_launch();
  return cudaGetLastError();
}

Segment make_segment(int first_item, int mode, int head_dim, int map_a, int map_b, int dest, void* C, int ldc) {
  Segment sg;
  sg.first_item = first_item; sg.mode = mode; sg.head_dim = head_dim;
  sg.map_a = map_a; sg.map_b = map_b; sg.dest = dest;
  sg.C = reinterpret_cast<__nv_bfloat16*>(C); sg.ldc = ldc;
  return sg;
}

}  // namespace

cudaError_t launch_linear_skinny(const void* A, const void* B0, const void* B1, void* C, long long M, int N, int K,
                                 int* dev_status, cudaStream_t stream, const float* rope_cos, const float* rope_sin,
                                 int head_dim) {
  const int xrows = M <= 8 ? 8 : 16;
  CUtensorMap mx, mw[4];
  if (!make_rows_map(&mx, A, M, K, xrows) || !make_rows_map(&mw[0], B0, N, K, 8) ||
      !make_rows_map(&mw[1], B1 ? B1 : B0, N, K, 8))
    return cudaErrorNotSupported;
  mw[2] = mw[0];
  mw[3] = mw[0];
  SkinnyParams p = {};
  const int mode = B1 ? kGateUp : (rope_cos ? kRotary : kPlain);
  p.seg[0] = make_segment(0, mode, head_dim, 0, B1 ? 1 : 0, kToMatrix, C, N);
  p.n_seg = 1;
  p.M = (int)M; p.K = K;
  p.items = mode == kGateUp ? N / 8 : N / 16;
  p.rope_cos = rope_cos; p.rope_sin = rope_sin;
  p.dev_status = dev_status;
  return launch_segments(mx, mw, p, xrows, stream);
}

// One launch for everything a decode step computes from the hidden state h [M, K]: x = h W_Q^T into C (the first
// product of the aug-Q chain), k = rope(h W_K^T) and v = h W_V^T straight into the cache rows of the new tokens.
cudaError_t launch_qkv_skinny(const void* h, const void* W_Q, void* x, int d_q0, const void* W_K, const void* W_V,
                              long long M, int K, const float* rope_cos, const float* rope_sin, const CacheView& cache,
                              int n_k, int n_v, int d_qk, int d_v, int* dev_status, cudaStream_t stream) {
  const int xrows = M <= 8 ? 8 : 16;
  CUtensorMap mx, mw[4];
  if (!make_rows_map(&mx, h, M, K, xrows) || !make_rows_map(&mw[0], W_Q, d_q0, K, 8) ||
      !make_rows_map(&mw[1], W_K, (long long)n_k * d_qk, K, 8) || !make_rows_map(&mw[2], W_V, (long long)n_v * d_v, K, 8))
    return cudaErrorNotSupported;
  mw[3] = mw[0];
  SkinnyParams p = {};
  const int items_q = d_q0 / 16, items_k = n_k * d_qk / 16, items_v = n_v * d_v / 16;
  p.seg[0] = make_segment(0, kPlain, 0, 0, 0, kToMatrix, x, d_q0);
  p.seg[1] = make_segment(items_q, rope_cos ? kRotary : kPlain, d_qk, 1, 1, kToKCache, nullptr, 0);
  p.seg[2] = make_segment(items_q + items_k, kPlain, 0, 2, 2, kToVCache, nullptr, 0);
  p.n_seg = 3;
  p.M = (int)M; p.K = K;
  p.items = items_q + items_k + items_v;
  p.rope_cos = rope_cos; p.rope_sin = rope_sin;
  p.cache = cache;
  p.d_qk = d_qk; p.d_v = d_v;
  p.dev_status = dev_status;
  return launch_segments(mx, mw, p, xrows, stream);
}

}  // namespace diffqkv
