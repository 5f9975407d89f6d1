// Generic DiffQKV attention kernels: plain fp32 FMAs, any head counts, any strides, fp32 or bf16 storage.  They are
// the path for the fp32 mode and for shapes the TMA / tensor-core kernels do not take.  Decode: one block per (split,
// query head, sequence); causal prefill: one block per (query row, query head, sequence).  The head map is Eq. (idx)
// of the paper.
#include <atomic>

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


// ---------------------------------------------------------------------------------------------------------------
// Decode by units: one block per (split, unit, sequence), where a unit is the U = n_q / min(n_k, n_v) consecutive
// query heads that share their K heads (KPU of them) and V heads (VPU) among themselves only (Eq. (idx) makes the
// head maps contiguous blocks).  Every K and V row of the chunk is read from memory exactly once and serves all query
// heads of the unit: the decode design of the TMA kernel on plain loads and fp32 FMAs, for fp32 storage and for
// bf16 shapes no tensor map describes.  A warp takes every eighth token: its lanes split the row's channels
// (CQ = d_qk / 32 and CV = d_v / 32 consecutive channels per lane, one vector load each), the U partial inner products
// are summed across the lanes by shuffles, every lane keeps the running maxima and sums of all U heads and the
// un-normalised outputs of its own channels; the eight warps' states are merged through shared memory at the end.
constexpr int kUnitWarps = 8;
constexpr int kUnitThreads = kUnitWarps * 32;
constexpr int kUnitMaxHeads = 8;

template <typename T, int C>
__device__ __forceinline__ void load_slice(const T* p, float (&x)[C]);
template <>
__device__ __forceinline__ void load_slice<float, 2>(const float* p, float (&x)[2]) {
  const float2 v = *reinterpret_cast<const float2*>(p);
  x[0] = v.x; x[1] = v.y;
}
template <>
__device__ __forceinline__ void load_slice<float, 4>(const float* p, float (&x)[4]) {
  const float4 v = *reinterpret_cast<const float4*>(p);
  x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
}
template <>
__device__ __forceinline__ void load_slice<float, 8>(const float* p, float (&x)[8]) {
  const float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
  x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}
template <>
__device__ __forceinline__ void load_slice<__nv_bfloat16, 2>(const __nv_bfloat16* p, float (&x)[2]) {
  const uint32_t w = *reinterpret_cast<const uint32_t*>(p);
  x[0] = __uint_as_float(w << 16); x[1] = __uint_as_float(w & 0xffff0000u);
}
template <>
__device__ __forceinline__ void load_slice<__nv_bfloat16, 4>(const __nv_bfloat16* p, float (&x)[4]) {
  const uint2 v = *reinterpret_cast<const uint2*>(p);
  x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xffff0000u);
  x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xffff0000u);
}
template <>
__device__ __forceinline__ void load_slice<__nv_bfloat16, 8>(const __nv_bfloat16* p, float (&x)[8]) {
  Vec<__nv_bfloat16>::load(p, x);
}

// Sums each of eight per-lane values over the 32 lanes of a warp and leaves all eight sums in every lane, in 15
// shuffles instead of 40: three exchange steps in which a lane hands over the half of its values it will not sum
// (8 -> 4 -> 2 -> 1 values per lane), two plain steps, and a gather of the eight sums from the lanes that hold them.
__device__ __forceinline__ void warp_sum8(float (&v)[8], int lane) {
  const bool h16 = lane & 16, h8 = lane & 8, h4 = lane & 4;
  float a[4], b[2], c;
#pragma unroll
  for (int x = 0; x < 4; ++x) {
    const float send = h16 ? v[x] : v[x + 4], keep = h16 ? v[x + 4] : v[x];
    a[x] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
  }
#pragma unroll
  for (int x = 0; x < 2; ++x) {
    const float send = h8 ? a[x] : a[x + 2], keep = h8 ? a[x + 2] : a[x];
    b[x] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
  }
  {
    const float send = h4 ? b[0] : b[1], keep = h4 ? b[1] : b[0];
    c = keep + __shfl_xor_sync(0xffffffffu, send, 4);
  }
  c += __shfl_xor_sync(0xffffffffu, c, 2);
  c += __shfl_xor_sync(0xffffffffu, c, 1);
  // the lane with bits (16, 8, 4) = (x4, x2, x1) holds the sum of value x = 4 x4 + 2 x2 + x1
#pragma unroll
  for (int x = 0; x < 8; ++x) v[x] = __shfl_sync(0xffffffffu, c, ((x & 4) ? 16 : 0) + ((x & 2) ? 8 : 0) + ((x & 1) ? 4 : 0));
}

struct UnitParams {
  int U, kpu, vpu;  // query heads, K heads and V heads per unit
};

template <typename T, int CQ, int CV>
__global__ void __launch_bounds__(kUnitThreads) decode_unit_kernel(DecodeParams p, UnitParams up) {
  extern __shared__ float unit_smem[];  // [warps][U] maxima, [warps][U] sums, [warps][U][32 * CV] outputs
  constexpr int DV = 32 * CV;
  const int U = up.U;
  float* m_s = unit_smem;
  float* l_s = m_s + kUnitWarps * kUnitMaxHeads;
  float* o_s = l_s + kUnitWarps * kUnitMaxHeads;

  const int s = blockIdx.x, u = blockIdx.y, b = blockIdx.z;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const CacheView& c = p.cache;
  const int len = min(max(c.seqlens[b], 0), c.max_seqlen);
  const int t0 = s * p.chunk;
  const int t1 = min(len, t0 + p.chunk);
  const int h0 = u * U;  // first query head of the unit
  if (t0 >= t1) {       // empty split: the combine step skips -inf entries
    if (tid < U) p.lse_partial[((long long)b * p.n_q + h0 + tid) * p.splits + s] = -INFINITY;
    return;
  }
  const int heads_per_k = U / up.kpu, heads_per_v = U / up.vpu;
  const T* kbase = reinterpret_cast<const T*>(c.k);
  const T* vbase = reinterpret_cast<const T*>(c.v);

  // this lane's channels of every query of the unit, times scale * log2(e)
  float qr[kUnitMaxHeads][CQ];
#pragma unroll
  for (int i = 0; i < kUnitMaxHeads; ++i) {
    if (i < U) {
      load_slice<T, CQ>(reinterpret_cast<const T*>(p.q) + ((long long)b * p.n_q + h0 + i) * p.d_qk + lane * CQ, qr[i]);
#pragma unroll
      for (int e = 0; e < CQ; ++e) qr[i][e] *= p.scale_log2;
    } else {
#pragma unroll
      for (int e = 0; e < CQ; ++e) qr[i][e] = 0.f;
    }
  }
  float m_run[kUnitMaxHeads], l_run[kUnitMaxHeads], acc[kUnitMaxHeads][CV];
#pragma unroll
  for (int i = 0; i < kUnitMaxHeads; ++i) {
    m_run[i] = -INFINITY;
    l_run[i] = 0.f;
#pragma unroll
    for (int e = 0; e < CV; ++e) acc[i][e] = 0.f;
  }

  // kTok tokens per warp and pass (tokens j0 + i * kUnitWarps): their rows are requested together, so that a warp has
  // kTok times (KPU + VPU) rows in flight instead of one.
  constexpr int kTok = 4;
  for (int j0 = t0 + warp; j0 < t1; j0 += kUnitWarps * kTok) {
    long long koff[kTok], voff[kTok];  // element offsets of the token's head-0 rows; -1: not a token of this pass
#pragma unroll
    for (int i = 0; i < kTok; ++i) {
      const int j = j0 + i * kUnitWarps;
      koff[i] = voff[i] = -1;
      if (j < t1) {
        long long blk = b, slot = j;
        bool ok = true;
        if (c.page_table) {
          blk = c.page_table[(long long)b * c.max_pages_per_seq + j / c.page_size];
          slot = j % c.page_size;
          if (blk < 0 || blk >= c.num_blocks) {  // never read outside the pool: report it and leave the token out
            if (lane == 0) report(p.dev_status, DIFFQKV_ERR_INDEX);
            ok = false;
          }
        }
        if (ok) {
          koff[i] = blk * c.k_sb + (long long)(u * up.kpu) * c.k_sh + slot * c.k_st + lane * CQ;
          voff[i] = blk * c.v_sb + (long long)(u * up.vpu) * c.v_sh + slot * c.v_st + lane * CV;
        }
      }
    }
    // the first V head's rows are requested now, ahead of the scores they do not depend on
    float v0[kTok][CV];
#pragma unroll
    for (int i = 0; i < kTok; ++i) {
      if (voff[i] >= 0) {
        load_slice<T, CV>(vbase + voff[i], v0[i]);
      } else {
#pragma unroll
        for (int e = 0; e < CV; ++e) v0[i][e] = 0.f;
      }
    }
    // ---- scores of the U heads: each K head's row once, partial sums over this lane's channels, then over the lanes
    float sc[kTok][kUnitMaxHeads];
#pragma unroll
    for (int i = 0; i < kTok; ++i)
#pragma unroll
      for (int x = 0; x < kUnitMaxHeads; ++x) sc[i][x] = 0.f;
#pragma unroll
    for (int kh = 0; kh < kUnitMaxHeads; ++kh) {
      if (kh < up.kpu) {
        float kr[kTok][CQ];
#pragma unroll
        for (int i = 0; i < kTok; ++i) {
          if (koff[i] >= 0) {
            load_slice<T, CQ>(kbase + koff[i] + (long long)kh * c.k_sh, kr[i]);
          } else {
#pragma unroll
            for (int e = 0; e < CQ; ++e) kr[i][e] = 0.f;
          }
        }
#pragma unroll
        for (int x = 0; x < kUnitMaxHeads; ++x) {
          if (x < U && x / heads_per_k == kh) {
#pragma unroll
            for (int i = 0; i < kTok; ++i)
#pragma unroll
              for (int e = 0; e < CQ; ++e) sc[i][x] = fmaf(qr[x][e], kr[i][e], sc[i][x]);
          }
        }
      }
    }
    static_assert(kUnitMaxHeads == 8, "warp_sum8 sums eight values");
#pragma unroll
    for (int i = 0; i < kTok; ++i) warp_sum8(sc[i], lane);
    // ---- online softmax over the pass's tokens (every lane holds the same state, so the branches are uniform)
    float pw[kTok][kUnitMaxHeads];
#pragma unroll
    for (int x = 0; x < kUnitMaxHeads; ++x) {
#pragma unroll
      for (int i = 0; i < kTok; ++i) pw[i][x] = 0.f;
      if (x < U) {
        float mx = m_run[x];
#pragma unroll
        for (int i = 0; i < kTok; ++i)
          if (koff[i] >= 0) mx = fmaxf(mx, sc[i][x]);
        if (mx > m_run[x]) {
          const float alpha = exp2f(m_run[x] - mx);  // 0 on the first pass (m_run = -inf)
          l_run[x] *= alpha;
#pragma unroll
          for (int e = 0; e < CV; ++e) acc[x][e] *= alpha;
          m_run[x] = mx;
        }
#pragma unroll
        for (int i = 0; i < kTok; ++i) {
          if (koff[i] >= 0) {
            pw[i][x] = exp2f(sc[i][x] - mx);
            l_run[x] += pw[i][x];
          }
        }
      }
    }
    // ---- weighted V rows: each V head's row once, for the heads that read it
#pragma unroll
    for (int vh = 0; vh < kUnitMaxHeads; ++vh) {
      if (vh < up.vpu) {
        float vr[kTok][CV];
#pragma unroll
        for (int i = 0; i < kTok; ++i) {
          if (vh == 0) {
#pragma unroll
            for (int e = 0; e < CV; ++e) vr[i][e] = v0[i][e];
          } else if (voff[i] >= 0) {
            load_slice<T, CV>(vbase + voff[i] + (long long)vh * c.v_sh, vr[i]);
          } else {
#pragma unroll
            for (int e = 0; e < CV; ++e) vr[i][e] = 0.f;
          }
        }
#pragma unroll
        for (int x = 0; x < kUnitMaxHeads; ++x) {
          if (x < U && x / heads_per_v == vh) {
#pragma unroll
            for (int i = 0; i < kTok; ++i)
#pragma unroll
              for (int e = 0; e < CV; ++e) acc[x][e] = fmaf(pw[i][x], vr[i][e], acc[x][e]);
          }
        }
      }
    }
  }

  // ---- merge the warps' states and write the split's normalised result per head
#pragma unroll
  for (int i = 0; i < kUnitMaxHeads; ++i) {
    if (i < U) {
      if (lane == 0) {
        m_s[warp * kUnitMaxHeads + i] = m_run[i];
        l_s[warp * kUnitMaxHeads + i] = l_run[i];
      }
#pragma unroll
      for (int e = 0; e < CV; ++e) o_s[(warp * kUnitMaxHeads + i) * DV + lane * CV + e] = acc[i][e];
    }
  }
  __syncthreads();
  for (int x = tid; x < U * DV; x += kUnitThreads) {
    const int i = x / DV, ch = x % DV;
    float M = -INFINITY;
#pragma unroll
    for (int ww = 0; ww < kUnitWarps; ++ww) M = fmaxf(M, m_s[ww * kUnitMaxHeads + i]);
    float L = 0.f, o = 0.f;
#pragma unroll
    for (int ww = 0; ww < kUnitWarps; ++ww) {
      const float mw = m_s[ww * kUnitMaxHeads + i];
      if (mw == -INFINITY) continue;  // a warp without tokens
      const float wgt = exp2f(mw - M);
      L += wgt * l_s[ww * kUnitMaxHeads + i];
      o = fmaf(wgt, o_s[(ww * kUnitMaxHeads + i) * DV + ch], o);
    }
    const long long row_id = ((long long)b * p.n_q + h0 + i) * p.splits + s;
    p.o_partial[row_id * p.d_v + ch] = L > 0.f ? o / L : 0.f;
    if (ch == 0) p.lse_partial[row_id] = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
  }
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

// The unit kernel takes head counts whose groups nest (min(n_k, n_v) divides both), at most 8 query heads per unit
// and head dimensions of 64, 128 or 256 channels; everything else stays on the kernel with one block per query head.
std::atomic<int> g_per_head_only{0};  // test hook: 1 = never take the unit kernel

template <typename T>
static bool launch_unit(const DecodeParams& p, cudaStream_t stream, cudaError_t* err) {
  const int mn = p.n_k < p.n_v ? p.n_k : p.n_v;
  if (p.n_k % mn != 0 || p.n_v % mn != 0) return false;
  UnitParams up;
  up.U = p.n_q / mn; up.kpu = p.n_k / mn; up.vpu = p.n_v / mn;
  if (up.U > kUnitMaxHeads || up.U % up.kpu != 0 || up.U % up.vpu != 0) return false;
  if (p.batch > 65535 || p.n_q / up.U > 65535) return false;
  void (*fn)(DecodeParams, UnitParams) = nullptr;
#define DIFFQKV_UNIT_CASE(DQ, DV) \
  if (p.d_qk == DQ && p.d_v == DV) fn = decode_unit_kernel<T, DQ / 32, DV / 32>;
  DIFFQKV_UNIT_CASE(64, 64) DIFFQKV_UNIT_CASE(64, 128) DIFFQKV_UNIT_CASE(64, 256)
  DIFFQKV_UNIT_CASE(128, 64) DIFFQKV_UNIT_CASE(128, 128) DIFFQKV_UNIT_CASE(128, 256)
  DIFFQKV_UNIT_CASE(256, 64) DIFFQKV_UNIT_CASE(256, 128) DIFFQKV_UNIT_CASE(256, 256)
#undef DIFFQKV_UNIT_CASE
  if (!fn) return false;
  const size_t smem = sizeof(float) * kUnitWarps * kUnitMaxHeads * (2 + (size_t)p.d_v);
  *err = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (*err != cudaSuccess) return true;
  dim3 grid(p.splits, p.n_q / up.U, p.batch);
  fn<<<grid, kUnitThreads, smem, stream>>>(p, up);
  count_launch();
  *err = cudaGetLastError();
  return true;
}

void set_decode_per_head_only(int on) { g_per_head_only = on != 0; }

cudaError_t launch_decode_generic(const DecodeParams& p, diffqkv_dtype dtype, cudaStream_t stream) {
  if (!g_per_head_only.load()) {
    cudaError_t err = cudaSuccess;
    const bool taken = dtype == DIFFQKV_F32 ? launch_unit<float>(p, stream, &err)
                                            : launch_unit<__nv_bfloat16>(p, stream, &err);
    if (taken) return err;
  }
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
