// Causal DiffQKV prefill attention on the sm_100a tensor cores (paper Section 2 formulation with the head map of
// Eq. (idx); appendix attention listing: cache update first, then the causal attention call).
//
// Step 1, cache_append_kernel: the new K and V rows go to positions past_b .. past_b + q_len - 1 of the pools.
// Step 2, prefill_attn_kernel: one block per (sequence, query head, 256 query rows), longest blocks first.
//   The 256 rows are two M-tiles of 128 that share every K/V tile the block stages (K head h*n_k/n_q, V head
//   h*n_v/n_q, read from the cache, so a cached prefix is attended as well); KV tiles hold 64 tokens.
//     warp 0      TMA producer: both Q tiles once, then K tiles and V tiles into 4-slot rings with their own barriers
//     warp 1      MMA issuer: S_t = Q_t K^T (tcgen05.mma 128x64x16, fp32 in TMEM), O_t += P_t V (128x128x16, V as an
//                 N-major operand straight from the token-major tile); scores are double-buffered per M-tile, so
//                 the next QK^T is issued before the softmax of the current tile ends, and the two M-tiles alternate
//     warps 2-5   softmax of M-tile 0, warps 6-9 of M-tile 1: one thread per query row (= TMEM lane) reads its 64
//                 scores with tcgen05.ld, masks the diagonal tiles, keeps a running reference maximum that is only
//                 raised when the row maximum exceeds it by 2^8 (then O is rescaled in TMEM), writes P as bf16 into
//                 shared memory in the swizzled K-major layout the second product reads, and sums the fp32 values
//   fp32 scores, softmax statistics and output accumulation; P is rounded to bf16 for the second product.
// Every wait is bounded; on expiry the block reports DIFFQKV_ERR_TIMEOUT, drains and frees its TMEM.
#include "common.cuh"
#include "ptx.cuh"
#include "tcgen05.cuh"
#include "tmap.cuh"

namespace diffqkv {
namespace {

constexpr int kQT = 128;  // query rows per M-tile
constexpr int kKT = 64;   // cached tokens per KV tile
constexpr int kD = 128;   // channels per head (Q/K and V)
constexpr int kKVStages = 4;
constexpr int kQBytes = kQT * kD * 2;   // 32 KB: [half][128 rows][128 B]
constexpr int kKBytes = kKT * kD * 2;   // 16 KB: [half][64 rows][128 B]
constexpr int kKVBytes = 2 * kKBytes;   // K tile then V tile
constexpr int kPBytes = kQT * kKT * 2;  // 16 KB: [128 rows][128 B]
constexpr int kPrefillThreads = 320;
constexpr int kTmemCols = 512;          // S[t][buf] at (2 t + buf) * 64 (0..255), O[t] at 256 + 128 t
constexpr int kPrefillSmem = 1024 + 2 * kQBytes + kKVStages * kKVBytes + 2 * kPBytes + 256;
constexpr float kRescaleThreshold = 8.f;  // log2 domain

struct PrefillParams {
  const int* seqlens;
  const int* page_table;
  int page_size, max_pages_per_seq, num_blocks, max_seqlen;
  int batch, q_len, n_q, n_k, n_v, n_qpairs;
  int box_tok;  // tokens per TMA box of the cache maps (64, or the page size when smaller)
  float scale_log2;
  void* out;
  int out_is_f32;
  float* lse;
  int* dev_status;
};

__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
// 2^x by the special-function unit alone (flushes denormal results to zero; -inf gives +0).
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

__device__ __forceinline__ bool wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  return __all_sync(0xffffffffu, ptx::mbar_wait(bar, parity, abort_flag));
}

__global__ void __launch_bounds__(kPrefillThreads, 1)
prefill_attn_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                    const __grid_constant__ CUtensorMap tmap_v, const PrefillParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* q_s = smem;                            // 2 M-tiles
  unsigned char* kv_s = q_s + 2 * kQBytes;              // ring of (K, V)
  unsigned char* p_s = kv_s + kKVStages * kKVBytes;     // 2 M-tiles
  uint64_t* bars = reinterpret_cast<uint64_t*>(p_s + 2 * kPBytes);
  // q_full, k_full[S], k_empty[S], v_full[S], v_empty[S], s_full[2 tiles][2 buffers], p_full[2], o_done[2], drain
  const uint32_t q_full = ptx::smem_u32(bars);
  const uint32_t k_full0 = q_full + 8, k_empty0 = k_full0 + 8 * kKVStages;
  const uint32_t v_full0 = k_empty0 + 8 * kKVStages, v_empty0 = v_full0 + 8 * kKVStages;
  const uint32_t s_full0 = v_empty0 + 8 * kKVStages, p_full0 = s_full0 + 32, o_done0 = p_full0 + 16;
  const uint32_t drain = o_done0 + 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 + 4 * kKVStages + 8);
  volatile int* abort_flag = reinterpret_cast<int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    *abort_flag = 0;
    ptx::mbar_init(q_full, 1);
    for (int s = 0; s < kKVStages; ++s) {
      ptx::mbar_init(k_full0 + 8 * s, 1);
      ptx::mbar_init(k_empty0 + 8 * s, 1);
      ptx::mbar_init(v_full0 + 8 * s, 1);
      ptx::mbar_init(v_empty0 + 8 * s, 1);
    }
    for (int t = 0; t < 2; ++t) {
      ptx::mbar_init(s_full0 + 16 * t, 1);
      ptx::mbar_init(s_full0 + 16 * t + 8, 1);
      ptx::mbar_init(p_full0 + 8 * t, 4);
      ptx::mbar_init(o_done0 + 8 * t, 1);
    }
    ptx::mbar_init(drain, 1);
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmap_q);
    ptx::prefetch_tmap(&tmap_k);
    ptx::prefetch_tmap(&tmap_v);
  }
  if (warp == 1) {
    tc::tmem_alloc(ptx::smem_u32(tmem_slot), kTmemCols);
    tc::tmem_relinquish();
  }
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  // ---- this block's work: sequence b, query head h, query rows [q0, q0 + 256)
  const int per = p.batch * p.n_q;
  const int qp = p.n_qpairs - 1 - (int)(blockIdx.x / per);  // longest first
  const int b = (int)(blockIdx.x % per) / p.n_q, h = (int)(blockIdx.x % per) % p.n_q;
  const int hk = (int)(((long long)h * p.n_k) / p.n_q);  // Eq. (idx)
  const int hv = (int)(((long long)h * p.n_v) / p.n_q);
  const int past = min(max(p.seqlens[b], 0), p.max_seqlen);
  const int kv_len = min(past + p.q_len, p.max_seqlen);
  const int q0 = qp * 2 * kQT;
  int nkv[2];
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    const int r0 = q0 + t * kQT;
    nkv[t] = r0 < p.q_len ? (min(kv_len, past + r0 + kQT) + kKT - 1) / kKT : 0;
  }
  const int nkv_max = max(nkv[0], nkv[1]);
  const uint32_t q_u32 = ptx::smem_u32(q_s), kv_u32 = ptx::smem_u32(kv_s), p_u32 = ptx::smem_u32(p_s);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      const int active = (nkv[0] > 0) + (nkv[1] > 0);
      ptx::mbar_arrive_expect_tx(q_full, (uint32_t)active * kQBytes);
#pragma unroll
      for (int t = 0; t < 2; ++t)
        if (nkv[t] > 0) ptx::tma_load_5d(q_u32 + t * kQBytes, &tmap_q, q_full, 0, q0 + t * kQT, 0, h, b);
    }
    // One box per (K or V, token part, channel half): lane x owns box x of every tile.  K and V tiles have their
    // own full/empty barriers: a K slot is free again as soon as its QK^T is done, two tiles before its V slot.
    const int parts = kKT / p.box_tok;
    const int boxes = 4 * parts;
    const int my_kv = lane / (2 * parts), my_part = (lane / 2) % parts, my_half = lane & 1;
    const uint32_t my_off = my_kv * kKBytes + my_half * (kKT * 128) + my_part * (p.box_tok * 128);
    int stage = 0, issued = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (int j = 0; j < nkv_max && ok; ++j) {
      const int tok0 = j * kKT;
      const int parts_valid = min(parts, (kv_len - tok0 + p.box_tok - 1) / p.box_tok);
      int blk = b, slot = tok0 + my_part * p.box_tok;
      const bool mine = lane < boxes && my_part < parts_valid;
      if (mine && p.page_table) {
        const int tok = slot;
        blk = p.page_table[(long long)b * p.max_pages_per_seq + tok / p.page_size];
        slot = tok % p.page_size;
        if (blk < 0 || blk >= p.num_blocks) {  // never read outside the pool: flag it, read block 0 instead
          report(p.dev_status, DIFFQKV_ERR_INDEX);
          blk = 0;
        }
      }
      const uint32_t dst = kv_u32 + stage * kKVBytes + my_off;
#pragma unroll
      for (int kv = 0; kv < 2; ++kv) {
        if (!wait_warp((kv ? v_empty0 : k_empty0) + 8 * stage, phase ^ 1, abort_flag)) { ok = false; break; }
        const uint32_t bar = (kv ? v_full0 : k_full0) + 8 * stage;
        if (lane == 0) ptx::mbar_arrive_expect_tx(bar, (uint32_t)parts_valid * p.box_tok * 128u * 2u);
        __syncwarp();
        if (mine && my_kv == kv) {
          if (kv == 0) ptx::tma_load_5d(dst, &tmap_k, bar, 0, slot, my_half, hk, blk);
          else ptx::tma_load_5d(dst, &tmap_v, bar, 0, slot, my_half, hv, blk);
        }
        if (kv) ++issued;
      }
      if (++stage == kKVStages) { stage = 0; phase ^= 1; }
    }
    if (!ok) {
      report(p.dev_status, DIFFQKV_ERR_TIMEOUT);
      // give copies in flight a bounded chance to land before the block's shared memory is released (a K copy
      // whose V twin was never issued is covered by the wait on the next use of its barrier timing out)
      ptx::mbar_wait(q_full, 0, nullptr);
      for (int s2 = 0; s2 < min(issued, kKVStages); ++s2) {
        const int uses = (issued - s2 + kKVStages - 1) / kKVStages;
        ptx::mbar_wait(k_full0 + 8 * s2, (uint32_t)(uses - 1) & 1u, nullptr);
        ptx::mbar_wait(v_full0 + 8 * s2, (uint32_t)(uses - 1) & 1u, nullptr);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // One thread runs the whole issue loop.  The products here are small (32 or 64 tensor-pipe cycles each), so the
    // loop is kept lean: descriptor halves are precomputed and only their address field is stepped.
    constexpr uint32_t idesc_s = tc::idesc_bf16_f32(kQT, kKT, 0, 0);
    constexpr uint32_t idesc_pv = tc::idesc_bf16_f32(kQT, kD, 0, 1);
    constexpr uint32_t hi_k = tc::smem_desc_hi_sw128(1024);  // K-major operands (Q, K, P) and the N-major V alike:
                                                             // 8-row groups are 1024 bytes apart
    bool ok = true;
    if (lane == 0) {
      const uint32_t q_lo = tc::smem_desc_lo(q_u32, 16), k_lo = tc::smem_desc_lo(kv_u32, 16);
      const uint32_t p_lo = tc::smem_desc_lo(p_u32, 16), v_lo = tc::smem_desc_lo(kv_u32 + kKBytes, kKT * 128);
      auto issue_s = [&](int t, int j) {  // S_t = Q_t . K_j^T
        const uint32_t qa = q_lo + t * (kQBytes >> 4), ka = k_lo + (j % kKVStages) * (kKVBytes >> 4);
        const uint32_t d = tmem_base + (2 * t + (j & 1)) * kKT;
        tc::mma_ss_halves<false>(d, qa, hi_k, ka, hi_k, idesc_s);
#pragma unroll
        for (int ks = 1; ks < kD / 16; ++ks)
          tc::mma_ss_halves<true>(d, qa + (((ks / 4) * (kQT * 128) + (ks % 4) * 32) >> 4), hi_k,
                                  ka + (((ks / 4) * (kKT * 128) + (ks % 4) * 32) >> 4), hi_k, idesc_s);
        tc::commit(s_full0 + 16 * t + 8 * (j & 1));
      };
      auto issue_pv = [&](int t, int j) {  // O_t += P_t . V_j
        const uint32_t pa = p_lo + t * (kPBytes >> 4), va = v_lo + (j % kKVStages) * (kKVBytes >> 4);
        const uint32_t d = tmem_base + 256 + t * kD;
        if (j == 0) tc::mma_ss_halves<false>(d, pa, hi_k, va, hi_k, idesc_pv);
        else tc::mma_ss_halves<true>(d, pa, hi_k, va, hi_k, idesc_pv);
#pragma unroll
        for (int k = 1; k < kKT / 16; ++k)
          tc::mma_ss_halves<true>(d, pa + ((k * 32) >> 4), hi_k, va + ((k * 16 * 128) >> 4), hi_k, idesc_pv);
        tc::commit(o_done0 + 8 * t);
      };
      // The scores of a tile have two buffers per M-tile: S(t, j + 2) is issued as soon as the softmax warps have
      // consumed S(t, j) (which p_full(t, j) implies), so S(t, j + 1) is ready long before they ask for it.
      ok = ptx::mbar_wait(q_full, 0, abort_flag);
      for (int j = 0; j < min(2, nkv_max) && ok; ++j) {
        ok = ptx::mbar_wait(k_full0 + 8 * j, 0, abort_flag);
        if (!ok) break;
        tc::fence_after_sync();
        if (j < nkv[0]) issue_s(0, j);
        if (j < nkv[1]) issue_s(1, j);
        tc::commit(k_empty0 + 8 * j);  // K tile j is free once these products are done
      }
      for (int j = 0; j < nkv_max && ok; ++j) {
        const int st = j % kKVStages, st2 = (j + 2) % kKVStages;
        const uint32_t ph = (j / kKVStages) & 1, ph2 = ((j + 2) / kKVStages) & 1;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          if (j < nkv[t]) {
            if (!ptx::mbar_wait(p_full0 + 8 * t, j & 1, abort_flag) || !ptx::mbar_wait(v_full0 + 8 * st, ph, abort_flag)) {
              ok = false;
              break;
            }
            tc::fence_after_sync();
            issue_pv(t, j);
          }
          if (t == 1) tc::commit(v_empty0 + 8 * st);  // every MMA that reads V tile j has been issued
          if (j + 2 < nkv[t]) {
            if (!ptx::mbar_wait(k_full0 + 8 * st2, ph2, abort_flag)) { ok = false; break; }
            tc::fence_after_sync();
            issue_s(t, j + 2);
          }
          if (t == 1 && j + 2 < nkv_max) tc::commit(k_empty0 + 8 * st2);  // ... and every MMA that reads K tile j + 2
        }
      }
      if (!ok) report(p.dev_status, DIFFQKV_ERR_TIMEOUT);
      tc::commit(drain);
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ softmax warps
    const int t = (warp - 2) >> 2;  // M-tile
    const int quarter = warp & 3;   // TMEM lanes this warp may touch
    const int r = quarter * 32 + lane;
    const int n = nkv[t];
    if (n > 0) {
      const int qrow = q0 + t * kQT + r;
      const int qpos = past + qrow;
      const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
      const uint32_t o_taddr = lane_base + 256 + t * kD;
      unsigned char* prow = p_s + t * kPBytes + r * 128;
      float m_ref = -INFINITY, l = 0.f;
      bool ok = true;
      for (int j = 0; j < n; ++j) {
        if (!wait_warp(s_full0 + 16 * t + 8 * (j & 1), (j >> 1) & 1, abort_flag)) { ok = false; break; }
        const uint32_t s_taddr = lane_base + (2 * t + (j & 1)) * kKT;
        tc::fence_after_sync();
        uint32_t s[64];
        tc::ld_32x32b_x32(s_taddr, *reinterpret_cast<uint32_t(*)[32]>(&s[0]));
        tc::ld_32x32b_x32(s_taddr + 32, *reinterpret_cast<uint32_t(*)[32]>(&s[32]));
        tc::wait_ld();
        const int k0 = j * kKT;
        const bool diag = k0 + kKT - 1 > past + q0 + t * kQT;  // block-uniform: the tile reaches past some row's position
        if (diag) {
#pragma unroll
          for (int c = 0; c < 64; ++c)
            if (k0 + c > qpos) s[c] = 0xff800000u;  // -inf: this token lies after the row's position
        }
        // row maximum of the raw scores (scale > 0 keeps the order), three inputs per instruction
        float mx_raw = __uint_as_float(s[0]);
#pragma unroll
        for (int c = 1; c < 63; c += 2) mx_raw = max3(mx_raw, __uint_as_float(s[c]), __uint_as_float(s[c + 1]));
        mx_raw = fmaxf(mx_raw, __uint_as_float(s[63]));
        const float mx = mx_raw * p.scale_log2;
        float alpha = 1.f;
        const bool bump = mx > m_ref + kRescaleThreshold;  // true on the first tile (m_ref = -inf)
        if (bump) {
          alpha = exp2f(m_ref - mx);
          m_ref = mx;
        }
        if (j > 0) {
          if (!wait_warp(o_done0 + 8 * t, (j - 1) & 1, abort_flag)) { ok = false; break; }
          tc::fence_after_sync();
          if (__any_sync(0xffffffffu, bump)) {  // rescale this warp's rows of O in tensor memory
#pragma unroll 1
            for (int c = 0; c < kD / 32; ++c) {
              uint32_t o[32];
              tc::ld_32x32b_x32(o_taddr + c * 32, o);
              tc::wait_ld();
#pragma unroll
              for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
              tc::st_32x32b_x32(o_taddr + c * 32, o);
            }
            tc::wait_st();
          }
        }
        l *= alpha;
        const float neg_m = -m_ref;
        // P = 2^(S - m_ref), rounded to bf16; row r of the tile, 16-byte chunks XORed with the row index
#pragma unroll
        for (int c8 = 0; c8 < 8; ++c8) {
          uint32_t w[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float p0 = ex2(fmaf(__uint_as_float(s[c8 * 8 + 2 * e]), p.scale_log2, neg_m));
            const float p1 = ex2(fmaf(__uint_as_float(s[c8 * 8 + 2 * e + 1]), p.scale_log2, neg_m));
            w[e] = pack2(p0, p1);
            l += p0 + p1;
          }
          *reinterpret_cast<uint4*>(prow + ((c8 ^ (r & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
        }
        if (j == nkv_max - 1 && (kv_len & (kKT - 1)) != 0) {
          // ragged last tile: V rows past the sequence end hold whatever followed in memory; zero them
          // (0 * NaN would poison the product).  Both M-tiles may do this; they write the same zeros.
          if (!wait_warp(v_full0 + 8 * (j % kKVStages), (j / kKVStages) & 1, abort_flag)) { ok = false; break; }
          const int row = r & 63, half = r >> 6;
          if (row >= kv_len - k0) {
            uint4* dst = reinterpret_cast<uint4*>(kv_s + (j % kKVStages) * kKVBytes + kKBytes + half * (kKT * 128) + row * 128);
#pragma unroll
            for (int e = 0; e < 8; ++e) dst[e] = make_uint4(0, 0, 0, 0);
          }
        }
        ptx::fence_proxy_async();
        tc::fence_before_sync();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(p_full0 + 8 * t);
      }
      if (ok && !wait_warp(o_done0 + 8 * t, (n - 1) & 1, abort_flag)) ok = false;
      if (ok) {
        tc::fence_after_sync();
        const float inv = 1.f / l;
        const bool store = qrow < p.q_len;
        const long long orow = (((long long)b * p.q_len + qrow) * p.n_q + h) * kD;
#pragma unroll 1
        for (int c = 0; c < kD / 32; ++c) {
          uint32_t o[32];
          tc::ld_32x32b_x32(o_taddr + c * 32, o);
          tc::wait_ld();
          if (store) {
            if (p.out_is_f32) {
              float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + orow + c * 32);
#pragma unroll
              for (int e = 0; e < 8; ++e)
                dst[e] = make_float4(__uint_as_float(o[4 * e]) * inv, __uint_as_float(o[4 * e + 1]) * inv,
                                     __uint_as_float(o[4 * e + 2]) * inv, __uint_as_float(o[4 * e + 3]) * inv);
            } else {
              uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.out) + orow + c * 32);
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                uint32_t w[4];
#pragma unroll
                for (int x = 0; x < 4; ++x)
                  w[x] = pack2(__uint_as_float(o[8 * e + 2 * x]) * inv, __uint_as_float(o[8 * e + 2 * x + 1]) * inv);
                dst[e] = make_uint4(w[0], w[1], w[2], w[3]);
              }
            }
          }
        }
        if (store && p.lse) p.lse[((long long)b * p.q_len + qrow) * p.n_q + h] = (m_ref + log2f(l)) * kLn2;
      } else {
        report(p.dev_status, DIFFQKV_ERR_TIMEOUT);
      }
    }
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

// The new rows of one pool: src [batch, q_len, heads, d] -> cache position past_b + i; 16-byte vectors.
struct AppendParams {
  const uint4* k_new;
  const uint4* v_new;
  uint4* k_cache;
  uint4* v_cache;
  long long k_sb, k_sh, k_st, v_sb, v_sh, v_st;  // in 16-byte vectors
  const int* seqlens;
  const int* page_table;
  int page_size, max_pages_per_seq, num_blocks, max_seqlen;
  int batch, q_len, n_k, n_v, vec_k, vec_v;  // vectors per head row
  int* dev_status;
};

__global__ void __launch_bounds__(256) cache_append_kernel(const AppendParams p) {
  const long long per_tok = (long long)p.n_k * p.vec_k + (long long)p.n_v * p.vec_v;
  const long long total = (long long)p.batch * p.q_len * per_tok;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const long long tokidx = idx / per_tok;
    int rem = (int)(idx % per_tok);
    const int b = (int)(tokidx / p.q_len), i = (int)(tokidx % p.q_len);
    const int tok = p.seqlens[b] + i;
    if (p.seqlens[b] < 0 || tok >= p.max_seqlen) {
      report(p.dev_status, DIFFQKV_ERR_INDEX);
      continue;
    }
    long long blk = b, slot = tok;
    if (p.page_table) {
      blk = p.page_table[(long long)b * p.max_pages_per_seq + tok / p.page_size];
      slot = tok % p.page_size;
      if (blk < 0 || blk >= p.num_blocks) {
        report(p.dev_status, DIFFQKV_ERR_INDEX);
        continue;
      }
    }
    const bool is_k = rem < p.n_k * p.vec_k;
    if (is_k) {
      const int head = rem / p.vec_k, c = rem % p.vec_k;
      p.k_cache[blk * p.k_sb + head * p.k_sh + slot * p.k_st + c] =
          p.k_new[(tokidx * p.n_k + head) * p.vec_k + c];
    } else {
      rem -= p.n_k * p.vec_k;
      const int head = rem / p.vec_v, c = rem % p.vec_v;
      p.v_cache[blk * p.v_sb + head * p.v_sh + slot * p.v_st + c] =
          p.v_new[(tokidx * p.n_v + head) * p.vec_v + c];
    }
  }
}

// Tensor map over one cache pool: dims (64 channels, token slot, channel half, head, block); a box brings
// box_tok tokens of one 64-channel half.
bool make_cache_map(CUtensorMap* map, const void* base, long long tok_extent, int heads, long long blocks,
                    long long st_tok, long long st_head, long long st_blk, int box_tok) {
  const cuuint64_t dims[5] = {64, (cuuint64_t)tok_extent, (cuuint64_t)(kD / 64), (cuuint64_t)heads, (cuuint64_t)blocks};
  const cuuint64_t strides[4] = {(cuuint64_t)st_tok * 2, 128, (cuuint64_t)st_head * 2, (cuuint64_t)st_blk * 2};
  const cuuint32_t box[5] = {64, (cuuint32_t)box_tok, 1, 1, 1};
  return make_tmap_bf16_sw128(map, base, 5, dims, strides, box);
}

}  // namespace

bool prefill_supported(const diffqkv_shape& s, const diffqkv_cache& c, int* box_tok) {
  if (s.dtype != DIFFQKV_BF16 || s.d_qk != kD || s.d_v != kD) return false;
  int bt = kKT;
  if (c.page_table) {
    if (c.page_size >= kKT) { if (c.page_size % kKT != 0) return false; }
    else { if (c.page_size < 8 || kKT % c.page_size != 0) return false; bt = c.page_size; }
  }
  *box_tok = bt;
  return true;
}

cudaError_t launch_prefill(const void* q, const void* k_new, const void* v_new, int q_len, const diffqkv_cache& c,
                           const diffqkv_shape& s, int box_tok, void* out, float* lse, int* dev_status,
                           cudaStream_t stream) {
  // ---- step 1: cache update
  AppendParams a;
  a.k_new = reinterpret_cast<const uint4*>(k_new);
  a.v_new = reinterpret_cast<const uint4*>(v_new);
  a.k_cache = reinterpret_cast<uint4*>(c.k_cache);
  a.v_cache = reinterpret_cast<uint4*>(c.v_cache);
  a.k_sb = c.k_stride_blk / 8; a.k_sh = c.k_stride_head / 8; a.k_st = c.k_stride_tok / 8;
  a.v_sb = c.v_stride_blk / 8; a.v_sh = c.v_stride_head / 8; a.v_st = c.v_stride_tok / 8;
  a.seqlens = c.seqlens; a.page_table = c.page_table;
  a.page_size = c.page_size; a.max_pages_per_seq = c.max_pages_per_seq;
  a.num_blocks = c.num_blocks; a.max_seqlen = c.max_seqlen;
  a.batch = s.batch; a.q_len = q_len; a.n_k = s.n_k; a.n_v = s.n_v;
  a.vec_k = s.d_qk / 8; a.vec_v = s.d_v / 8;
  a.dev_status = dev_status;
  const long long vecs = (long long)s.batch * q_len * ((long long)s.n_k * a.vec_k + (long long)s.n_v * a.vec_v);
  long long blocks = (vecs + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  cache_append_kernel<<<(unsigned)blocks, 256, 0, stream>>>(a);
  count_launch();
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;

  // ---- step 2: attention over the cache
  CUtensorMap mq, mk, mv;
  {
    const cuuint64_t dims[5] = {64, (cuuint64_t)q_len, (cuuint64_t)(kD / 64), (cuuint64_t)s.n_q, (cuuint64_t)s.batch};
    const cuuint64_t strides[4] = {(cuuint64_t)s.n_q * kD * 2, 128, (cuuint64_t)kD * 2,
                                   (cuuint64_t)q_len * s.n_q * kD * 2};
    const cuuint32_t box[5] = {64, kQT, kD / 64, 1, 1};
    if (!make_tmap_bf16_sw128(&mq, q, 5, dims, strides, box)) return cudaErrorNotSupported;
  }
  const long long tok_extent = c.page_table ? c.page_size : c.max_seqlen;
  if (!make_cache_map(&mk, c.k_cache, tok_extent, s.n_k, c.num_blocks, c.k_stride_tok, c.k_stride_head,
                      c.k_stride_blk, box_tok) ||
      !make_cache_map(&mv, c.v_cache, tok_extent, s.n_v, c.num_blocks, c.v_stride_tok, c.v_stride_head,
                      c.v_stride_blk, box_tok))
    return cudaErrorNotSupported;
  PrefillParams p;
  p.seqlens = c.seqlens; p.page_table = c.page_table;
  p.page_size = c.page_size; p.max_pages_per_seq = c.max_pages_per_seq;
  p.num_blocks = c.num_blocks; p.max_seqlen = c.max_seqlen;
  p.batch = s.batch; p.q_len = q_len; p.n_q = s.n_q; p.n_k = s.n_k; p.n_v = s.n_v;
  p.n_qpairs = (q_len + 2 * kQT - 1) / (2 * kQT);
  p.box_tok = box_tok;
  p.scale_log2 = s.scale * kLog2e;
  p.out = out; p.out_is_f32 = s.out_dtype == DIFFQKV_F32; p.lse = lse; p.dev_status = dev_status;
  const long long grid = (long long)p.n_qpairs * s.batch * s.n_q;
  if (grid > 0x7fffffffLL) return cudaErrorNotSupported;
  err = cudaFuncSetAttribute(prefill_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPrefillSmem);
  if (err != cudaSuccess) return err;
  prefill_attn_kernel<<<(unsigned)grid, kPrefillThreads, kPrefillSmem, stream>>>(mq, mk, mv, p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace diffqkv
