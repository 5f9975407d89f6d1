// Causal DiffQKV prefill attention on the sm_100a tensor cores (paper Section 2 formulation with the head map of
// Eq. (idx); appendix attention listing: cache update first, then the causal attention call).
//
// Step 1, cache_append_kernel: the new K and V rows go to positions past_b .. past_b + q_len - 1 of the pools.
// Step 2, prefill_attn_kernel: one block per (sequence, query head, 256 query rows), longest blocks first.
//   The 256 rows are two M-tiles of 128 that share every K/V tile the block stages (K head h*n_k/n_q, V head
//   h*n_v/n_q, read from the cache, so a cached prefix is attended as well); KV tiles hold 128 tokens.
//     warp 0      TMA producer: both Q tiles once, then K tiles (ring of 3) and V tiles (ring of 2), 128-byte swizzle,
//                 each ring with its own barriers: a K slot is free as soon as its QK^T is done
//     warp 1      one thread issues the MMAs: S_t = Q_t K^T (tcgen05.mma 128x128x16 from shared memory, fp32 in
//                 TMEM) and O_t += P_t V (128x128x16, P read from TMEM, V as an N-major operand straight from its
//                 token-major tile); the two M-tiles alternate, so the tensor core works on one while the softmax
//                 warps work on the other.  Operands are what bounds these products (about 100 bytes per cycle
//                 reach the tensor core from shared memory), hence 128-wide tiles and P kept out of shared memory.
//     warps 2-3   idle: they complete the first group of four warps, which hands most of its registers to the
//                 softmax warps (setmaxnreg works on aligned groups of four warps)
//     warps 4-7   softmax of M-tile 0, warps 8-11 of M-tile 1: one thread per query row (= TMEM lane).  The thread
//                 reads its 128 scores into registers (tcgen05.ld), takes the row maximum (a running reference
//                 maximum is only raised when exceeded by 2^8; then O is rescaled in TMEM), computes
//                 P = 2^(S scale - m) (scale-and-shift and row sum as packed fp32 pairs, to leave the issue slots
//                 to the exponentials), sums it in fp32 and writes it as packed bf16 over the first 64 score columns
//                 (tcgen05.st), where the second product reads it; the first 64 tokens of P are announced on a
//                 barrier of their own, so that half of the second product runs under the rest of the exponentials.
//   fp32 scores, softmax statistics and output accumulation; P is rounded to bf16 for the second product.
//   The kernel is a template on the head dimensions (channels of Q/K and of V): (128, 128), (64, 64) with half-width
//   tiles, four K steps in the first product and 64 TMEM columns of O per M-tile, and (64, 128) for keys cached at half
//   the value width.  With 64-channel values P has tensor-memory columns of its own, and the next tile's scores are
//   issued as soon as the softmax warps hold the current ones (see kSepP).
// Every wait is bounded; on expiry the block reports DIFFQKV_ERR_TIMEOUT, drains and frees its TMEM.
#include "common.cuh"
#include "ptx.cuh"
#include "tcgen05.cuh"
#include "tmap.cuh"

namespace diffqkv {
namespace {

constexpr int kQT = 128;  // query rows per M-tile
constexpr int kKT = 128;  // cached tokens per KV tile
constexpr int kDMax = 128;  // channels per head (Q/K and V): the kernel is built for 128 and for 64
constexpr int kKSlots = 3, kVSlots = 2;
// Three groups of four warps: {TMA producer, MMA issuer, two idle warps}, the softmax warps of M-tile 0 and those of
// M-tile 1.  The first group hands most of its registers to the other two (setmaxnreg works on aligned groups of four
// warps): 12 x 168 = 4 x 56 + 8 x 224.
constexpr int kPrefillThreads = 384;
constexpr int kSoftmaxWarp0 = 4;
constexpr int kTmemCols = 512;         // S[t] (and P[t] over its first 64 columns) at 128 t, O[t] at 256 + D t
// Shared memory is sized for D = 128 whatever D is: one block per SM, since a block takes all of the tensor memory.
constexpr int kPrefillSmem = 1024 + 2 * (kQT * kDMax * 2) + (kKSlots + kVSlots) * (kKT * kDMax * 2) + 256;
constexpr float kRescaleThreshold = 8.f;  // log2 domain

struct PrefillParams {
  const int* seqlens;
  const int* page_table;
  int page_size, max_pages_per_seq, num_blocks, max_seqlen;
  int batch, q_len, n_q, n_k, n_v, n_qpairs;
  int box_tok;  // tokens per TMA box of the cache maps (128, or the page size when smaller)
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

// Packed fp32 pairs (one instruction, two lanes of the FMA pipe over two cycles: half the issue slots of the scalar
// forms, which is what the softmax warps are short of next to their special-function instructions).
__device__ __forceinline__ uint64_t pair(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ uint64_t pair(uint32_t lo, uint32_t hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
  return r;
}
__device__ __forceinline__ void unpair(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ bool wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  return __all_sync(0xffffffffu, ptx::mbar_wait(bar, parity, abort_flag));
}

template <int kDQK, int kD>  // channels per head of Q/K and of V: (128, 128), (64, 64) or (64, 128)
__global__ void __launch_bounds__(kPrefillThreads, 1)
prefill_attn_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                    const __grid_constant__ CUtensorMap tmap_v, const PrefillParams p) {
  constexpr int kHalvesK = kDQK / 64, kHalves = kD / 64;  // 64-channel halves of a Q/K row and of a V row
  constexpr int kHalvesMax = kHalvesK > kHalves ? kHalvesK : kHalves;
  constexpr int kQBytes = kQT * kDQK * 2;   // a Q tile: [half][128 rows][128 B]
  constexpr int kKBytes = kKT * kDQK * 2;   // a K tile: [half][128 rows][128 B]
  constexpr int kTBytes = kKT * kD * 2;     // a V tile: [half][128 rows][128 B]
  // With 64-channel values the two output accumulators take 128 of the 512 tensor-memory columns instead of 256, which
  // leaves room for P outside the score columns: [S0 128][S1 128][O0 64][O1 64][P0 64][P1 64].  The next tile's
  // scores can then be issued as soon as the softmax warps have taken the current ones into registers, instead of
  // after the product that reads P, and the softmax warps find them ready when they come back.
  constexpr bool kSepP = kD == 64;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* q_s = smem;                      // 2 M-tiles
  unsigned char* k_s = q_s + 2 * kQBytes;         // ring of K tiles
  unsigned char* v_s = k_s + kKSlots * kKBytes;   // ring of V tiles
  uint64_t* bars = reinterpret_cast<uint64_t*>(v_s + kVSlots * kTBytes);
  // q_full, k_full[3], k_empty[3], v_full[2], v_empty[2], s_full[2], p_full[2], o_done[2], drain, p_half[2]
  const uint32_t q_full = ptx::smem_u32(bars);
  const uint32_t k_full0 = q_full + 8, k_empty0 = k_full0 + 8 * kKSlots;
  const uint32_t v_full0 = k_empty0 + 8 * kKSlots, v_empty0 = v_full0 + 8 * kVSlots;
  const uint32_t s_full0 = v_empty0 + 8 * kVSlots, p_full0 = s_full0 + 16, o_done0 = p_full0 + 16;
  const uint32_t drain = o_done0 + 16;
  const uint32_t p_half0 = drain + 8;  // the first 64 tokens of P_t are in place
  const uint32_t s_free0 = p_half0 + 16;  // (kSepP) the scores of M-tile t have been read out of tensor memory
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 + 2 * kKSlots + 2 * kVSlots + 6 + 2 + 2);
  volatile int* abort_flag = reinterpret_cast<int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    *abort_flag = 0;
    ptx::mbar_init(q_full, 1);
    for (int s = 0; s < kKSlots; ++s) {
      ptx::mbar_init(k_full0 + 8 * s, 1);
      ptx::mbar_init(k_empty0 + 8 * s, 1);
    }
    for (int s = 0; s < kVSlots; ++s) {
      ptx::mbar_init(v_full0 + 8 * s, 1);
      ptx::mbar_init(v_empty0 + 8 * s, 1);
    }
    for (int t = 0; t < 2; ++t) {
      ptx::mbar_init(s_full0 + 8 * t, 1);
      ptx::mbar_init(p_full0 + 8 * t, 4);
      ptx::mbar_init(p_half0 + 8 * t, 4);
      ptx::mbar_init(s_free0 + 8 * t, 4);
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
  const uint32_t q_u32 = ptx::smem_u32(q_s), k_u32 = ptx::smem_u32(k_s), v_u32 = ptx::smem_u32(v_s);

  if (warp < kSoftmaxWarp0) {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      const int active = (nkv[0] > 0) + (nkv[1] > 0);
      ptx::mbar_arrive_expect_tx(q_full, (uint32_t)active * kQBytes);
#pragma unroll
      for (int t = 0; t < 2; ++t)
        if (nkv[t] > 0) ptx::tma_load_5d(q_u32 + t * kQBytes, &tmap_q, q_full, 0, q0 + t * kQT, 0, h, b);
    }
    // One box per (token part, channel half) of a tile: lane x owns box x of every K tile and of every V tile.
    const int parts = kKT / p.box_tok;
    const int boxes = kHalvesMax * parts;
    const int my_part = lane / kHalvesMax, my_half = lane % kHalvesMax;
    const uint32_t my_off = my_half * (kKT * 128) + my_part * (p.box_tok * 128);
    int ks = 0, vs = 0, issued_k = 0, issued_v = 0;
    uint32_t kph = 0, vph = 0;
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
      const uint32_t tx = (uint32_t)parts_valid * p.box_tok * 128u * kHalves;
      const uint32_t tx_k = (uint32_t)parts_valid * p.box_tok * 128u * kHalvesK;
      if (!wait_warp(k_empty0 + 8 * ks, kph ^ 1, abort_flag)) { ok = false; break; }
      if (lane == 0) ptx::mbar_arrive_expect_tx(k_full0 + 8 * ks, tx_k);
      __syncwarp();
      if (mine && my_half < kHalvesK)
        ptx::tma_load_5d(k_u32 + ks * kKBytes + my_off, &tmap_k, k_full0 + 8 * ks, 0, slot, my_half, hk, blk);
      ++issued_k;
      if (++ks == kKSlots) { ks = 0; kph ^= 1; }
      if (!wait_warp(v_empty0 + 8 * vs, vph ^ 1, abort_flag)) { ok = false; break; }
      if (lane == 0) ptx::mbar_arrive_expect_tx(v_full0 + 8 * vs, tx);
      __syncwarp();
      if (mine && my_half < kHalves)
        ptx::tma_load_5d(v_u32 + vs * kTBytes + my_off, &tmap_v, v_full0 + 8 * vs, 0, slot, my_half, hv, blk);
      ++issued_v;
      if (++vs == kVSlots) { vs = 0; vph ^= 1; }
    }
    if (!ok) {
      report(p.dev_status, DIFFQKV_ERR_TIMEOUT);
      // give copies in flight a bounded chance to land before the block's shared memory is released
      ptx::mbar_wait(q_full, 0, nullptr);
      for (int s2 = 0; s2 < min(issued_k, kKSlots); ++s2)
        ptx::mbar_wait(k_full0 + 8 * s2, (uint32_t)((issued_k - s2 + kKSlots - 1) / kKSlots - 1) & 1u, nullptr);
      for (int s2 = 0; s2 < min(issued_v, kVSlots); ++s2)
        ptx::mbar_wait(v_full0 + 8 * s2, (uint32_t)((issued_v - s2 + kVSlots - 1) / kVSlots - 1) & 1u, nullptr);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (one thread)
    constexpr uint32_t idesc = tc::idesc_bf16_f32(kQT, 128, 0, 0);     // S: Q and K both K-major, N = 128 tokens
    constexpr uint32_t idesc_pv = tc::idesc_bf16_f32(kQT, kD, 0, 1);   // O: V is N-major, N = kD channels
    constexpr uint32_t hi = tc::smem_desc_hi_sw128(1024);              // 8-row groups are 1024 bytes apart everywhere
    bool ok = true;
    if (lane == 0) {
      const uint32_t q_lo = tc::smem_desc_lo(q_u32, 16), k_lo = tc::smem_desc_lo(k_u32, 16);
      const uint32_t v_lo = tc::smem_desc_lo(v_u32, kKT * 128);  // 64-channel chunks of V are one half tile apart
      auto issue_s = [&](int t, int slot) {  // S_t = Q_t . K^T
        const uint32_t qa = q_lo + t * (kQBytes >> 4), ka = k_lo + slot * (kKBytes >> 4);
        const uint32_t d = tmem_base + t * 128;
        tc::mma_ss_halves<false>(d, qa, hi, ka, hi, idesc);
#pragma unroll
        for (int ks = 1; ks < kDQK / 16; ++ks) {
          const uint32_t step = ((ks / 4) * (128 * 128) + (ks % 4) * 32) >> 4;
          tc::mma_ss_halves<true>(d, qa + step, hi, ka + step, hi, idesc);
        }
        tc::commit(s_full0 + 8 * t);
      };
      // O_t += P_t . V in two halves of 64 tokens: the first is issued while the softmax warps still work on the
      // second half of P_t
      auto issue_pv = [&](int t, int slot, bool first, int half) {
        const uint32_t va = v_lo + slot * (kTBytes >> 4);
        const uint32_t d = tmem_base + 256 + t * kD, pa = kSepP ? tmem_base + 384 + t * 64 : tmem_base + t * 128;
        constexpr int kSteps = kKT / 32;  // K steps of 16 tokens per half
        if (half == 0) {
          if (first) tc::mma_ts_halves<false>(d, pa, va, hi, idesc_pv);
          else tc::mma_ts_halves<true>(d, pa, va, hi, idesc_pv);
#pragma unroll
          for (int k = 1; k < kSteps; ++k) tc::mma_ts_halves<true>(d, pa + k * 8, va + ((k * 16 * 128) >> 4), hi, idesc_pv);
        } else {
#pragma unroll
          for (int k = kSteps; k < 2 * kSteps; ++k)
            tc::mma_ts_halves<true>(d, pa + k * 8, va + ((k * 16 * 128) >> 4), hi, idesc_pv);
          tc::commit(o_done0 + 8 * t);
        }
      };
      ok = ptx::mbar_wait(q_full, 0, abort_flag);
      if (ok && nkv_max > 0) ok = ptx::mbar_wait(k_full0, 0, abort_flag);
      if (ok && nkv_max > 0) {
        tc::fence_after_sync();
        if (nkv[0] > 0) issue_s(0, 0);
        if (nkv[1] > 0) issue_s(1, 0);
        tc::commit(k_empty0);  // K tile 0 is free once these products are done
      }
      int ks = 1 % kKSlots, vs = 0;  // slot of K tile j + 1, slot of V tile j
      uint32_t kph = 0, vph = 0;
      if (kSepP) {
        for (int j = 0; j < nkv_max && ok; ++j) {
          // the next tile's scores first: their columns are free once the softmax warps hold the current ones
          if (j + 1 < nkv_max) {
            if (!ptx::mbar_wait(k_full0 + 8 * ks, kph, abort_flag)) { ok = false; break; }
#pragma unroll
            for (int t = 0; t < 2; ++t) {
              if (j + 1 < nkv[t]) {
                if (!ptx::mbar_wait(s_free0 + 8 * t, j & 1, abort_flag)) { ok = false; break; }
                tc::fence_after_sync();
                issue_s(t, ks);
              }
            }
            if (!ok) break;
            tc::commit(k_empty0 + 8 * ks);
          }
#pragma unroll
          for (int t = 0; t < 2; ++t) {
            if (j < nkv[t]) {
              if (!ptx::mbar_wait(p_half0 + 8 * t, j & 1, abort_flag) || !ptx::mbar_wait(v_full0 + 8 * vs, vph, abort_flag)) {
                ok = false;
                break;
              }
              tc::fence_after_sync();
              issue_pv(t, vs, j == 0, 0);
              if (!ptx::mbar_wait(p_full0 + 8 * t, j & 1, abort_flag)) { ok = false; break; }
              tc::fence_after_sync();
              issue_pv(t, vs, j == 0, 1);
            }
          }
          if (!ok) break;
          tc::commit(v_empty0 + 8 * vs);  // every MMA that reads V tile j has been issued
          if (++ks == kKSlots) { ks = 0; kph ^= 1; }
          if (++vs == kVSlots) { vs = 0; vph ^= 1; }
        }
      } else {
      for (int j = 0; j < nkv_max && ok; ++j) {
#pragma unroll
        for (int t = 0; t < 2; ++t) {
          if (j < nkv[t]) {
            if (!ptx::mbar_wait(p_half0 + 8 * t, j & 1, abort_flag) || !ptx::mbar_wait(v_full0 + 8 * vs, vph, abort_flag)) {
              ok = false;
              break;
            }
            tc::fence_after_sync();
            issue_pv(t, vs, j == 0, 0);
            if (!ptx::mbar_wait(p_full0 + 8 * t, j & 1, abort_flag)) { ok = false; break; }
            tc::fence_after_sync();
            issue_pv(t, vs, j == 0, 1);
          }
          if (t == 1) tc::commit(v_empty0 + 8 * vs);  // every MMA that reads V tile j has been issued
          if (j + 1 < nkv[t]) {  // P_t of tile j has been consumed by then (same pipe, in order): S_t may be overwritten
            if (!ptx::mbar_wait(k_full0 + 8 * ks, kph, abort_flag)) { ok = false; break; }
            tc::fence_after_sync();
            issue_s(t, ks);
          }
          if (t == 1 && j + 1 < nkv_max) tc::commit(k_empty0 + 8 * ks);  // ... and every MMA that reads K tile j + 1
        }
        if (++ks == kKSlots) { ks = 0; kph ^= 1; }
        if (++vs == kVSlots) { vs = 0; vph ^= 1; }
      }
      }
      if (!ok) report(p.dev_status, DIFFQKV_ERR_TIMEOUT);
      tc::commit(drain);
    }
    __syncwarp();
  }
  } else {
    // ------------------------------------------------------------------ softmax warps
    asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
    const int t = (warp - kSoftmaxWarp0) >> 2;  // M-tile
    const int quarter = warp & 3;   // TMEM lanes this warp may touch
    const int r = quarter * 32 + lane;
    const int n = nkv[t];
    if (n > 0) {
      const int qrow = q0 + t * kQT + r;
      const int qpos = past + qrow;
      const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
      const uint32_t s_taddr = lane_base + t * 128;  // scores, and (unless P has columns of its own) P over their first 64
      const uint32_t p_taddr = kSepP ? lane_base + 384 + t * 64 : s_taddr;
      const uint32_t o_taddr = lane_base + 256 + t * kD;
      float m_ref = -INFINITY, l = 0.f;
      bool ok = true;
      for (int j = 0; j < n; ++j) {
        if (!wait_warp(s_full0 + 8 * t, j & 1, abort_flag)) { ok = false; break; }
        tc::fence_after_sync();
        const int k0 = j * kKT;
        const bool diag = k0 + kKT - 1 > past + q0 + t * kQT;  // block-uniform: the tile reaches past some row's position
        // ---- all 128 scores of the row into registers; row maximum of the raw scores (scale > 0 keeps the order)
        uint32_t s[128];
#pragma unroll
        for (int c = 0; c < 4; ++c) tc::ld_32x32b_x32(s_taddr + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
        tc::wait_ld();
        if (kSepP) {  // the score columns may take the next tile's scores from here on
          tc::fence_before_sync();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(s_free0 + 8 * t);
        }
        if (diag) {
#pragma unroll
          for (int e = 0; e < 128; ++e)
            if (k0 + e > qpos) s[e] = 0xff800000u;  // -inf: this token lies after the row's position
        }
        float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
        for (int e = 0; e < 128; e += 8) {  // four independent chains, three inputs per instruction
          mx0 = max3(mx0, __uint_as_float(s[e]), __uint_as_float(s[e + 1]));
          mx1 = max3(mx1, __uint_as_float(s[e + 2]), __uint_as_float(s[e + 3]));
          mx2 = max3(mx2, __uint_as_float(s[e + 4]), __uint_as_float(s[e + 5]));
          mx3 = max3(mx3, __uint_as_float(s[e + 6]), __uint_as_float(s[e + 7]));
        }
        const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * p.scale_log2;
        float alpha = 1.f;
        const bool bump = mx > m_ref + kRescaleThreshold;  // true on the first tile (m_ref = -inf)
        if (bump) {
          alpha = exp2f(m_ref - mx);
          m_ref = mx;
        }
        if (j > 0 && __any_sync(0xffffffffu, bump)) {  // rescale this warp's rows of O in tensor memory
          if (!wait_warp(o_done0 + 8 * t, (j - 1) & 1, abort_flag)) { ok = false; break; }
          tc::fence_after_sync();
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
        l *= alpha;
        const float neg_m = -m_ref;
        if (j == nkv_max - 1 && (kv_len & (kKT - 1)) != 0) {
          // ragged last tile: V rows past the sequence end hold whatever followed in memory; zero them before any
          // product reads the tile (0 * NaN would poison it).  Both M-tiles may do this; they write the same zeros.
          const int vslot = j % kVSlots;
          if (!wait_warp(v_full0 + 8 * vslot, (j / kVSlots) & 1, abort_flag)) { ok = false; break; }
          if (r >= kv_len - k0) {
#pragma unroll
            for (int half = 0; half < kHalves; ++half) {
              uint4* dst = reinterpret_cast<uint4*>(v_s + vslot * kTBytes + half * (kKT * 128) + r * 128);
#pragma unroll
              for (int e = 0; e < 8; ++e) dst[e] = make_uint4(0, 0, 0, 0);
            }
          }
          ptx::fence_proxy_async();
        }
        // ---- P = 2^(S scale - m_ref) as packed bf16 over the first 64 score columns; fp32 row sum.  The first 64
        // tokens are announced on their own, so that their half of the product runs during the second half's work.
        if (kSepP && j > 0) {  // P's own columns still hold the previous tile's P until its product is done
          if (!wait_warp(o_done0 + 8 * t, (j - 1) & 1, abort_flag)) { ok = false; break; }
          tc::fence_after_sync();
        }
        // Scale-and-shift and the row sum are packed: with a special-function instruction taking most of the issue
        // slots of its eight cycles, the other instructions of the loop are what the exponentials wait for.
        uint64_t l2 = 0;  // two partial row sums
        const uint64_t scale2 = pair(p.scale_log2, p.scale_log2), negm2 = pair(neg_m, neg_m);
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          uint32_t w[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            float x0, x1;
            unpair(fma2(pair(s[c * 64 + 2 * e], s[c * 64 + 2 * e + 1]), scale2, negm2), x0, x1);
            const float p0 = ex2(x0), p1 = ex2(x1);
            w[e] = pack2(p0, p1);
            l2 = add2(l2, pair(p0, p1));
          }
          tc::st_32x32b_x32(p_taddr + c * 32, w);
          if (c == 0) {
            tc::wait_st();
            tc::fence_before_sync();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(p_half0 + 8 * t);
          }
        }
        float l0, l1;
        unpair(l2, l0, l1);
        l += l0 + l1;
        tc::wait_st();
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
bool make_cache_map(CUtensorMap* map, const void* base, int d, long long tok_extent, int heads, long long blocks,
                    long long st_tok, long long st_head, long long st_blk, int box_tok) {
  const cuuint64_t dims[5] = {64, (cuuint64_t)tok_extent, (cuuint64_t)(d / 64), (cuuint64_t)heads, (cuuint64_t)blocks};
  const cuuint64_t strides[4] = {(cuuint64_t)st_tok * 2, 128, (cuuint64_t)st_head * 2, (cuuint64_t)st_blk * 2};
  const cuuint32_t box[5] = {64, (cuuint32_t)box_tok, 1, 1, 1};
  return make_tmap_bf16_sw128(map, base, 5, dims, strides, box);
}

}  // namespace

bool prefill_supported(const diffqkv_shape& s, const diffqkv_cache& c, int* box_tok) {
  if (s.dtype != DIFFQKV_BF16) return false;
  const bool dims_ok = (s.d_qk == 128 && s.d_v == 128) || (s.d_qk == 64 && s.d_v == 64) || (s.d_qk == 64 && s.d_v == 128);
  if (!dims_ok) return false;
  // The kernel takes the row maximum of the raw scores and scales it afterwards, which keeps the order only for a
  // positive scale; zero and negative scales go to the generic kernel.
  if (!(s.scale > 0.f)) return false;
  int bt = kKT;
  if (c.page_table) {
    if (c.page_size >= kKT) { if (c.page_size % kKT != 0) return false; }
    else { if (c.page_size < 8 || kKT % c.page_size != 0) return false; bt = c.page_size; }
  }
  *box_tok = bt;
  return true;
}

// The cache update alone: rows past_b .. past_b + q_len - 1 of both pools (any strides, paged or contiguous, bf16 or fp32).
cudaError_t launch_cache_append(const void* k_new, const void* v_new, int q_len, const diffqkv_cache& c,
                                const diffqkv_shape& s, int* dev_status, cudaStream_t stream) {
  const int epv = s.dtype == DIFFQKV_BF16 ? 8 : 4;  // elements per 16-byte vector
  AppendParams a;
  a.k_new = reinterpret_cast<const uint4*>(k_new);
  a.v_new = reinterpret_cast<const uint4*>(v_new);
  a.k_cache = reinterpret_cast<uint4*>(c.k_cache);
  a.v_cache = reinterpret_cast<uint4*>(c.v_cache);
  a.k_sb = c.k_stride_blk / epv; a.k_sh = c.k_stride_head / epv; a.k_st = c.k_stride_tok / epv;
  a.v_sb = c.v_stride_blk / epv; a.v_sh = c.v_stride_head / epv; a.v_st = c.v_stride_tok / epv;
  a.seqlens = c.seqlens; a.page_table = c.page_table;
  a.page_size = c.page_size; a.max_pages_per_seq = c.max_pages_per_seq;
  a.num_blocks = c.num_blocks; a.max_seqlen = c.max_seqlen;
  a.batch = s.batch; a.q_len = q_len; a.n_k = s.n_k; a.n_v = s.n_v;
  a.vec_k = s.d_qk / epv; a.vec_v = s.d_v / epv;
  a.dev_status = dev_status;
  const long long vecs = (long long)s.batch * q_len * ((long long)s.n_k * a.vec_k + (long long)s.n_v * a.vec_v);
  if (vecs == 0) return cudaSuccess;
  long long blocks = (vecs + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  cache_append_kernel<<<(unsigned)blocks, 256, 0, stream>>>(a);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_prefill(const void* q, const void* k_new, const void* v_new, int q_len, const diffqkv_cache& c,
                           const diffqkv_shape& s, int box_tok, void* out, float* lse, int* dev_status,
                           cudaStream_t stream) {
  // Tensor maps first: when one cannot be built the caller runs both steps on the generic kernels, and nothing
  // has been launched yet.
  const int d = s.d_qk;
  CUtensorMap mq, mk, mv;
  {
    const cuuint64_t dims[5] = {64, (cuuint64_t)q_len, (cuuint64_t)(d / 64), (cuuint64_t)s.n_q, (cuuint64_t)s.batch};
    const cuuint64_t strides[4] = {(cuuint64_t)s.n_q * d * 2, 128, (cuuint64_t)d * 2,
                                   (cuuint64_t)q_len * s.n_q * d * 2};
    const cuuint32_t box[5] = {64, kQT, (cuuint32_t)(d / 64), 1, 1};
    if (!make_tmap_bf16_sw128(&mq, q, 5, dims, strides, box)) return cudaErrorNotSupported;
  }
  const long long tok_extent = c.page_table ? c.page_size : c.max_seqlen;
  if (!make_cache_map(&mk, c.k_cache, d, tok_extent, s.n_k, c.num_blocks, c.k_stride_tok, c.k_stride_head,
                      c.k_stride_blk, box_tok) ||
      !make_cache_map(&mv, c.v_cache, s.d_v, tok_extent, s.n_v, c.num_blocks, c.v_stride_tok, c.v_stride_head,
                      c.v_stride_blk, box_tok))
    return cudaErrorNotSupported;
  // ---- step 1: cache update
  cudaError_t err = launch_cache_append(k_new, v_new, q_len, c, s, dev_status, stream);
  if (err != cudaSuccess) return err;
  // ---- step 2: attention over the cache
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
  using PrefillFn = void (*)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const PrefillParams);
  const PrefillFn fn = s.d_v == 64 ? prefill_attn_kernel<64, 64>
                                   : (d == 128 ? prefill_attn_kernel<128, 128> : prefill_attn_kernel<64, 128>);
  err = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, kPrefillSmem);
  if (err != cudaSuccess) return err;
  fn<<<(unsigned)grid, kPrefillThreads, kPrefillSmem, stream>>>(mq, mk, mv, p);
  count_launch();
  return cudaGetLastError();
}

}  // namespace diffqkv
