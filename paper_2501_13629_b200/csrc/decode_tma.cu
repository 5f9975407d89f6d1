// DiffQKV split-sequence decode for bf16 caches on sm_100a: TMA-fed shared-memory ring, warp-level
// tensor-core scoring, probabilities reused across the group's V heads.
//
// Work decomposition.  Query heads are handled in "units": U = n_q / min(n_k, n_v) consecutive query
// heads that share K heads and V heads among themselves only (Eq. (idx) of the paper makes the head
// maps contiguous blocks).  A unit holds KPU = n_k / min K heads and VPU = n_v / min V heads, one of
// the two being 1; where that makes tiles smaller than 32 KB, up to four neighbouring units are taken
// together as one.  The sequence axis is cut into tiles of 64 tokens.  All (sequence, unit, tile)
// triples, in that order, form one flat list that is divided evenly over the persistent blocks of
// the grid; a maximal run of one block's tiles inside one (sequence, unit) is a segment and yields
// one partial result (or the final result when the segment covers the whole sequence).
//
// Per block: one producer warp issues TMA loads of the K tile(s) and V tile(s) of each 64-token tile
// into a ring of stages (128-byte swizzle, completion counted on an mbarrier per stage); four
// consumer warps each own 16 tokens of a tile:
//   S^T[16 tok x 8 heads] = K[16 tok x d] . Q^T        mma.sync m16n8k16, K rows via ldmatrix
//   online softmax over tokens per head column         warp shuffles across the 8 row groups
//   O^T[d x 8 heads] += V^T[d x 16 tok] . P^T          V via ldmatrix.trans, P^T via movmatrix
// so every K and V byte is read from shared memory exactly once and scored against all query
// heads of its unit.  Accumulation is fp32; P is rounded to bf16 for the second product and the
// softmax denominator sums the rounded values.
//
// Tail balance.  Equal shares do not finish at the same time (blocks end several microseconds apart on a step of
// 60), so the last few tiles of every block's last segment are not owned but pooled with those of the other blocks
// whose last segment lies in the same (sequence, unit) row; the blocks of a row draw from their pool one tile at a
// time through a counter in the workspace, and a block that runs ahead ends up with more tiles than one that runs
// behind.  A drawn tile joins the running softmax state of the drawing block's segment (the state does not care
// which tokens it has seen), so the number of partial results stays the same.  The counters carry the call's
// epoch, so that nothing has to be zeroed between calls and a counter of an earlier call is recognised as such.
#include <cuda.h>

#include <atomic>
#include <vector>
#include <mutex>
#include <random>

#include "common.cuh"
#include "ptx.cuh"
#include "tmap.cuh"
#include "walker.cuh"

namespace diffqkv {
namespace {

constexpr int kTT = 64;             // tokens per tile
constexpr int kConsumerWarps = 4;   // 16 tokens each
constexpr int kThreads = (kConsumerWarps + 1) * 32;
// Shared-memory layout of one head's 64-token tile with D channels: rows of 128 bytes (64 channels,
// 128-byte swizzle).  One TMA box brings `box_tok` tokens of all D/64 channel halves, so the tile is
// [token part][channel half][box_tok rows]; with box_tok = 64 that is simply [half][64 rows].
constexpr int kHeadsPerMma = 8;
constexpr int kMaxBatchTma = 2048;  // the per-sequence tile prefix lives in shared memory
// Hook state: process-wide, set and read from any calling thread, hence atomics.
std::atomic<int> g_max_blocks{0};     // tuning / test hook: 0 = one block per SM
std::atomic<int> g_cluster_mode{-1};  // test hook: -1 = automatic, 0 = never, 1 = whenever the shape allows
std::atomic<int> g_tail_reserve{-1};  // tuning / test hook: -1 = automatic, 0 = no reserve, n = at most n tiles per block
std::atomic<long long> g_wait_limit_ns{0};  // test hook: 0 = the default limit of every bounded wait
std::atomic<long long> g_skip_tile{-1};     // test hook: flat tile whose copies are never issued (-1 = none)
constexpr int kAutoReserve = 8;     // tiles a block holds back at most (automatic mode)
constexpr int kEpochShift = 24;     // a reserve counter is (epoch << 24) | tiles taken

struct TmaParams {
  const __nv_bfloat16* q;
  const int* seqlens;
  const int* page_table;
  int page_size, max_pages_per_seq, num_blocks, max_seqlen;
  int batch, n_q, n_units, U;
  int hk_per_unit, hv_per_unit;  // KPU, VPU
  int k_shift, v_shift;          // units that share their K (V) head with 2^shift - 1 neighbours: head = (u * KPU) >> shift
  int box_tok;                   // tokens per TMA box (64, or the page size when smaller)
  int stages;
  float scale_log2;
  float* o_partial;    // [slots][U][d_v] normalised partial outputs
  float* lse_partial;  // [slots][U] base-2 log-sum-exp of the scaled scores
  int* meta;           // [batch + 1] exclusive prefix of tiles per sequence
  unsigned long long* steal;  // [grid] reserve counters, (epoch << 24) | tiles taken
  unsigned long long epoch;   // of this call, below 2^40
  int reserve;                // most tiles a block holds back for the tail (0 = none)
  int reserve_auto;           // 1: and never more than a sixth of a block's share
  unsigned long long wait_ns; // limit of every bounded wait
  long long skip_tile;        // test hook: flat tile whose copies the producer does not issue (-1 = none)
  int cluster;                // 0, or blocks per (sequence, unit) row: the row's blocks form a cluster and merge on chip
  void* out;
  float* lse;
  int out_is_f32;
  int* dev_status;
};

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

using Walker = FlatWalker;  // position in the flat (sequence, unit, tile) list

// SHARED: neighbouring units read the same K or V head (see k_shift / v_shift); the plain case keeps its own code.
template <int D_QK, int D_V, int KPU, int VPU, bool SHARED = false>
__global__ void __launch_bounds__(kThreads, 1)
decode_tma_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                  const TmaParams p) {
  constexpr int HK = D_QK / 64, HV = D_V / 64;  // 64-channel halves per row
  constexpr int K_TILE = kTT * D_QK * 2;        // bytes of one K head tile
  constexpr int V_TILE = kTT * D_V * 2;
  constexpr int STAGE_BYTES = KPU * K_TILE + VPU * V_TILE;
  constexpr int KS = D_QK / 16;  // k-steps of the score product
  constexpr int MT = D_V / 16;   // 16-channel blocks of the output
  constexpr int OROW = D_V + 4;  // padded row of the merge buffer (bank-conflict free)

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* stage_base = smem;
  float* obuf = reinterpret_cast<float*>(smem + (size_t)p.stages * STAGE_BYTES);  // [warps][8][OROW]
  float* mbuf = obuf + kConsumerWarps * kHeadsPerMma * OROW;                      // [warps][8]
  float* lbuf = mbuf + kConsumerWarps * kHeadsPerMma;                             // [warps][8]
  uint64_t* bars = reinterpret_cast<uint64_t*>(lbuf + kConsumerWarps * kHeadsPerMma);  // full[s], empty[s]
  volatile int* abort_flag = reinterpret_cast<int*>(bars + 2 * p.stages);         // set when a wait ran out
  int* prefix = const_cast<int*>(abort_flag) + 2;                                 // [batch + 1]
  int* lens_s = prefix + p.batch + 1;                                             // [batch] lengths, clamped
  volatile int* ctrl = lens_s + p.batch;  // [stages] tail phase: valid tokens of the tile in the stage, 0 = no more tiles
  // (cluster mode) this block's share of its row for the on-chip merge: [8 heads][D_V] normalised outputs and their
  // base-2 log-sum-exps, over the first stage of the ring, which is free once the block's last tile has been consumed
  float* xo = reinterpret_cast<float*>(stage_base);
  float* xl = xo + kHeadsPerMma * D_V;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t full0 = ptx::smem_u32(bars), empty0 = ptx::smem_u32(bars + p.stages);

  if (tid == 0) {
    *abort_flag = 0;
    for (int s = 0; s < p.stages; ++s) {
      ptx::mbar_init(full0 + 8 * s, 1);
      ptx::mbar_init(empty0 + 8 * s, kConsumerWarps);
    }
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmap_k);
    ptx::prefetch_tmap(&tmap_v);
  }
  // Everything above touches only this block's shared memory and the kernel parameters; from here on the
  // kernel reads what earlier work in the stream may still be producing (lengths, q, the cache).
  ptx::grid_dependency_wait();
  // This block's reserve counter starts at zero tiles taken, under this call's epoch (ordered before every draw of
  // this block by the barriers below; a draw of another block that comes earlier finds a stale epoch and moves on).
  if (p.reserve > 0 && tid == 0) atomicExch(p.steal + blockIdx.x, p.epoch << kEpochShift);
  // One round of global loads for the lengths (a dependent round trip costs most of a microsecond here); the
  // prefix below comes out of shared memory.  The per-sequence reads further down go to global memory again
  // (by then first-level cache hits): measured, that streams config 5 about 4 % faster than reading lens_s.
  for (int b = tid; b < p.batch; b += kThreads) lens_s[b] = min(max(p.seqlens[b], 0), p.max_seqlen);
  __syncthreads();
  // exclusive prefix of tiles per sequence (warp 0: per-lane chunks, then a warp scan)
  if (warp == 0) {
    const int per = (p.batch + 31) / 32;
    const int lo = lane * per, hi = min(p.batch, lo + per);
    int sum = 0;
    for (int b = lo; b < hi; ++b) sum += (lens_s[b] + kTT - 1) / kTT;
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    int run = incl - sum;
    for (int b = lo; b < hi; ++b) {
      prefix[b] = run;
      run += (lens_s[b] + kTT - 1) / kTT;
    }
    if (lane == 31) prefix[p.batch] = incl;
  }
  __syncthreads();
  if (blockIdx.x == 0)
    for (int b = tid; b <= p.batch; b += kThreads) p.meta[b] = prefix[b];

  const long long total = (long long)p.n_units * prefix[p.batch];
  // Only min(grid, total) blocks take part, so that every participating block owns at least one tile
  // (the combine kernel relies on the blocks between a row's first and last owner all having written).
  const long long nblk = min((long long)gridDim.x, total);
  if (!p.cluster && blockIdx.x >= nblk) return;
  long long g_begin = 0, g_end = 0;
  if (p.cluster) {
    // Cluster mode (short rows): the p.cluster blocks of a cluster share one (sequence, unit) row, each takes an equal
    // run of its tiles and the first block merges all of them out of the others' shared memory: no partials in global
    // memory and no second kernel.  Every thread of every block reaches the two cluster barriers at the end.
    const int row = (int)blockIdx.x / p.cluster, rank = (int)blockIdx.x % p.cluster;
    const int b = row / p.n_units, u = row % p.n_units;
    const long long nt = prefix[b + 1] - prefix[b];
    const long long lo = (long long)p.n_units * prefix[b] + u * nt;
    g_begin = lo + nt * rank / p.cluster;
    g_end = lo + nt * (rank + 1) / p.cluster;
  } else {
    g_begin = (total * blockIdx.x) / nblk;
    g_end = (total * (blockIdx.x + 1)) / nblk;
  }
  const bool have_tiles = g_begin < g_end;

  // ---- the tail reserve: the last R tiles of this block's last segment (never all of the segment)
  const int reserve = p.cluster ? 0 : (p.reserve_auto ? (int)min((long long)p.reserve, (total / nblk) / 6) : p.reserve);
  Walker wl;  // the row (sequence, unit) of the last segment
  wl.b = 0; wl.u = 0; wl.nt = 0; wl.t = 0; wl.g = 0;
  if (have_tiles) wl.seek(g_end - 1, prefix, p.batch, p.n_units);
  const long long row_lo = (long long)p.n_units * prefix[wl.b] + (long long)wl.u * wl.nt, row_hi = row_lo + wl.nt;
  const int R = reserve > 0 ? min(reserve, (int)(g_end - max(g_begin, row_lo)) - 1) : 0;
  const long long g_stat = g_end - R;  // tiles [g_begin, g_stat) are this block's own

  Walker w;
  w.b = 0; w.u = 0; w.nt = 0; w.t = 0; w.g = g_begin;
  if (have_tiles) w.seek(g_begin, prefix, p.batch, p.n_units);

  if (warp == kConsumerWarps) {
    // ------------------------------------------------------------------ producer warp
    // One TMA box per (head tile, token part): lane x < boxes owns box x of every tile.
    const int parts = kTT / p.box_tok;
    const int boxes = (KPU + VPU) * parts;
    const int my_tile = lane / parts, my_part = lane % parts;
    const bool my_is_k = my_tile < KPU;
    const uint32_t my_off = my_is_k ? my_tile * K_TILE + my_part * (p.box_tok * 128 * HK)
                                    : KPU * K_TILE + (my_tile - KPU) * V_TILE + my_part * (p.box_tok * 128 * HV);
    const uint32_t tile_part_bytes = (uint32_t)p.box_tok * 128u * (KPU * HK + VPU * HV);
    int stage = 0;
    uint32_t phase = 0;
    int issued = 0;
    bool ok = true;
    int len = min(max(p.seqlens[w.b], 0), p.max_seqlen);
    // page id of this lane's box for the tile about to be issued (fetched one tile ahead)
    auto fetch_blk = [&]() -> int {
      if (!p.page_table) return w.b;
      const int tok = w.t * kTT + my_part * p.box_tok;
      if (lane >= boxes || tok >= len) return 0;
      return p.page_table[(long long)w.b * p.max_pages_per_seq + tok / p.page_size];
    };
    // This lane's box of tile (unit u, tokens from tok0) of a sequence of `len` tokens into `stage`.
    auto issue_box = [&](int u, int tok0, int parts_valid, int blk, uint32_t bar) {
      if (lane < boxes && my_part < parts_valid) {
        const int tok = tok0 + my_part * p.box_tok;
        const int slot = p.page_table ? tok % p.page_size : tok;
        if (blk < 0 || blk >= p.num_blocks) {  // never read outside the pool: flag it, read block 0 instead
          report(p.dev_status, DIFFQKV_ERR_INDEX);
          blk = 0;
        }
        const uint32_t dst = ptx::smem_u32(stage_base + (size_t)stage * STAGE_BYTES) + my_off;
        if (SHARED) {
          if (my_is_k) ptx::tma_load_5d(dst, &tmap_k, bar, 0, slot, 0, ((u * KPU) >> p.k_shift) + my_tile, blk);
          else ptx::tma_load_5d(dst, &tmap_v, bar, 0, slot, 0, ((u * VPU) >> p.v_shift) + (my_tile - KPU), blk);
        } else {
          if (my_is_k) ptx::tma_load_5d(dst, &tmap_k, bar, 0, slot, 0, u * KPU + my_tile, blk);
          else ptx::tma_load_5d(dst, &tmap_v, bar, 0, slot, 0, u * VPU + (my_tile - KPU), blk);
        }
      }
    };
    int blk = fetch_blk();
    for (; w.g < g_stat; ++w.g) {
      if (issued >= p.stages) {
        if (!ptx::mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag, p.wait_ns)) {
          report(p.dev_status, DIFFQKV_ERR_TIMEOUT);
          ok = false;
          break;
        }
      }
      const int tok0 = w.t * kTT;
      const int parts_valid = min(parts, (len - tok0 + p.box_tok - 1) / p.box_tok);
      const uint32_t bar = full0 + 8 * stage;
      if (w.g != p.skip_tile) {  // (test hook: a tile that is never requested; its stage's barrier stays incomplete)
        if (lane == 0) ptx::mbar_arrive_expect_tx(bar, (uint32_t)parts_valid * tile_part_bytes);
        __syncwarp();
        issue_box(w.u, tok0, parts_valid, blk, bar);
      }
      ++issued;
      if (++stage == p.stages) { stage = 0; phase ^= 1; }
      if (++w.t == w.nt) {
        w.t = 0;
        if (++w.u == p.n_units) {
          w.u = 0;
          w.next_sequence(prefix, p.batch);
          if (w.b < p.batch) len = min(max(p.seqlens[w.b], 0), p.max_seqlen);
        }
      }
      if (w.g + 1 < g_stat) blk = fetch_blk();
    }
    if (reserve > 0 && ok) {
      // ---- tail: the reserves of the blocks whose last segment lies in this block's last row form a pool that all
      // of them draw from until it is empty, so that they finish within about a tile of each other whatever their
      // speeds were.  Lane 0 draws, the warp follows.
      const int len_l = min(max(p.seqlens[wl.b], 0), p.max_seqlen);
      auto draw = [&](int k) -> unsigned long long {  // raw old value of block k's counter (lane 0 only)
        return lane == 0 ? atomicAdd(p.steal + k, 1ull) : 0ull;
      };
      auto taken = [&](unsigned long long raw) -> uint32_t {  // tiles taken so far, huge when the counter is stale
        return (raw >> kEpochShift) == p.epoch ? (uint32_t)(raw & ((1ull << kEpochShift) - 1)) : 0xffffffffu;
      };
      auto issue_reserve_tile = [&](long long g) -> bool {  // flat tile g of this row
        if (issued >= p.stages && !ptx::mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag, p.wait_ns)) {
          report(p.dev_status, DIFFQKV_ERR_TIMEOUT);
          return false;
        }
        const int tok0 = (int)(g - row_lo) * kTT;
        const int parts_valid = min(parts, (len_l - tok0 + p.box_tok - 1) / p.box_tok);
        const uint32_t bar = full0 + 8 * stage;
        if (lane == 0) {
          ctrl[stage] = min(kTT, len_l - tok0);
          ptx::mbar_arrive_expect_tx(bar, (uint32_t)parts_valid * tile_part_bytes);
        }
        __syncwarp();
        int blk_t = wl.b;
        if (p.page_table && lane < boxes && my_part < parts_valid)
          blk_t = p.page_table[(long long)wl.b * p.max_pages_per_seq + (tok0 + my_part * p.box_tok) / p.page_size];
        issue_box(wl.u, tok0, parts_valid, blk_t, bar);
        ++issued;
        if (++stage == p.stages) { stage = 0; phase ^= 1; }
        return true;
      };
      // The pool: the reserves of up to 32 consecutive blocks whose last segment is in this row (lane i <-> block
      // k_first + i), numbered block after block; its counter is the slot of the pool's first block.
      const int k_lo = (int)(((row_lo + 1) * nblk - 1) / total), k_hi = (int)(((row_hi + 1) * nblk - 1) / total) - 1;
      const int k_first = k_lo + (((int)blockIdx.x - k_lo) & ~31);
      const int kc = k_first + lane;
      int Rc = 0;       // this lane's block: size of its reserve, first tile of it
      long long sc = 0;
      if (kc <= k_hi) {
        const long long kb = (total * kc) / nblk, ke = (total * (kc + 1)) / nblk;
        Rc = min(reserve, (int)(ke - max(kb, row_lo)) - 1);
        sc = ke - Rc;
      }
      int incl = Rc;  // tiles of the pool up to and including this lane's block
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
      }
      const uint32_t pool = (uint32_t)__shfl_sync(0xffffffffu, incl, 31);
      auto tile_of = [&](uint32_t idx) -> long long {  // flat tile of pool entry idx < pool
        const int src = __popc(__ballot_sync(0xffffffffu, (uint32_t)incl <= idx));
        const long long s0 = __shfl_sync(0xffffffffu, sc, src);
        const int before = __shfl_sync(0xffffffffu, incl - Rc, src);
        return s0 + ((int)idx - before);
      };
      // One tile per draw; the next draw is in flight while the current tile is issued.
      uint32_t cur = pool > 0 ? taken(__shfl_sync(0xffffffffu, draw(k_first), 0)) : 0u;
      while (cur < pool) {
        const unsigned long long next_raw = draw(k_first);
        if (!issue_reserve_tile(tile_of(cur))) { ok = false; break; }
        cur = taken(__shfl_sync(0xffffffffu, next_raw, 0));
      }
      if (ok) {  // tell the consumers that the segment is complete: a stage without data
        if (issued >= p.stages && !ptx::mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag, p.wait_ns)) {
          report(p.dev_status, DIFFQKV_ERR_TIMEOUT);
          ok = false;
        } else {
          // Every lane has polled the barrier on its own: all of them must have seen the slot free before lane 0
          // hands it to the consumers, whose release would otherwise complete the barrier's next phase under the
          // lanes still polling for this one (they would then wait until their limit and report a timeout).
          __syncwarp();
          if (lane == 0) {
            ctrl[stage] = 0;
            ptx::mbar_arrive(full0 + 8 * stage);
          }
          __syncwarp();
          ++issued;
          if (++stage == p.stages) { stage = 0; phase ^= 1; }
        }
      }
    }
    // All loads of this block are on their way: let the combine kernel (launched with programmatic stream
    // serialisation) become resident now rather than earlier -- blocks that wait for this grid take issue
    // slots while they wait.  It still waits for this whole grid to finish before it reads any partial.
    ptx::grid_launch_dependents();
    if (!ok) {
      // Give copies already in flight a bounded chance to land before the block's shared memory is released.
      for (int s = 0; s < min(issued, p.stages); ++s) {
        const int uses = (issued - s + p.stages - 1) / p.stages;
        ptx::mbar_wait(full0 + 8 * s, (uint32_t)(uses - 1) & 1u, nullptr, p.wait_ns);
      }
    }
    if (p.cluster) {  // the two barriers of the on-chip merge (see the end of the kernel)
      ptx::cluster_sync();
      ptx::cluster_sync();
    }
    return;
  }

  // -------------------------------------------------------------------- consumer warps
  const int g8 = lane >> 2, t4 = lane & 3;  // row group and column pair of the mma fragments
  const int heads_per_k = p.U / KPU, heads_per_v = p.U / VPU;
  const int row0 = warp * 16;  // this warp's token rows inside a tile
  const int bt_shift = 31 - __clz(p.box_tok), bt_mask = p.box_tok - 1;
  // 128-byte row index of (token row r, channel half h) inside a head tile with H halves
  auto row_index = [&](int r, int h, int H) { return (((r >> bt_shift) * H + h) << bt_shift) + (r & bt_mask); };
  int stage = 0;
  uint32_t phase = 0;
  bool dead = false;

  while (w.g < g_stat) {
    // ---- one segment: tiles [w.t, w.t + seg_tiles) of (sequence w.b, unit w.u); the block's last segment goes
    // on with whatever the producer draws from the reserves of this row, until it posts a stage without data
    const int seg_tiles = (int)min((long long)(w.nt - w.t), g_stat - w.g);
    const bool tail = reserve > 0 && w.g + seg_tiles == g_stat;
    const bool whole = (w.t == 0 && seg_tiles + (tail ? R : 0) == w.nt);
    const int len = min(max(p.seqlens[w.b], 0), p.max_seqlen);
    const long long wlin = (long long)w.b * p.n_units + w.u;

    // Q^T fragments (B operand): column g8 = head g8 of the unit, masked per K head of the unit
    uint32_t qf[KPU][KS][2];
    {
      const bool head_ok = g8 < p.U;
      const __nv_bfloat16* qrow = p.q + ((long long)w.b * p.n_q + (long long)w.u * p.U + (head_ok ? g8 : 0)) * D_QK;
#pragma unroll
      for (int i = 0; i < KPU; ++i) {
        const bool use = head_ok && (g8 / heads_per_k == i);
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
          qf[i][ks][0] = use ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 2 * t4) : 0u;
          qf[i][ks][1] = use ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 2 * t4 + 8) : 0u;
        }
      }
    }
    float m_run[2] = {-INFINITY, -INFINITY};
    float l_run[2] = {0.f, 0.f};
    float acc[VPU][MT][4];
#pragma unroll
    for (int j = 0; j < VPU; ++j)
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[j][mt][e] = 0.f;

    for (int it = 0; it < seg_tiles || tail; ++it) {
      // A wait that runs out marks the block dead: the warp stops waiting and computing but keeps
      // walking, so that it still meets the other warps at the named barriers below.
      if (dead && it >= seg_tiles) break;
      if (!dead && !ptx::mbar_wait(full0 + 8 * stage, phase, abort_flag, p.wait_ns)) {
        report(p.dev_status, DIFFQKV_ERR_TIMEOUT);
        dead = true;
        if (it >= seg_tiles) break;
      }
      int n_valid = dead ? 0 : min(kTT, len - (w.t + it) * kTT);
      if (it >= seg_tiles) {  // a tile out of a reserve, or the end of the segment
        n_valid = ctrl[stage];
        if (n_valid == 0) {
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(empty0 + 8 * stage);
          if (++stage == p.stages) { stage = 0; phase ^= 1; }
          break;
        }
      }
      unsigned char* st = stage_base + (size_t)stage * STAGE_BYTES;
      const uint32_t st_u32 = ptx::smem_u32(st);
      if (row0 < n_valid) {
        if (row0 + 16 > n_valid) {
          // ragged tail: rows past the sequence end hold whatever followed in memory; zero the V rows
          // (0 * NaN would poison the product) -- the scores of those rows are masked below.
          for (int x = lane; x < VPU * HV * 16 * 8; x += 32) {
            const int sub = x / 128, r = row0 + (x % 128) / 8, c = x % 8;
            if (r >= n_valid)
              *reinterpret_cast<uint4*>(st + KPU * K_TILE + (sub / HV) * V_TILE + row_index(r, sub % HV, HV) * 128 +
                                        c * 16) = make_uint4(0, 0, 0, 0);
          }
          __syncwarp();
        }
        // ---- scores S^T = K . Q^T (two accumulators to shorten the dependent mma chain)
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
        {
          const int r = row0 + (lane & 7) + 8 * ((lane >> 3) & 1);
          const int csel = lane >> 4;
          uint32_t rbase[HK];
#pragma unroll
          for (int h = 0; h < HK; ++h) rbase[h] = st_u32 + row_index(r, h, HK) * 128;
#pragma unroll
          for (int i = 0; i < KPU; ++i) {
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
              const int chunk = (ks % 4) * 2 + csel;
              uint32_t a[4];
              ptx::ldmatrix_x4(rbase[ks / 4] + i * K_TILE + ((chunk ^ (r & 7)) << 4), a);
              if (ks & 1) ptx::mma_bf16_16816(s1, a, qf[i][ks][0], qf[i][ks][1]);
              else ptx::mma_bf16_16816(s0, a, qf[i][ks][0], qf[i][ks][1]);
            }
          }
        }
        // ---- online softmax; thread holds rows g8, g8+8 and head columns 2*t4, 2*t4+1
        const bool v0 = row0 + g8 < n_valid, v1 = row0 + g8 + 8 < n_valid;
        float x[4];
        x[0] = v0 ? (s0[0] + s1[0]) * p.scale_log2 : -INFINITY;
        x[1] = v0 ? (s0[1] + s1[1]) * p.scale_log2 : -INFINITY;
        x[2] = v1 ? (s0[2] + s1[2]) * p.scale_log2 : -INFINITY;
        x[3] = v1 ? (s0[3] + s1[3]) * p.scale_log2 : -INFINITY;
        float mx[2] = {fmaxf(x[0], x[2]), fmaxf(x[1], x[3])};
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {
          mx[0] = fmaxf(mx[0], __shfl_xor_sync(0xffffffffu, mx[0], o));
          mx[1] = fmaxf(mx[1], __shfl_xor_sync(0xffffffffu, mx[1], o));
        }
        float alpha[2];
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const float m_new = fmaxf(m_run[c], mx[c]);  // finite: row0 < n_valid means a visible token
          alpha[c] = exp2f(m_run[c] - m_new);
          m_run[c] = m_new;
        }
        const uint32_t p_lo = pack_bf16(exp2f(x[0] - m_run[0]), exp2f(x[1] - m_run[1]));
        const uint32_t p_hi = pack_bf16(exp2f(x[2] - m_run[0]), exp2f(x[3] - m_run[1]));
        l_run[0] = l_run[0] * alpha[0] + bf16_lo(p_lo) + bf16_lo(p_hi);
        l_run[1] = l_run[1] * alpha[1] + bf16_hi(p_lo) + bf16_hi(p_hi);
        if (__any_sync(0xffffffffu, alpha[0] != 1.f || alpha[1] != 1.f)) {
#pragma unroll
          for (int j = 0; j < VPU; ++j)
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
              acc[j][mt][0] *= alpha[0]; acc[j][mt][1] *= alpha[1];
              acc[j][mt][2] *= alpha[0]; acc[j][mt][3] *= alpha[1];
            }
        }
        const uint32_t b0 = ptx::movmatrix_trans(p_lo);  // P^T: tokens 2*t4, 2*t4+1 of head g8
        const uint32_t b1 = ptx::movmatrix_trans(p_hi);  //      tokens 2*t4+8, 2*t4+9
        // ---- O^T += V^T . P^T for every V head of the unit
        {
          const int r = row0 + (lane & 7) + 8 * (lane >> 4);
          const int csel = (lane >> 3) & 1;
          uint32_t rbase[HV];
#pragma unroll
          for (int h = 0; h < HV; ++h) rbase[h] = st_u32 + KPU * K_TILE + row_index(r, h, HV) * 128;
#pragma unroll
          for (int j = 0; j < VPU; ++j) {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
              const int chunk = (mt % 4) * 2 + csel;
              uint32_t a[4];
              ptx::ldmatrix_x4_trans(rbase[mt / 4] + j * V_TILE + ((chunk ^ (r & 7)) << 4), a);
              ptx::mma_bf16_16816(acc[j][mt], a, b0, b1);
            }
          }
        }
        if (row0 + 16 > n_valid) ptx::fence_proxy_async();  // the zero fill above vs. the next TMA write
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(empty0 + 8 * stage);
      if (++stage == p.stages) { stage = 0; phase ^= 1; }
    }

    // ---- merge the four warps' (m, l, O) and write the segment's result
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
      l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], o);
      l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], o);
    }
    if (g8 == 0) {
      mbuf[warp * kHeadsPerMma + 2 * t4] = m_run[0];
      mbuf[warp * kHeadsPerMma + 2 * t4 + 1] = m_run[1];
      lbuf[warp * kHeadsPerMma + 2 * t4] = l_run[0];
      lbuf[warp * kHeadsPerMma + 2 * t4 + 1] = l_run[1];
    }
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const int col = 2 * t4 + c;
      if (col < p.U) {
        const int jv = col / heads_per_v;
        float* orow = obuf + (warp * kHeadsPerMma + col) * OROW;
#pragma unroll
        for (int j = 0; j < VPU; ++j) {
          if (j == jv) {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
              orow[mt * 16 + g8] = acc[j][mt][c];
              orow[mt * 16 + g8 + 8] = acc[j][mt][2 + c];
            }
          }
        }
      }
    }
    ptx::named_barrier_sync(1, kConsumerWarps * 32);
    {
      constexpr int TPH = (kConsumerWarps * 32) / kHeadsPerMma;  // 16 threads per head
      constexpr int CPT = D_V / TPH;                             // channels per thread
      const int col = tid / TPH, ch0 = (tid % TPH) * CPT;
      if (col < p.U) {
        float mw[kConsumerWarps], M = -INFINITY;
#pragma unroll
        for (int ww = 0; ww < kConsumerWarps; ++ww) {
          mw[ww] = mbuf[ww * kHeadsPerMma + col];
          M = fmaxf(M, mw[ww]);
        }
        float L = 0.f, o[CPT];
#pragma unroll
        for (int e = 0; e < CPT; ++e) o[e] = 0.f;
#pragma unroll
        for (int ww = 0; ww < kConsumerWarps; ++ww) {
          const float wgt = mw[ww] == -INFINITY ? 0.f : exp2f(mw[ww] - M);
          L += wgt * lbuf[ww * kHeadsPerMma + col];
          if (wgt != 0.f) {
            const float* src = obuf + (ww * kHeadsPerMma + col) * OROW + ch0;
#pragma unroll
            for (int e = 0; e < CPT; ++e) o[e] = fmaf(wgt, src[e], o[e]);
          }
        }
        const float inv = 1.f / L;
        const float lse2 = M + log2f(L);
        if (p.cluster) {  // this block's share of the row, for the first block of the cluster to merge
          float* dst = xo + col * D_V + ch0;
#pragma unroll
          for (int e = 0; e < CPT; ++e) dst[e] = o[e] * inv;
          if (ch0 == 0) xl[col] = lse2;
        } else if (whole) {
          const long long orow = ((long long)w.b * p.n_q + (long long)w.u * p.U + col) * D_V + ch0;
          if (p.out_is_f32) {
            float* dst = reinterpret_cast<float*>(p.out) + orow;
#pragma unroll
            for (int e = 0; e < CPT; ++e) dst[e] = o[e] * inv;
          } else {
            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.out) + orow;
#pragma unroll
            for (int e = 0; e < CPT; ++e) dst[e] = __float2bfloat16_rn(o[e] * inv);
          }
          if (p.lse && ch0 == 0) p.lse[(long long)w.b * p.n_q + (long long)w.u * p.U + col] = lse2 * kLn2;
        } else {
          const long long slot = blockIdx.x + wlin;
          float* dst = p.o_partial + (slot * p.U + col) * D_V + ch0;
#pragma unroll
          for (int e = 0; e < CPT; ++e) dst[e] = o[e] * inv;
          if (ch0 == 0) p.lse_partial[slot * p.U + col] = lse2;
        }
      }
    }
    ptx::named_barrier_sync(1, kConsumerWarps * 32);

    // advance to the next (sequence, unit)
    w.g += seg_tiles;
    w.t += seg_tiles;
    if (w.t == w.nt) {
      w.t = 0;
      if (++w.u == p.n_units) { w.u = 0; w.next_sequence(prefix, p.batch); }
    }
  }

  if (p.cluster) {
    // ---- on-chip merge of the row's shares.  A block without tiles (fewer tiles than blocks, an empty sequence)
    // contributes log-sum-exp -inf.  First barrier: every share is in place; then the first block of the cluster reads
    // them out of its peers' shared memory (same weights as the combine kernel: 2^(lse_r - max)) and writes the row;
    // second barrier: nobody leaves, and gives up its shared memory, before that is done.
    constexpr int TPH = (kConsumerWarps * 32) / kHeadsPerMma;
    constexpr int CPT = D_V / TPH;
    const int col = tid / TPH, ch0 = (tid % TPH) * CPT;
    if (!have_tiles && tid < kHeadsPerMma) xl[tid] = -INFINITY;
    ptx::cluster_sync();
    const int row = (int)blockIdx.x / p.cluster, rank = (int)blockIdx.x % p.cluster;
    if (rank == 0 && col < p.U) {
      const uint32_t xl_u32 = ptx::smem_u32(xl + col), xo_u32 = ptx::smem_u32(xo + col * D_V + ch0);
      float M = -INFINITY;
      for (int r = 0; r < p.cluster; ++r) M = fmaxf(M, ptx::ld_cluster_f32(ptx::cluster_map(xl_u32, r)));
      float L = 0.f, o[CPT];
#pragma unroll
      for (int e = 0; e < CPT; ++e) o[e] = 0.f;
      if (M > -INFINITY) {
        for (int r = 0; r < p.cluster; ++r) {
          const float lr = ptx::ld_cluster_f32(ptx::cluster_map(xl_u32, r));
          if (lr == -INFINITY) continue;
          const float wgt = exp2f(lr - M);
          L += wgt;
          const uint32_t src = ptx::cluster_map(xo_u32, r);
#pragma unroll
          for (int e = 0; e < CPT; e += 4) {
            const float4 v = ptx::ld_cluster_f32x4(src + e * 4);
            o[e] = fmaf(wgt, v.x, o[e]); o[e + 1] = fmaf(wgt, v.y, o[e + 1]);
            o[e + 2] = fmaf(wgt, v.z, o[e + 2]); o[e + 3] = fmaf(wgt, v.w, o[e + 3]);
          }
        }
      }
      const float inv = L > 0.f ? 1.f / L : 0.f;
      const int b = row / p.n_units, u = row % p.n_units;
      const long long orow = ((long long)b * p.n_q + (long long)u * p.U + col) * D_V + ch0;
      if (p.out_is_f32) {
        float* dst = reinterpret_cast<float*>(p.out) + orow;
#pragma unroll
        for (int e = 0; e < CPT; ++e) dst[e] = o[e] * inv;
      } else {
        __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.out) + orow;
#pragma unroll
        for (int e = 0; e < CPT; ++e) dst[e] = __float2bfloat16_rn(o[e] * inv);
      }
      if (p.lse && ch0 == 0)
        p.lse[(long long)b * p.n_q + (long long)u * p.U + col] = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
    }
    ptx::cluster_sync();
  }
}

// Merge of the segment partials written above: one block per output row (sequence, query head), the
// partials dealt round-robin to its four warps so that their loads are in flight together.
// A row whose sequence fits inside one block was already written in final form by the decode kernel.
// Launched with programmatic stream serialisation: everything before grid_dependency_wait() only
// touches inputs of the call (seqlens), so it overlaps the decode kernel's tail.
constexpr int kCombineSmallBatch = 256;
__global__ void __launch_bounds__(128)
combine_segments_kernel(const float* __restrict__ o_partial, const float* __restrict__ lse_partial,
                        const int* __restrict__ meta, const int* __restrict__ seqlens, int max_seqlen, int batch,
                        int n_q, int n_units, int U, int d_v, int grid_decode, void* __restrict__ out,
                        float* __restrict__ lse, int out_is_f32) {
  __shared__ float4 part[4][128];  // per-warp weighted sums, d_v <= 512
  ptx::grid_launch_dependents();   // whatever follows in the stream may begin its own prologue
  const long long row = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = (int)(row / n_q), h = (int)(row % n_q);
  const int u = h / U, col = h % U;
  int nt = 0;
  long long before = 0, all = 0;  // tiles of earlier sequences / of all sequences
  const bool small = batch <= kCombineSmallBatch;
  if (small) {
    for (int bb = lane; bb < batch; bb += 32) {
      const int t = (min(max(seqlens[bb], 0), max_seqlen) + kTT - 1) / kTT;
      all += t;
      if (bb < b) before += t;
      if (bb == b) nt = t;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      all += __shfl_xor_sync(0xffffffffu, all, o);
      before += __shfl_xor_sync(0xffffffffu, before, o);
      nt += __shfl_xor_sync(0xffffffffu, nt, o);
    }
  }
  ptx::grid_dependency_wait();
  if (!small) {
    nt = meta[b + 1] - meta[b];
    before = meta[b];
    all = meta[batch];
  }
  const long long total = (long long)n_units * all;
  float4* out4 = reinterpret_cast<float4*>(out);
  if (nt == 0) {  // empty sequence: the decode kernel never touched this row
    for (int ch = threadIdx.x * 4; ch < d_v; ch += 512) {
      if (out_is_f32) out4[(row * d_v + ch) >> 2] = make_float4(0.f, 0.f, 0.f, 0.f);
      else *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(out) + row * d_v + ch) = make_uint2(0u, 0u);
    }
    if (lse && threadIdx.x == 0) lse[row] = -INFINITY;
    return;
  }
  const long long base = (long long)n_units * before + (long long)u * nt;
  const long long nblk = min((long long)grid_decode, total);  // blocks that took part
  const long long first = ((base + 1) * nblk - 1) / total;    // block that owns flat tile `base`
  const long long last = ((base + nt) * nblk - 1) / total;
  if (first == last) return;  // single segment: final result already in place
  const long long wlin = (long long)b * n_units + u;
  const int n = (int)(last - first + 1);
  const float* lp = lse_partial + (first + wlin) * U + col;  // partial c at lp[c * U]
  const float* op = o_partial + ((first + wlin) * U + col) * d_v;  // partial c at op[c * U * d_v]
  // The first partials of this warp's share (channels 0 .. 127) are requested together with the log-sum-exps, so
  // that the step costs one trip to L2 and not two: it is all that is left on the stream once the split kernel ends.
  constexpr int kEarly = 4;
  float4 early[kEarly];
  const int ch_e = lane * 4;
#pragma unroll
  for (int i = 0; i < kEarly; ++i) {
    const int c = warp + 4 * i;
    early[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (c < n && ch_e < d_v) early[i] = *reinterpret_cast<const float4*>(op + (long long)c * U * d_v + ch_e);
  }
  float M = -INFINITY;
  for (int c = lane; c < n; c += 32) M = fmaxf(M, lp[(long long)c * U]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
  float L = 0.f;
  for (int c = lane; c < n; c += 32) L += exp2f(lp[(long long)c * U] - M);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
  for (int ch0 = 0; ch0 < d_v; ch0 += 128) {
    const int ch = ch0 + lane * 4;
    const bool in = ch < d_v;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
    int c = warp;
    if (ch0 == 0) {
#pragma unroll
      for (int i = 0; i < kEarly; ++i, c += 4)
        if (c < n) {
          const float wgt = exp2f(lp[(long long)c * U] - M);
          const float4 v = early[i];
          a.x = fmaf(wgt, v.x, a.x); a.y = fmaf(wgt, v.y, a.y); a.z = fmaf(wgt, v.z, a.z); a.w = fmaf(wgt, v.w, a.w);
        }
    }
#pragma unroll 4
    for (; c < n; c += 4) {
      const float wgt = exp2f(lp[(long long)c * U] - M);
      if (in) {
        const float4 v = *reinterpret_cast<const float4*>(op + (long long)c * U * d_v + ch);
        a.x = fmaf(wgt, v.x, a.x); a.y = fmaf(wgt, v.y, a.y); a.z = fmaf(wgt, v.z, a.z); a.w = fmaf(wgt, v.w, a.w);
      }
    }
    part[warp][ch0 / 4 + lane] = a;
  }
  __syncthreads();
  const float inv = 1.f / L;
  for (int i = threadIdx.x; i < d_v / 4; i += 128) {
    float4 a = part[0][i];
#pragma unroll
    for (int w = 1; w < 4; ++w) {
      const float4 v = part[w][i];
      a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
    }
    a.x *= inv; a.y *= inv; a.z *= inv; a.w *= inv;
    const int ch = i * 4;
    if (out_is_f32) {
      out4[(row * d_v + ch) >> 2] = a;
    } else {
      uint2 pk;
      pk.x = pack_bf16(a.x, a.y);
      pk.y = pack_bf16(a.z, a.w);
      *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(out) + row * d_v + ch) = pk;
    }
  }
  if (lse && threadIdx.x == 0) lse[row] = (M + log2f(L)) * kLn2;
}

// ---------------------------------------------------------------------------- host side
// Tensor map over one cache pool: dims (64 channels, token slot, channel half, head, block); one box
// brings box_tok tokens x all halves of one head, each half landing as 128-byte swizzled rows.
bool make_pool_map(CUtensorMap* map, const void* base, int d, long long tok_extent, int heads, long long blocks,
                   long long st_tok, long long st_head, long long st_blk, int box_tok) {
  TmapEncodeTiledFn fn = tmap_encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[5] = {64, (cuuint64_t)tok_extent, (cuuint64_t)(d / 64), (cuuint64_t)heads, (cuuint64_t)blocks};
  const cuuint64_t strides[4] = {(cuuint64_t)st_tok * 2, 128, (cuuint64_t)st_head * 2, (cuuint64_t)st_blk * 2};
  const cuuint32_t box[5] = {64, (cuuint32_t)box_tok, (cuuint32_t)(d / 64), 1, 1};
  const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  for (int i = 0; i < 4; ++i)
    if (strides[i] == 0 || strides[i] % 16 != 0 || strides[i] >= (1ull << 40)) return false;
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

struct DeviceInfo {
  int sms = 0;
  int max_smem = 0;
};
DeviceInfo device_info() {
  static std::mutex mu;
  static DeviceInfo info[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return DeviceInfo();
  std::lock_guard<std::mutex> lock(mu);
  if (info[dev].sms == 0) {
    cudaDeviceGetAttribute(&info[dev].sms, cudaDevAttrMultiProcessorCount, dev);
    cudaDeviceGetAttribute(&info[dev].max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  }
  return info[dev];
}

using KernelFn = void (*)(const CUtensorMap, const CUtensorMap, const TmaParams);
struct Variant {
  KernelFn fn;
  KernelFn fn_shared;  // the SHARED instantiation, where one exists (a shared pool has one head per unit)
  int stage_bytes;
  int d_v;
};

template <int D_QK, int D_V, int KPU, int VPU>
Variant variant() {
  KernelFn shared = nullptr;
  if constexpr (KPU == 1 || VPU == 1) shared = decode_tma_kernel<D_QK, D_V, KPU, VPU, true>;
  return Variant{decode_tma_kernel<D_QK, D_V, KPU, VPU>, shared, kTT * 2 * (KPU * D_QK + VPU * D_V), D_V};
}

bool pick_variant(int d_qk, int d_v, int kpu, int vpu, Variant* v) {
#define DIFFQKV_CASE(DQ, DV, KP, VP) \
  if (d_qk == DQ && d_v == DV && kpu == KP && vpu == VP) { *v = variant<DQ, DV, KP, VP>(); return true; }
  DIFFQKV_CASE(128, 128, 1, 1) DIFFQKV_CASE(128, 128, 1, 2) DIFFQKV_CASE(128, 128, 1, 4)
  DIFFQKV_CASE(128, 128, 2, 1) DIFFQKV_CASE(128, 128, 4, 1)
  DIFFQKV_CASE(64, 64, 1, 1) DIFFQKV_CASE(64, 64, 1, 2) DIFFQKV_CASE(64, 64, 1, 4)
  DIFFQKV_CASE(64, 64, 2, 1) DIFFQKV_CASE(64, 64, 4, 1)
  DIFFQKV_CASE(64, 128, 1, 1) DIFFQKV_CASE(64, 128, 1, 2) DIFFQKV_CASE(64, 128, 1, 4)
  DIFFQKV_CASE(64, 64, 2, 2) DIFFQKV_CASE(64, 64, 4, 4) DIFFQKV_CASE(64, 64, 2, 4) DIFFQKV_CASE(64, 64, 4, 2)
#undef DIFFQKV_CASE
  return false;
}

// How many clusters of `size` blocks of this kernel (one block per SM at `smem` bytes) the GPU runs at once; asked of
// the driver once per (kernel, shared memory, size) and device.
int max_active_clusters(KernelFn fn, int smem, int size) {
  struct Entry { KernelFn fn; int smem, size, dev, n; };
  static std::mutex mu;
  static std::vector<Entry> seen;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  std::lock_guard<std::mutex> lock(mu);
  for (const Entry& e : seen)
    if (e.fn == fn && e.smem == smem && e.size == size && e.dev == dev) return e.n;
  int n = 0;
  if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) == cudaSuccess) {
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)size;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)size);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaOccupancyMaxActiveClusters(&n, fn, &cfg) != cudaSuccess) {
      n = 0;
      cudaGetLastError();  // not an error of the call being served
    }
  }
  seen.push_back(Entry{fn, smem, size, dev, n});
  return n;
}

}  // namespace

bool tma_decode_supported(const diffqkv_shape& s, const diffqkv_cache& c, TmaPlan* plan) {
  if (s.dtype != DIFFQKV_BF16) return false;
  const int mn = s.n_k < s.n_v ? s.n_k : s.n_v;
  if (s.n_k % mn != 0 || s.n_v % mn != 0) return false;
  int U = s.n_q / mn, kpu = s.n_k / mn, vpu = s.n_v / mn, k_shift = 0, v_shift = 0;
  if (U > kHeadsPerMma) {
    // More query heads per unit than one MMA takes: cut the unit into sub-units of kHeadsPerMma query heads.  A
    // sub-unit needs its share of the unit's K and V heads, at least one each; neighbouring sub-units that share a
    // head stream it again (mostly out of L2: they run at the same time on other SMs).
    if (U % kHeadsPerMma != 0) return false;
    const int sub = U / kHeadsPerMma;
    auto share = [&](int& per_unit, int* shift) {  // heads per sub-unit, and how many sub-units share one (2^shift)
      if (per_unit >= sub) { if (per_unit % sub != 0) return false; per_unit /= sub; return true; }
      int sh = 0;
      while ((per_unit << sh) < sub) ++sh;
      if ((per_unit << sh) != sub) return false;  // powers of two only
      *shift = sh;
      per_unit = 1;
      return true;
    };
    if (!share(kpu, &k_shift) || !share(vpu, &v_shift)) return false;
    U = kHeadsPerMma;
  }
  if (s.batch > kMaxBatchTma || s.batch < 1) return false;
  Variant v;
  if (!pick_variant(s.d_qk, s.d_v, kpu, vpu, &v)) return false;
  if ((k_shift || v_shift) && !v.fn_shared) return false;
  // Small units make small tiles (16-24 KB per 64 tokens at d = 64), and the fixed cost per tile then shows.  Several
  // neighbouring units can share a tile: m units are one unit of m*U query heads with m*KPU K heads and m*VPU V
  // heads (the head maps are contiguous blocks, so nothing else changes).  Merge while the tile stays within 64 KB.
  if (v.stage_bytes < 32768) {
    for (int m = 4; m >= 2; m >>= 1) {
      Variant vm;
      if (U * m <= kHeadsPerMma && mn % m == 0 && pick_variant(s.d_qk, s.d_v, kpu * m, vpu * m, &vm) &&
          vm.stage_bytes <= 65536) {
        U *= m; kpu *= m; vpu *= m; v = vm;
        break;
      }
    }
  }
  int box_tok = kTT;
  if (c.page_table) {
    if (c.page_size % 16 != 0) return false;
    if (c.page_size < kTT) { if (kTT % c.page_size != 0) return false; box_tok = c.page_size; }
    else if (c.page_size % kTT != 0) return false;
  }
  const DeviceInfo di = device_info();
  if (di.sms <= 0) return false;
  const int fixed = 1024 + kConsumerWarps * kHeadsPerMma * (s.d_v + 4 + 2) * 4 + 2 * 16 * 8 + (2 * s.batch + 1) * 4 + 64 + 8 * 4;
  int stages = (di.max_smem - fixed) / v.stage_bytes;
  if (stages > 8) stages = 8;
  if (stages < 2) return false;
  const long long tiles_max = (long long)s.batch * (s.n_q / U) * ((c.max_seqlen + kTT - 1) / kTT);
  long long grid = di.sms;
  const int max_blocks = g_max_blocks.load();
  if (max_blocks > 0 && grid > max_blocks) grid = max_blocks;
  if (grid > tiles_max) grid = tiles_max;
  if (grid < 1) grid = 1;
  plan->U = U; plan->kpu = kpu; plan->vpu = vpu; plan->box_tok = box_tok; plan->stages = stages;
  plan->k_shift = k_shift; plan->v_shift = v_shift;
  plan->grid = (int)grid;
  plan->smem = fixed + stages * v.stage_bytes;
  plan->slots = grid + (long long)s.batch * (s.n_q / U);
  const int tail_reserve = g_tail_reserve.load();
  plan->reserve = tail_reserve < 0 ? kAutoReserve : tail_reserve;
  plan->reserve_auto = tail_reserve < 0;
  // Cluster mode: with few, short rows the step is mostly fixed costs (the partials' trip through global memory, the
  // second launch and its dependency, about 4 us), and a row's blocks can merge through each other's shared memory
  // instead.  The blocks per row are chosen (2 to 8, the portable cluster size) to cover as many SMs as possible with
  // all clusters resident at once (one block takes a whole SM's shared memory, and a cluster has to fit one GPC: the
  // driver says how many clusters of each size can run together).  It is taken when the streaming time lost on the
  // SMs left idle is less than those 4 us; lengths are not known here, so the cache's capacity stands in for them.
  plan->cluster = 0;
  const int mode = g_cluster_mode.load();
  // blocks per row for units of `u_heads` query heads on kernel `fn`, 0 when the mode does not pay
  auto blocks_per_row = [&](int u_heads, KernelFn fn, int smem, int stage_bytes) -> int {
    const long long rows = (long long)s.batch * (s.n_q / u_heads);
    if (mode == 0 || max_blocks > 0 || !fn || rows * 2 > di.sms) return 0;
    int best = 0;
    for (int per_row = 8; per_row >= 2; --per_row) {
      if (rows * per_row > di.sms || per_row <= best) continue;
      if (rows <= max_active_clusters(fn, smem, per_row)) best = per_row;
    }
    if (best < 2) return 0;
    const double cover = (double)(rows * best) / di.sms;
    const double cap_bytes = (double)rows * c.max_seqlen * (stage_bytes / kTT);
    // (below 0.85 of the SMs the rows' tiles also divide badly over the blocks: 16 rows of 64 tiles on 7 blocks
    // each measured slower than the two-kernel path on all 148 SMs)
    return (mode > 0 || (cover >= 0.85 && cap_bytes * (1.0 / cover - 1.0) <= 26e6)) ? best : 0;
  };
  int per_row = blocks_per_row(U, (k_shift || v_shift) ? v.fn_shared : v.fn, plan->smem, v.stage_bytes);
  if (per_row == 0 && mode != 0 && U % 2 == 0) {
    // Too few rows: halve the units.  Each half takes half of the unit's K and V heads, or shares the head when the
    // unit has only one (its two halves then stream that head twice, the second time mostly out of L2: they run at
    // the same time in neighbouring clusters).  Worth it only here, where the step is not bound by bandwidth.
    int kpu2 = kpu, vpu2 = vpu, ks2 = k_shift, vs2 = v_shift;
    if (kpu2 % 2 == 0) kpu2 /= 2; else if (kpu2 == 1) ++ks2; else kpu2 = 0;
    if (vpu2 % 2 == 0) vpu2 /= 2; else if (vpu2 == 1) ++vs2; else vpu2 = 0;
    Variant v2;
    if (kpu2 > 0 && vpu2 > 0 && pick_variant(s.d_qk, s.d_v, kpu2, vpu2, &v2) && (!(ks2 || vs2) || v2.fn_shared)) {
      int stages2 = (di.max_smem - fixed) / v2.stage_bytes;
      if (stages2 > 8) stages2 = 8;
      const int smem2 = fixed + stages2 * v2.stage_bytes;
      const int pr2 = stages2 >= 2 ? blocks_per_row(U / 2, (ks2 || vs2) ? v2.fn_shared : v2.fn, smem2, v2.stage_bytes) : 0;
      if (pr2 > 0) {
        per_row = pr2;
        U /= 2;
        plan->U = U; plan->kpu = kpu2; plan->vpu = vpu2; plan->k_shift = ks2; plan->v_shift = vs2;
        plan->stages = stages2;
        plan->smem = smem2;
      }
    }
  }
  if (per_row > 0) {
    const long long rows = (long long)s.batch * (s.n_q / U);
    plan->cluster = per_row;
    plan->grid = (int)(rows * per_row);
    plan->slots = plan->grid + rows;
    plan->reserve = 0;
    plan->reserve_auto = 0;
  }
  return true;
}

void set_tma_max_blocks(int n) { g_max_blocks = n > 0 ? n : 0; }
void set_tma_tail_reserve(int n) { g_tail_reserve = n < 0 ? -1 : (n > 4096 ? 4096 : n); }
void set_tma_cluster_mode(int mode) { g_cluster_mode = mode < 0 ? -1 : (mode > 0 ? 1 : 0); }
void set_tma_debug_timeout(long long wait_limit_ns, long long skip_tile) {
  g_wait_limit_ns = wait_limit_ns > 0 ? wait_limit_ns : 0;
  g_skip_tile = skip_tile >= 0 ? skip_tile : -1;
}

// Every launch gets an epoch of its own (below 2^40), counted up from a random start, so that a reserve counter
// left in a workspace by an earlier call, or whatever else the memory held, is not mistaken for this call's.
static unsigned long long next_epoch() {
  static std::atomic<unsigned long long> counter{[] {
    std::random_device rd;
    return ((unsigned long long)rd() << 20) ^ (unsigned long long)rd();
  }()};
  return counter.fetch_add(1, std::memory_order_relaxed) & ((1ull << 40) - 1);
}

size_t tma_decode_workspace_bytes(const diffqkv_shape& s, const TmaPlan& plan) {
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  return up((size_t)plan.slots * plan.U * s.d_v * 4) + up((size_t)plan.slots * plan.U * 4) +
         up((size_t)(s.batch + 1) * 4) + up((size_t)plan.grid * 8);
}

// Returns cudaErrorNotSupported when no tensor map can describe the cache (the caller then falls back to
// the generic kernel); any other error is a real launch failure.
cudaError_t launch_decode_tma(const void* q, const diffqkv_cache& c, const diffqkv_shape& s, const TmaPlan& plan,
                              void* workspace, void* out, float* lse, int* dev_status, cudaStream_t stream) {
  Variant v;
  if (!pick_variant(s.d_qk, s.d_v, plan.kpu, plan.vpu, &v)) return cudaErrorNotSupported;
  CUtensorMap mk, mv;
  const long long tok_extent = c.page_table ? c.page_size : c.max_seqlen;
  if (!make_pool_map(&mk, c.k_cache, s.d_qk, tok_extent, s.n_k, c.num_blocks, c.k_stride_tok, c.k_stride_head,
                     c.k_stride_blk, plan.box_tok) ||
      !make_pool_map(&mv, c.v_cache, s.d_v, tok_extent, s.n_v, c.num_blocks, c.v_stride_tok, c.v_stride_head,
                     c.v_stride_blk, plan.box_tok))
    return cudaErrorNotSupported;
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  TmaParams p;
  p.q = reinterpret_cast<const __nv_bfloat16*>(q);
  p.seqlens = c.seqlens;
  p.page_table = c.page_table;
  p.page_size = c.page_size; p.max_pages_per_seq = c.max_pages_per_seq;
  p.num_blocks = c.num_blocks; p.max_seqlen = c.max_seqlen;
  p.batch = s.batch; p.n_q = s.n_q; p.n_units = s.n_q / plan.U; p.U = plan.U;
  p.hk_per_unit = plan.kpu; p.hv_per_unit = plan.vpu;
  p.k_shift = plan.k_shift; p.v_shift = plan.v_shift;
  p.box_tok = plan.box_tok; p.stages = plan.stages;
  p.scale_log2 = s.scale * kLog2e;
  char* ws = reinterpret_cast<char*>(workspace);
  p.o_partial = reinterpret_cast<float*>(ws);
  ws += up((size_t)plan.slots * plan.U * s.d_v * 4);
  p.lse_partial = reinterpret_cast<float*>(ws);
  ws += up((size_t)plan.slots * plan.U * 4);
  p.meta = reinterpret_cast<int*>(ws);
  ws += up((size_t)(s.batch + 1) * 4);
  p.steal = reinterpret_cast<unsigned long long*>(ws);
  p.epoch = next_epoch();
  p.reserve = plan.reserve;
  p.reserve_auto = plan.reserve_auto;
  const long long wait_ns = g_wait_limit_ns.load();
  p.wait_ns = wait_ns > 0 ? (unsigned long long)wait_ns : ptx::kWaitLimitNs;
  p.skip_tile = g_skip_tile.load();
  p.cluster = plan.cluster;
  p.out = out; p.lse = lse; p.out_is_f32 = s.out_dtype == DIFFQKV_F32;
  p.dev_status = dev_status;

  const KernelFn fn = (plan.k_shift || plan.v_shift) ? v.fn_shared : v.fn;
  if (!fn) return cudaErrorNotSupported;
  cudaError_t err = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, plan.smem);
  if (err != cudaSuccess) return err;
  // both kernels may start before their predecessor in the stream has finished; each waits on the device
  // before it touches anything the predecessor may still be producing
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = (unsigned)(plan.cluster > 0 ? plan.cluster : 1);
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = plan.cluster > 0 ? 2 : 1;
  cfg.gridDim = dim3((unsigned)plan.grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = (size_t)plan.smem;
  err = cudaLaunchKernelEx(&cfg, fn, mk, mv, p);
  if (err != cudaSuccess) return err;
  count_launch();
  profile_after_split(stream);
  if (plan.cluster > 0) return cudaGetLastError();  // the rows were merged on chip
  cfg.numAttrs = 1;
  const long long rows = (long long)s.batch * s.n_q;
  cfg.gridDim = dim3((unsigned)rows);
  cfg.blockDim = dim3(128);
  cfg.dynamicSmemBytes = 0;
  err = cudaLaunchKernelEx(&cfg, combine_segments_kernel, (const float*)p.o_partial, (const float*)p.lse_partial,
                           (const int*)p.meta, c.seqlens, c.max_seqlen, s.batch, s.n_q, p.n_units, plan.U, s.d_v,
                           plan.grid, out, lse, p.out_is_f32);
  if (err != cudaSuccess) return err;
  count_launch();
  return cudaGetLastError();
}

}  // namespace diffqkv
