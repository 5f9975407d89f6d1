// Selective V cache fetching for decode (paper Section "Selective V Cache Fetching"): only the V vectors of the
// top-k attention scores of each query head enter the output, so V traffic drops from the whole cache to k rows
// per head while K is still streamed once.  Two kernels:
//
//   decode_scores_kernel   persistent blocks stream the K cache (TMA ring of 128-token tiles, 128-byte swizzle) and
//                          score every cached token against all query heads of its K head at once (mma.sync
//                          m16n8k16, fp32 accumulation); scores go to a workspace as fp32, already multiplied by
//                          scale * log2(e).  All (sequence, K head, tile) triples form one flat list divided evenly
//                          over one block per SM; tiles are independent, so nothing has to be merged.
//   topk_attend_kernel     one block per (sequence, query head) holds the row's scores in registers (64 per thread,
//                          32768 per pass), finds the k-th largest (radix select, 8 bits a pass over an order-
//                          preserving key, run on the few scores near the maximum), compacts the kept tokens in
//                          token order (equal scores: the earlier token first, as the definition says), takes the
//                          softmax over the kept scores, gathers the k V rows and accumulates them in fp32.
// Both are launched with programmatic stream serialisation and wait on the device before touching their inputs.
#include <cuda.h>

#include <atomic>

#include "common.cuh"
#include "ptx.cuh"
#include "walker.cuh"
#include "tmap.cuh"

namespace diffqkv {
namespace {

constexpr int kST = 128;            // tokens per K tile
constexpr int kTileWarps = 8;       // warps that score one tile together, 16 tokens each
// Teams of kTileWarps warps work on different tiles at the same time (team t takes every teams-th tile of the
// block's range): one team alone spends most of a tile waiting on its own dependent instructions.
__host__ __device__ constexpr int score_teams(int ng) { return ng <= 2 ? 2 : 1; }  // registers allow two up to 16 heads
__host__ __device__ constexpr int score_threads(int ng) { return (score_teams(ng) * kTileWarps + 1) * 32; }
constexpr int kMaxBatchScores = 2048;
constexpr int kMaxTopk = 1024;
constexpr int kMaxGroups = 4;       // query heads per K head <= 8 * kMaxGroups
constexpr int kAttendThreads = 512;

struct ScoreParams {
  const __nv_bfloat16* q;
  const int* seqlens;
  const int* page_table;
  int page_size, max_pages_per_seq, num_blocks, max_seqlen;
  int batch, n_q, n_k, g_k;  // g_k = query heads per K head
  int groups;                // ceil(g_k / 8)
  int box_tok, stages;
  long long lpad;            // row length of the score matrix
  float scale_log2;
  float* scores;             // [batch, n_q, lpad]
  float* bmax;               // [batch, n_q, lpad / 16] largest score of every 16 tokens
  int* dev_status;
};

using TileWalker = FlatWalker;  // position in the flat (sequence, K head, tile) list

template <int D_QK, int NG>  // NG: groups of 8 query heads per K head
__global__ void __launch_bounds__(score_threads(NG), 1)
decode_scores_kernel(const __grid_constant__ CUtensorMap tmap_k, const ScoreParams p) {
  constexpr int HK = D_QK / 64;            // 64-channel halves per row
  constexpr int K_TILE = kST * D_QK * 2;   // bytes of one K tile
  constexpr int KS = D_QK / 16;

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)p.stages * K_TILE);  // full[s], empty[s]
  volatile int* abort_flag = reinterpret_cast<int*>(bars + 2 * p.stages);
  int* prefix = const_cast<int*>(abort_flag) + 2;  // [batch + 1] tiles before each sequence

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t full0 = ptx::smem_u32(bars), empty0 = ptx::smem_u32(bars + p.stages);
  if (tid == 0) {
    *abort_flag = 0;
    for (int s = 0; s < p.stages; ++s) {
      ptx::mbar_init(full0 + 8 * s, 1);
      ptx::mbar_init(empty0 + 8 * s, kTileWarps);
    }
    ptx::fence_barrier_init();
    ptx::prefetch_tmap(&tmap_k);
  }
  ptx::grid_dependency_wait();  // from here on: inputs that earlier work in the stream may still be producing
  if (warp == 0) {
    const int per = (p.batch + 31) / 32;
    const int lo = min(p.batch, lane * per), hi = min(p.batch, lo + per);
    int sum = 0;
    for (int b = lo; b < hi; ++b) sum += (min(max(p.seqlens[b], 0), p.max_seqlen) + kST - 1) / kST;
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    int run = incl - sum;
    for (int b = lo; b < hi; ++b) {
      prefix[b] = run;
      run += (min(max(p.seqlens[b], 0), p.max_seqlen) + kST - 1) / kST;
    }
    if (lane == 31) prefix[p.batch] = incl;
  }
  __syncthreads();
  const long long total = (long long)p.n_k * prefix[p.batch];
  const long long nblk = min((long long)gridDim.x, total);
  if (blockIdx.x >= nblk) {
    ptx::grid_launch_dependents();
    return;
  }
  const long long g_begin = (total * blockIdx.x) / nblk, g_end = (total * (blockIdx.x + 1)) / nblk;
  TileWalker w;
  w.seek(g_begin, prefix, p.batch, p.n_k);

  constexpr int kTeams = score_teams(NG);
  if (warp == kTeams * kTileWarps) {
    // ------------------------------------------------------------------ producer warp: lane x owns token part x
    const int parts = kST / p.box_tok;
    const uint32_t my_off = lane * (p.box_tok * 128 * HK);
    int stage = 0, issued = 0;
    uint32_t phase = 0;
    bool ok = true;
    for (; w.g < g_end; w.advance(prefix, p.batch, p.n_k)) {
      const int len = min(max(p.seqlens[w.b], 0), p.max_seqlen);
      const int tok0 = w.t * kST;
      const int parts_valid = min(parts, (len - tok0 + p.box_tok - 1) / p.box_tok);
      int blk = w.b, slot = tok0 + lane * p.box_tok;
      if (p.page_table && lane < parts_valid) {
        const int tok = slot;
        blk = p.page_table[(long long)w.b * p.max_pages_per_seq + tok / p.page_size];
        slot = tok % p.page_size;
        if (blk < 0 || blk >= p.num_blocks) {  // never read outside the pool: flag it, read block 0 instead
          report(p.dev_status, DIFFQKV_ERR_INDEX);
          blk = 0;
        }
      }
      if (issued >= p.stages && !ptx::mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag)) {
        report(p.dev_status, DIFFQKV_ERR_TIMEOUT);
        ok = false;
        break;
      }
      const uint32_t bar = full0 + 8 * stage;
      if (lane == 0) ptx::mbar_arrive_expect_tx(bar, (uint32_t)parts_valid * p.box_tok * 128u * HK);
      __syncwarp();
      if (lane < parts_valid)
        ptx::tma_load_5d(ptx::smem_u32(smem + (size_t)stage * K_TILE) + my_off, &tmap_k, bar, 0, slot, 0, w.u, blk);
      ++issued;
      if (++stage == p.stages) { stage = 0; phase ^= 1; }
    }
    ptx::grid_launch_dependents();
    if (!ok) {
      for (int s = 0; s < min(issued, p.stages); ++s) {
        const int uses = (issued - s + p.stages - 1) / p.stages;
        ptx::mbar_wait(full0 + 8 * s, (uint32_t)(uses - 1) & 1u, nullptr);
      }
    }
    return;
  }

  // -------------------------------------------------------------------- consumer warps
  const int g8 = lane >> 2, t4 = lane & 3;
  const int bt_shift = 31 - __clz(p.box_tok), bt_mask = p.box_tok - 1;
  auto row_index = [&](int r, int h) { return (((r >> bt_shift) * HK + h) << bt_shift) + (r & bt_mask); };
  const int team = warp / kTileWarps, tw = warp % kTileWarps;
  int cur_b = -1, cur_u = -1, len = 0;
  float* srow = nullptr;  // score row of the first query head of the current K head
  float* brow = nullptr;  // its row of 16-token maxima
  const long long nbpad = p.lpad / 16;
  uint32_t qf[NG][KS][2];
  const int row0 = tw * 16;
  const int r = row0 + (lane & 7) + 8 * ((lane >> 3) & 1);
  const int csel = lane >> 4;
  uint32_t a_off[KS];  // byte offset of this lane's ldmatrix row in a stage, per 16-channel step
#pragma unroll
  for (int ks = 0; ks < KS; ++ks)
    a_off[ks] = row_index(r, ks / 4) * 128 + ((((ks % 4) * 2 + csel) ^ (r & 7)) << 4);
  for (int a = 0; a < team && w.g < g_end; ++a) w.advance(prefix, p.batch, p.n_k);
  for (int it = team; w.g < g_end; it += kTeams) {  // `it` counts the block's tiles: tile `it` sits in stage it % stages
    const int stage = it % p.stages;
    const uint32_t phase = (uint32_t)(it / p.stages) & 1u;
    if (w.b != cur_b || w.u != cur_u) {  // Q^T fragments of the query heads of this K head, 8 heads per group
      cur_b = w.b; cur_u = w.u;
      len = min(max(p.seqlens[w.b], 0), p.max_seqlen);
      srow = p.scores + ((long long)w.b * p.n_q + (long long)w.u * p.g_k) * p.lpad;
      brow = p.bmax + ((long long)w.b * p.n_q + (long long)w.u * p.g_k) * nbpad;
#pragma unroll
      for (int gq = 0; gq < NG; ++gq) {
        const int hq = gq * 8 + g8;
        const bool use = hq < p.g_k;
        const __nv_bfloat16* qrow = p.q + ((long long)w.b * p.n_q + (long long)w.u * p.g_k + (use ? hq : 0)) * D_QK;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
          qf[gq][ks][0] = use ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 2 * t4) : 0u;
          qf[gq][ks][1] = use ? *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 2 * t4 + 8) : 0u;
        }
      }
    }
    if (!ptx::mbar_wait(full0 + 8 * stage, phase, abort_flag)) {  // all warps give up at the same stage
      report(p.dev_status, DIFFQKV_ERR_TIMEOUT);
      break;
    }
    const int n_valid = min(kST, len - w.t * kST);
    if (row0 < n_valid) {
      const uint32_t st_u32 = ptx::smem_u32(smem + (size_t)stage * K_TILE);
      float s[NG][2][4];  // two accumulation chains per group (even and odd 16-channel steps)
#pragma unroll
      for (int gq = 0; gq < NG; ++gq)
#pragma unroll
        for (int e = 0; e < 4; ++e) s[gq][0][e] = s[gq][1][e] = 0.f;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) {
        uint32_t a[4];
        ptx::ldmatrix_x4(st_u32 + a_off[ks], a);
#pragma unroll
        for (int gq = 0; gq < NG; ++gq) ptx::mma_bf16_16816(s[gq][ks & 1], a, qf[gq][ks][0], qf[gq][ks][1]);
      }
      // thread holds token rows g8, g8 + 8 of the block and head columns 2 t4, 2 t4 + 1 of each group
      const long long tok = (long long)w.t * kST + row0 + g8;
#pragma unroll
      for (int gq = 0; gq < NG; ++gq) {
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const int hq = gq * 8 + 2 * t4 + c;
          const float lo = (s[gq][0][c] + s[gq][1][c]) * p.scale_log2;
          const float hi = (s[gq][0][2 + c] + s[gq][1][2 + c]) * p.scale_log2;
          float bm = fmaxf(row0 + g8 < n_valid ? lo : -INFINITY, row0 + g8 + 8 < n_valid ? hi : -INFINITY);
          bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 4));  // over the 16 tokens of the block
          bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 8));
          bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, 16));
          if (hq >= p.g_k) continue;
          float* dst = srow + (long long)hq * p.lpad + tok;
          if (row0 + g8 < n_valid) dst[0] = lo;
          if (row0 + g8 + 8 < n_valid) dst[8] = hi;
          if (g8 == 0) brow[(long long)hq * nbpad + w.t * (kST / 16) + tw] = bm;
        }
      }
    }
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive(empty0 + 8 * stage);
    for (int a = 0; a < kTeams && w.g < g_end; ++a) w.advance(prefix, p.batch, p.n_k);
  }
}

constexpr int kPiece = 32768;            // scores one selection holds in registers (64 per thread)
constexpr int kPerThread = kPiece / kAttendThreads;
constexpr int kQuads = kPerThread / 4;   // 16-byte loads per thread
constexpr int kWarpSpan = 32 * kPerThread;
constexpr int kMaxCand = 8192;           // keys the fast path of the selection holds; also the merge capacity
constexpr int kAttendWarps = kAttendThreads / 32;

constexpr int kMaxFlag = 1536;           // 16-token blocks the sparse selection copies to shared memory

struct AttendParams {
  const float* scores;
  const float* bmax;
  long long lpad;
  int general_only;  // test hook: skip the selection driven by the block maxima
  const __nv_bfloat16* v;
  long long v_sb, v_sh, v_st;
  const int* seqlens;
  const int* page_table;
  int page_size, max_pages_per_seq, num_blocks, max_seqlen;
  int batch, n_q, n_v, d_v, topk;
  void* out;
  float* lse;
  int out_is_f32;
  int* dev_status;
  int* kept_ids;  // [batch, n_q, topk] cached positions of the kept tokens (-1 padded), or NULL
};

// Larger float <=> larger key.
__device__ __forceinline__ uint32_t order_key(float x) {
  const uint32_t u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct SelectOut {
  int pos[kMaxTopk];
  float val[kMaxTopk];
};

struct SelectScratch {
  unsigned hist[4][256];  // one histogram per radix pass
  unsigned warp_tot[2][kAttendWarps];
  float warp_max[kAttendWarps], warp_min[kAttendWarps];
  unsigned prefix, need, count;
};

// From the top bin down: the bin of hist that holds the need-th largest of the keys counted there.  Warp 0 calls it;
// the winning lane publishes the prefix extended by the bin (at bit `shift`) and the rank that remains inside the bin.
__device__ __forceinline__ void pick_bin(const unsigned* hist, SelectScratch& sc, unsigned prefix, unsigned need,
                                         int shift) {
  const int lane = threadIdx.x & 31;
  unsigned mine = 0;  // lane owns bins 255 - 8 lane .. 248 - 8 lane
#pragma unroll
  for (int e = 0; e < 8; ++e) mine += hist[255 - (lane * 8 + e)];
  unsigned incl = mine;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  const unsigned before = incl - mine;
  if (before < need && need <= incl) {  // exactly one lane
    unsigned cum = before;
    for (int e = 0; e < 8; ++e) {
      const int bin = 255 - (lane * 8 + e);
      if (need <= cum + hist[bin]) {
        sc.prefix = prefix | ((unsigned)bin << shift);
        sc.need = need - cum;
        break;
      }
      cum += hist[bin];
    }
  }
}

// The k-th largest of a set of keys below 2^bits by radix select, up to 8 bits a pass from the top bit down: its key
// in *thr, and in *need_eq how many keys equal to it belong to the k largest.  count_pass(hist, top, shift, prefix)
// adds every key that agrees with prefix above bit `top` to hist[(key >> shift) & 255] (top - shift <= 8).  All
// threads of the block call it.  After max_passes passes it stops: *thr is then a lower bound (low bits zero).
template <typename CountPass>
__device__ void radix_kth(CountPass count_pass, int bits, int k, SelectScratch& sc, unsigned* thr, unsigned* need_eq,
                          int max_passes = 4) {
  const int tid = threadIdx.x;
  for (int i = tid; i < 4 * 256; i += kAttendThreads) (&sc.hist[0][0])[i] = 0;
  __syncthreads();
  unsigned prefix = 0, need = (unsigned)k;
  int pass = 0;
  for (int top = bits; top > 0 && pass < max_passes; ++pass) {
    const int shift = max(top - 8, 0);
    count_pass(sc.hist[pass], top, shift, prefix);
    __syncthreads();
    if (tid < 32) pick_bin(sc.hist[pass], sc, prefix, need, shift);
    __syncthreads();
    prefix = sc.prefix;
    need = sc.need;
    top = shift;
  }
  *thr = prefix;
  *need_eq = need;
}

// Do key and prefix agree in the bits from `top` up?
__device__ __forceinline__ bool same_above(unsigned key, unsigned prefix, int top) {
  return top >= 32 || (key >> top) == (prefix >> top);
}

// The k largest of vals[0 .. n) (shared or global memory, 16-byte aligned, n <= kPiece); of equal values the earlier
// position wins.  Their positions and values go to `out` in position order.  All threads of the block call it.
//
// Every thread keeps 64 values in registers: warp w, 16-byte load j, lane l hold positions 2048 w + 128 j + 4 l + c,
// so each load instruction of a warp reads 512 consecutive bytes.  The k-th largest value is first sought among the
// few values within a distance `band` of the maximum (every value outside is smaller than every value inside, so the
// rank is unchanged); the band doubles until it holds k values and is bisected back if it then holds more than the
// candidate buffer.  The candidates' keys are stored relative to the key of the band's lower end, which leaves few
// significant bits for the radix select.  Only when no band fits (values crowded on one point, or not finite) does
// the radix select run over all values.  A 64-bit mask per thread marks its candidates, so that the later steps touch
// only the 4-value groups that hold one.
__device__ __noinline__ void block_select(const float* vals, int n, int k, SelectOut& out, SelectScratch& sc,
                                          unsigned* cand_key) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int my0 = warp * kWarpSpan + lane * 4;  // position of quad j, element c: my0 + 128 j + c
  float sv[kPerThread];
  unsigned cm[2] = {0u, 0u};  // candidates: bit e of the pair; starts as "position below n"
#pragma unroll
  for (int j = 0; j < kQuads; ++j) {
    const int i = my0 + j * 128;
    float4 v = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    if (i + 3 < n) {
      v = *reinterpret_cast<const float4*>(vals + i);
      cm[j >> 3] |= 15u << (4 * (j & 7));
    } else if (i < n) {
      v.x = vals[i];
      if (i + 1 < n) v.y = vals[i + 1];
      if (i + 2 < n) v.z = vals[i + 2];
      cm[j >> 3] |= ((1u << (n - i)) - 1u) << (4 * (j & 7));
    }
    sv[4 * j] = v.x; sv[4 * j + 1] = v.y; sv[4 * j + 2] = v.z; sv[4 * j + 3] = v.w;
  }
  auto quad = [](const unsigned (&mk)[2], int j) { return (mk[j >> 3] >> (4 * (j & 7))) & 15u; };
  unsigned thr = 0, need_eq = 0;
  const bool all = n <= k;
  if (!all) {
    float m = -INFINITY;
#pragma unroll
    for (int e = 0; e < kPerThread; ++e) m = fmaxf(m, sv[e]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) sc.warp_max[warp] = m;
    __syncthreads();
    m = sc.warp_max[0];
#pragma unroll
    for (int ww = 1; ww < kAttendWarps; ++ww) m = fmaxf(m, sc.warp_max[ww]);

    int round = 0;
    unsigned ge[2] = {0u, 0u};
    auto count_ge = [&](float cut) {  // values >= cut in the block (cut finite: the padding never counts)
      ge[0] = ge[1] = 0u;
#pragma unroll
      for (int e = 0; e < kPerThread; ++e) ge[e >> 5] |= (unsigned)(sv[e] >= cut) << (e & 31);
      int c = __popc(ge[0]) + __popc(ge[1]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
      unsigned* tot = sc.warp_tot[round & 1];  // alternate buffers: one barrier a round is enough
      ++round;
      if (lane == 0) tot[warp] = (unsigned)c;
      __syncthreads();
      int total = 0;
#pragma unroll
      for (int ww = 0; ww < kAttendWarps; ++ww) total += (int)tot[ww];
      return total;
    };
    float cut = m, lo = 0.f, hi = 0.f;
    int count = 0;
    if (m > -INFINITY && m < INFINITY) {
      for (hi = 1.f; hi < 1e30f; hi *= 2.f) {
        cut = m - hi;
        count = count_ge(cut);
        if (count >= k) break;
        lo = hi;
      }
      for (int it = 0; it < 12 && count > kMaxCand; ++it) {  // too many: bisect between the last two bands
        const float mid = 0.5f * (lo + hi);
        cut = m - mid;
        count = count_ge(cut);
        if (count < k) { lo = mid; count = kMaxCand + 1; } else hi = mid;
      }
    }
    if (count >= k && count <= kMaxCand) {
      cm[0] = ge[0]; cm[1] = ge[1];
      // every thread appends its own candidates (any order will do for the rank)
      const int mine = __popc(cm[0]) + __popc(cm[1]);
      int incl = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
      }
      if (tid == 0) sc.count = 0;
      __syncthreads();
      unsigned base = 0;
      if (lane == 31 && incl) base = atomicAdd(&sc.count, (unsigned)incl);
      base = __shfl_sync(0xffffffffu, base, 31) + (unsigned)(incl - mine);
      const unsigned key_cut = order_key(cut);
#pragma unroll
      for (int j = 0; j < kQuads; ++j) {
        const unsigned c4 = quad(cm, j);
        if (c4 == 0) continue;
#pragma unroll
        for (int c = 0; c < 4; ++c)
          if ((c4 >> c) & 1u) cand_key[base++] = order_key(sv[4 * j + c]) - key_cut;
      }
      __syncthreads();
      const int ncand = count;
      const unsigned span = order_key(m) - key_cut;
      radix_kth(
          [&](unsigned* hist, int top, int shift, unsigned prefix) {
            for (int i = tid; i < ncand; i += kAttendThreads) {
              const unsigned key = cand_key[i];
              if (same_above(key, prefix, top)) atomicAdd(&hist[(key >> shift) & 255u], 1u);
            }
          },
          span ? 32 - __clz(span) : 0, k, sc, &thr, &need_eq);
      thr += key_cut;
    } else {
      radix_kth(
          [&](unsigned* hist, int top, int shift, unsigned prefix) {
#pragma unroll
            for (int e = 0; e < kPerThread; ++e) {
              const unsigned key = order_key(sv[e]);
              if (((cm[e >> 5] >> (e & 31)) & 1u) && same_above(key, prefix, top))
                atomicAdd(&hist[(key >> shift) & 255u], 1u);
            }
          },
          32, k, sc, &thr, &need_eq);
    }
  }
  // compaction in position order: kept = key > thr, or key == thr among the first need_eq such positions
  unsigned gm[2] = {0u, 0u}, qm[2] = {0u, 0u};
#pragma unroll
  for (int j = 0; j < kQuads; ++j) {
    const unsigned c4 = quad(cm, j);
    if (c4 == 0) continue;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      if (!((c4 >> c) & 1u)) continue;
      const unsigned key = order_key(sv[4 * j + c]);
      const unsigned bit = 1u << (4 * (j & 7) + c);
      if (all || key > thr) gm[j >> 3] |= bit;
      else if (key == thr) qm[j >> 3] |= bit;
    }
  }
  // kept-for-sure count in the low half, equal-to-threshold count in the high half
  unsigned packed = (__popc(gm[0]) + __popc(gm[1])) | ((unsigned)(__popc(qm[0]) + __popc(qm[1])) << 16);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) packed += __shfl_xor_sync(0xffffffffu, packed, o);
  unsigned* tot = sc.warp_tot[0];
  __syncthreads();  // earlier uses of the totals are over
  if (lane == 0) tot[warp] = packed;
  __syncthreads();
  unsigned run = 0;
  for (int ww = 0; ww < warp; ++ww) run += tot[ww];
#pragma unroll
  for (int j = 0; j < kQuads; ++j) {
    const unsigned g4 = quad(gm, j), q4 = quad(qm, j);
    if (__ballot_sync(0xffffffffu, (g4 | q4) != 0) == 0) continue;  // nothing of this warp's 128 positions is kept
    const unsigned cnt = __popc(g4) | ((unsigned)__popc(q4) << 16);
    unsigned incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    const unsigned before = run + incl - cnt;
    unsigned gt_before = before & 0xffffu, eq_before = before >> 16;
    if (g4 | q4) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const bool g = (g4 >> c) & 1u, q = (q4 >> c) & 1u;
        if (g || (q && eq_before < need_eq)) {
          const unsigned pos = gt_before + min(eq_before, need_eq);
          out.pos[pos] = my0 + j * 128 + c;
          out.val[pos] = sv[4 * j + c];
        }
        gt_before += g;
        eq_before += q;
      }
    }
    run += __shfl_sync(0xffffffffu, incl, 31);
  }
  __syncthreads();
}

// Exclusive prefix of v over the threads of the block, in thread order, and the block's total.
__device__ __noinline__ unsigned block_scan(unsigned v, unsigned* total, SelectScratch& sc) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  __syncthreads();  // earlier readers of the totals are done
  if (lane == 31) sc.warp_tot[0][warp] = incl;
  __syncthreads();
  unsigned before = incl - v, t = 0;
#pragma unroll 1
  for (int ww = 0; ww < kAttendWarps; ++ww) {
    const unsigned x = sc.warp_tot[0][ww];
    if (ww < warp) before += x;
    t += x;
  }
  *total = t;
  return before;
}

// radix_kth over keys[i] - rebase, i < n, keys in shared memory.  One copy of the code serves both selections of the
// sparse path: the kernel runs once per block, so what it costs is mostly the instructions it has to fetch.
__device__ __noinline__ void radix_kth_shared(const unsigned* keys, int n, unsigned rebase, int bits, int k,
                                              int max_passes, SelectScratch& sc, unsigned* thr, unsigned* need_eq) {
  const int tid = threadIdx.x;
  radix_kth(
      [&](unsigned* hist, int top, int shift, unsigned prefix) {
#pragma unroll 1
        for (int i = tid; i < n; i += kAttendThreads) {
          const unsigned key = keys[i] - rebase;
          if (same_above(key, prefix, top)) atomicAdd(&hist[(key >> shift) & 255u], 1u);
        }
      },
      bits, k, sc, thr, need_eq, max_passes);
}

constexpr int kSparseCand = 4096;  // candidates the sparse selection holds

// The same result as block_select over a whole row of `len` scores, found from the maxima of its 16-token blocks
// (bm): the k-th largest block maximum is a lower bound of the k-th largest score (k blocks hold k scores at least
// that large), so only blocks whose maximum reaches it can hold a kept score.  Those few blocks are copied to shared
// memory, their scores at or above the bound become the candidates (in token order), the exact k-th largest is found
// among them and the kept ones are compacted in token order.  The bound is taken from two radix passes only, i.e.
// rounded down to 16 significant bits of the maxima's range.  Returns false, the same for all threads, when the
// values do not suit it (not finite, or so crowded that the blocks or candidates overflow their buffers); nothing is
// written to `out` then.  The loops are kept rolled and the helpers shared on purpose (see radix_kth_shared).
//   keys      kMaxCand words: the block maxima's keys, later the candidates' keys (first half) and values (second)
//   cpos      kSparseCand candidates' tokens;  flag_id, foff: kMaxFlag words each;  stage: kMaxFlag * 16 scores
__device__ __noinline__ bool block_select_sparse(const float* row, const float* bm, int len, int k, SelectOut& out,
                                                 SelectScratch& sc, unsigned* keys, int* cpos, int* flag_id,
                                                 int* foff, float4* stage) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nblk = (len + 15) >> 4;
  if (nblk > kMaxCand) return false;
  float mx = -INFINITY, mn = INFINITY;
#pragma unroll 1
  for (int i = tid; i < nblk; i += kAttendThreads) {
    const float v = bm[i];
    keys[i] = order_key(v);
    mx = fmaxf(mx, v);
    mn = fminf(mn, v);
    if (!(v == v)) mn = -INFINITY;  // not a number: give up below
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
  }
  __syncthreads();
  if (lane == 0) { sc.warp_max[warp] = mx; sc.warp_min[warp] = mn; }
  __syncthreads();
#pragma unroll 1
  for (int ww = 0; ww < kAttendWarps; ++ww) {
    mx = fmaxf(mx, sc.warp_max[ww]);
    mn = fminf(mn, sc.warp_min[ww]);
  }
  if (!(mx < INFINITY && mn > -INFINITY)) return false;
  const unsigned key_min = order_key(mn), key_max = order_key(mx);
  unsigned pre = 0, dummy = 0;
  // With fewer blocks than kept scores the maxima bound nothing: every finite score is a candidate (the key just
  // above that of -inf, which is what positions past the row's end hold in the staging area).
  unsigned cut_key = order_key(-INFINITY) + 1u;
  if (k < nblk) {
    radix_kth_shared(keys, nblk, key_min, key_max != key_min ? 32 - __clz(key_max - key_min) : 0, k, 2, sc, &pre, &dummy);
    cut_key = key_min + pre;  // at most the k-th largest block maximum
  }

  // ---- the blocks that can hold a kept score, in order
  const int per = (nblk + kAttendThreads - 1) / kAttendThreads;
  const int b_lo = min(nblk, tid * per), b_hi = min(nblk, b_lo + per);
  unsigned cnt = 0;
#pragma unroll 1
  for (int i = b_lo; i < b_hi; ++i) cnt += keys[i] >= cut_key;
  unsigned nflag = 0;
  unsigned at = block_scan(cnt, &nflag, sc);
  if (nflag > (unsigned)kMaxFlag) return false;
#pragma unroll 1
  for (int i = b_lo; i < b_hi; ++i)
    if (keys[i] >= cut_key) flag_id[at++] = i;
  __syncthreads();

  // ---- copy them to shared memory, 16 bytes per thread and step (one trip to memory for all of them; positions past
  // the row's end become -inf); block f's quad q goes to stage[4 f + (q ^ (f & 3))], which spreads the banks
#pragma unroll 4
  for (int i = tid; i < 4 * (int)nflag; i += kAttendThreads) {
    const int f = i >> 2, q = i & 3;
    const int pos = flag_id[f] * 16 + q * 4;
    float4 v = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    if (pos + 3 < len) {
      v = *reinterpret_cast<const float4*>(row + pos);
    } else {
      if (pos < len) v.x = row[pos];
      if (pos + 1 < len) v.y = row[pos + 1];
      if (pos + 2 < len) v.z = row[pos + 2];
    }
    stage[4 * f + (q ^ (f & 3))] = v;
  }
  __syncthreads();
  // ---- candidates = staged scores at or above the bound: a thread per block counts, the counts become offsets, the
  // thread copies its block's candidates in token order
#pragma unroll 1
  for (int f = tid; f < (int)nflag; f += kAttendThreads) {
    int c = 0;
#pragma unroll 1
    for (int q = 0; q < 4; ++q) {
      const float4 v = stage[4 * f + (q ^ (f & 3))];
      c += (order_key(v.x) >= cut_key) + (order_key(v.y) >= cut_key) + (order_key(v.z) >= cut_key) +
           (order_key(v.w) >= cut_key);
    }
    foff[f] = c;
  }
  __syncthreads();
  const int per2 = ((int)nflag + kAttendThreads - 1) / kAttendThreads;
  const int f_lo = min((int)nflag, tid * per2), f_hi = min((int)nflag, f_lo + per2);
  cnt = 0;
#pragma unroll 1
  for (int i = f_lo; i < f_hi; ++i) cnt += (unsigned)foff[i];
  unsigned ncand = 0;
  at = block_scan(cnt, &ncand, sc);
  // fewer candidates than kept scores can only mean scores of -inf among the k largest: leave those rows to the
  // selection over all scores
  if (ncand > (unsigned)kSparseCand || ncand < (unsigned)k) return false;
#pragma unroll 1
  for (int i = f_lo; i < f_hi; ++i) {
    const unsigned c = (unsigned)foff[i];
    foff[i] = (int)at;
    at += c;
  }
  __syncthreads();  // also: the block maxima's keys are dead, the candidates take their place
  unsigned* cand_key = keys;
  float* cval = reinterpret_cast<float*>(keys + kSparseCand);
#pragma unroll 1
  for (int f = tid; f < (int)nflag; f += kAttendThreads) {
    int idx = foff[f];
    const int pos0 = flag_id[f] * 16;
#pragma unroll 1
    for (int q = 0; q < 4; ++q) {
      const float4 v = stage[4 * f + (q ^ (f & 3))];
      const float vv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const unsigned key = order_key(vv[c]);
        if (key >= cut_key) {
          cand_key[idx] = key - cut_key;
          cval[idx] = vv[c];
          cpos[idx] = pos0 + q * 4 + c;
          ++idx;
        }
      }
    }
  }
  __syncthreads();

  // ---- the exact k-th largest among the candidates
  unsigned thr = 0, need_eq = 0;
  radix_kth_shared(cand_key, (int)ncand, 0u, key_max != cut_key ? 32 - __clz(key_max - cut_key) : 0, k, 4, sc, &thr,
                   &need_eq);

  // ---- compaction in token order: kept = key > thr, or key == thr among the first need_eq such candidates
  const int per3 = ((int)ncand + kAttendThreads - 1) / kAttendThreads;
  const int c_lo = min((int)ncand, tid * per3), c_hi = min((int)ncand, c_lo + per3);
  unsigned packed = 0;
#pragma unroll 1
  for (int i = c_lo; i < c_hi; ++i) {
    const unsigned key = cand_key[i];
    packed += key > thr ? 1u : (key == thr ? 1u << 16 : 0u);
  }
  unsigned tot_unused = 0;
  const unsigned before = block_scan(packed, &tot_unused, sc);
  unsigned gt_before = before & 0xffffu, eq_before = before >> 16;
#pragma unroll 1
  for (int i = c_lo; i < c_hi; ++i) {
    const unsigned key = cand_key[i];
    const bool g = key > thr, q = key == thr;
    if (g || (q && eq_before < need_eq)) {
      const unsigned pos = gt_before + min(eq_before, need_eq);
      if (pos < (unsigned)kMaxTopk) {  // always true for a consistent threshold; never write past the arrays
        out.pos[pos] = cpos[i];
        out.val[pos] = cval[i];
      }
    }
    gt_before += g;
    eq_before += q;
  }
  __syncthreads();
  return true;
}

// Per (sequence, query head): the topk best scores of the row, softmax over them, gather of their V rows.  Rows longer
// than one selection are taken in pieces whose winners are merged by one more selection.
__global__ void __launch_bounds__(kAttendThreads, 1)
topk_attend_kernel(const AttendParams p) {
  // stage[kMaxFlag][16] (the all-scores selection keeps mval[kMaxCand], mtok[kMaxCand] there), cand_key[kMaxCand],
  // cpos[kSparseCand], flag_id[kMaxFlag], foff[kMaxFlag], acc[warps][d_v]
  extern __shared__ __align__(16) float attend_dyn[];
  static_assert(kMaxFlag * 16 >= 2 * kMaxCand, "the merge arrays share the staging area");
  float4* stage = reinterpret_cast<float4*>(attend_dyn);
  float* mval = attend_dyn;
  int* mtok = reinterpret_cast<int*>(attend_dyn + kMaxCand);
  unsigned* cand_key = reinterpret_cast<unsigned*>(attend_dyn + kMaxFlag * 16);
  int* cpos = reinterpret_cast<int*>(attend_dyn + kMaxFlag * 16 + kMaxCand);
  int* flag_id = cpos + kSparseCand;
  int* foff = flag_id + kMaxFlag;
  float* acc_dyn = reinterpret_cast<float*>(foff + kMaxFlag);
  __shared__ SelectOut sel;
  __shared__ SelectScratch sc;
  int* sel_idx = sel.pos;
  float* sel_s = sel.val;
  __shared__ float red[kAttendWarps];

  // whatever follows in the stream may take the SMs this grid leaves free; it waits for this grid's end before it
  // touches memory
  ptx::grid_launch_dependents();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int b = blockIdx.x / p.n_q, h = blockIdx.x % p.n_q;
  const int hv = (int)(((long long)h * p.n_v) / p.n_q);  // Eq. (idx)
  ptx::grid_dependency_wait();
  const int len = min(max(p.seqlens[b], 0), p.max_seqlen);
  const long long orow = ((long long)b * p.n_q + h) * p.d_v;
  if (len == 0) {
    for (int ch = tid; ch < p.d_v; ch += kAttendThreads) {
      if (p.out_is_f32) reinterpret_cast<float*>(p.out)[orow + ch] = 0.f;
      else reinterpret_cast<__nv_bfloat16*>(p.out)[orow + ch] = __float2bfloat16_rn(0.f);
    }
    if (p.lse && tid == 0) p.lse[(long long)b * p.n_q + h] = -INFINITY;
    if (p.kept_ids)
      for (int i = tid; i < p.topk; i += kAttendThreads) p.kept_ids[(long long)blockIdx.x * p.topk + i] = -1;
    return;
  }
  const float* row = p.scores + (long long)blockIdx.x * p.lpad;
  int k = min(p.topk, len);
  // worth trying when the bound from the block maxima cuts deep (at least two blocks per kept score), or when the row
  // is short enough for all of it to fit the candidate buffer
  const bool sparse = !p.general_only && (32LL * k <= len || len <= kSparseCand) &&
                      block_select_sparse(row, p.bmax + (long long)blockIdx.x * (p.lpad / 16), len, k, sel, sc,
                                          cand_key, cpos, flag_id, foff, stage);
  if (sparse) {
    // sel holds the kept tokens
  } else if (len <= kPiece) {
    block_select(row, len, k, sel, sc, cand_key);
  } else {
    int ncand = 0;
    for (int base = 0; base < len; base += kPiece) {
      const int n_p = min(kPiece, len - base), k_p = min(p.topk, n_p);
      block_select(row + base, n_p, k_p, sel, sc, cand_key);
      for (int i = tid; i < k_p; i += kAttendThreads) {
        mval[ncand + i] = sel_s[i];
        mtok[ncand + i] = base + sel_idx[i];
      }
      ncand += k_p;
      __syncthreads();
    }
    k = min(p.topk, ncand);
    block_select(mval, ncand, k, sel, sc, cand_key);
    for (int i = tid; i < k; i += kAttendThreads) sel_idx[i] = mtok[sel_idx[i]];
    __syncthreads();
  }

  if (p.kept_ids)  // which tokens were kept (in no particular order), for callers that check or reuse the selection
    for (int i = tid; i < p.topk; i += kAttendThreads) p.kept_ids[(long long)blockIdx.x * p.topk + i] = i < k ? sel_idx[i] : -1;

  // ---- softmax over the kept scores (base-2 domain)
  float m = -INFINITY;
  for (int i = tid; i < k; i += kAttendThreads) m = fmaxf(m, sel_s[i]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if (lane == 0) red[warp] = m;
  __syncthreads();
  m = red[0];
#pragma unroll
  for (int ww = 1; ww < kAttendWarps; ++ww) m = fmaxf(m, red[ww]);
  __syncthreads();
  float l = 0.f;
  for (int i = tid; i < k; i += kAttendThreads) {
    const float e = exp2f(sel_s[i] - m);
    sel_s[i] = e;
    l += e;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
  if (lane == 0) red[warp] = l;
  __syncthreads();
  l = 0.f;
#pragma unroll
  for (int ww = 0; ww < kAttendWarps; ++ww) l += red[ww];

  // ---- where the kept V rows start (element offsets; -1: page out of range), one table look-up per row, all at once
  long long* row_off = reinterpret_cast<long long*>(cand_key);  // the candidate keys are dead by now
  for (int i = tid; i < k; i += kAttendThreads) {
    const int j = sel_idx[i];
    long long blk = b, slot = j;
    if (p.page_table) {
      blk = p.page_table[(long long)b * p.max_pages_per_seq + j / p.page_size];
      slot = j % p.page_size;
    }
    long long off = blk * p.v_sb + (long long)hv * p.v_sh + slot * p.v_st;
    if (blk < 0 || blk >= p.num_blocks) {
      report(p.dev_status, DIFFQKV_ERR_INDEX);
      off = -1;
    }
    row_off[i] = off;
  }
  __syncthreads();
  // ---- gather: half a warp per row, a lane per 8 channels (128 channels per sweep), eight rows in flight per lane
  constexpr int kInFlight = 8;
  const int half = lane >> 4, hl = lane & 15;
  for (int ch0 = 0; ch0 < p.d_v; ch0 += 128) {
    const int ch = ch0 + hl * 8;
    const bool in = ch < p.d_v;
    float a[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) a[e] = 0.f;
    for (int i0 = warp * 2 + half; i0 < k; i0 += 2 * kAttendWarps * kInFlight) {
      uint4 raw[kInFlight];
      float wgt[kInFlight];
#pragma unroll
      for (int f = 0; f < kInFlight; ++f) {
        const int i = i0 + f * 2 * kAttendWarps;
        raw[f] = make_uint4(0u, 0u, 0u, 0u);
        wgt[f] = 0.f;
        if (i < k && in) {
          const long long off = row_off[i];
          if (off >= 0) {
            raw[f] = *reinterpret_cast<const uint4*>(p.v + off + ch);
            wgt[f] = sel_s[i];
          }
        }
      }
#pragma unroll
      for (int f = 0; f < kInFlight; ++f) {
        const uint32_t wd[4] = {raw[f].x, raw[f].y, raw[f].z, raw[f].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          a[2 * e] = fmaf(wgt[f], __uint_as_float(wd[e] << 16), a[2 * e]);
          a[2 * e + 1] = fmaf(wgt[f], __uint_as_float(wd[e] & 0xffff0000u), a[2 * e + 1]);
        }
      }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) a[e] += __shfl_xor_sync(0xffffffffu, a[e], 16);
    if (in && half == 0) {
      float* dst = acc_dyn + warp * p.d_v + ch;
#pragma unroll
      for (int e = 0; e < 8; ++e) dst[e] = a[e];
    }
  }
  __syncthreads();
  const float inv = 1.f / l;
  for (int ch = tid; ch < p.d_v; ch += kAttendThreads) {
    float o = 0.f;
#pragma unroll
    for (int ww = 0; ww < kAttendWarps; ++ww) o += acc_dyn[ww * p.d_v + ch];
    o *= inv;
    if (p.out_is_f32) reinterpret_cast<float*>(p.out)[orow + ch] = o;
    else reinterpret_cast<__nv_bfloat16*>(p.out)[orow + ch] = __float2bfloat16_rn(o);
  }
  if (p.lse && tid == 0) p.lse[(long long)b * p.n_q + h] = (m + log2f(l)) * kLn2;
}

int sm_count_topk() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
  return sms;
}

}  // namespace

static int topk_pieces(int max_seqlen) { return ((max_seqlen > 0 ? max_seqlen : 1) + kPiece - 1) / kPiece; }

bool topk_decode_supported(const diffqkv_shape& s, const diffqkv_cache& c, int topk, int* box_tok) {
  if (s.dtype != DIFFQKV_BF16 || (s.d_qk != 64 && s.d_qk != 128)) return false;
  if (s.d_v % 8 != 0 || s.d_v > 512 || topk < 1 || topk > kMaxTopk) return false;
  if (s.batch < 1 || s.batch > kMaxBatchScores || s.n_q / s.n_k > 8 * kMaxGroups) return false;
  if (c.v_stride_tok % 8 != 0 || c.v_stride_head % 8 != 0 || c.v_stride_blk % 8 != 0) return false;  // 16-byte loads
  if ((reinterpret_cast<uintptr_t>(c.v_cache) & 15u) != 0) return false;
  if ((long long)topk_pieces(c.max_seqlen) * topk > kMaxCand) return false;  // the pieces' winners are merged in one go
  int bt = kST;
  if (c.page_table) {
    if (c.page_size % 16 != 0) return false;
    if (c.page_size < kST) { if (kST % c.page_size != 0) return false; bt = c.page_size; }
    else if (c.page_size % kST != 0) return false;
  }
  *box_tok = bt;
  return true;
}

static size_t up256(size_t x) { return (x + 255) / 256 * 256; }

size_t topk_decode_workspace_bytes(const diffqkv_shape& s, int max_seqlen, int /*topk*/) {
  const size_t lpad = ((size_t)(max_seqlen > 0 ? max_seqlen : 1) + kST - 1) / kST * kST;
  const size_t rows = (size_t)s.batch * s.n_q;
  return up256(rows * lpad * sizeof(float)) + up256(rows * (lpad / 16) * sizeof(float));
}

static std::atomic<int> g_topk_general_only{0};  // test hook
void set_topk_general_only(int on) { g_topk_general_only = on != 0; }

cudaError_t launch_decode_topk(const void* q, const diffqkv_cache& c, const diffqkv_shape& s, int topk, int box_tok,
                               void* workspace, void* out, float* lse, int* dev_status, cudaStream_t stream,
                               int* kept_ids) {
  const int sms = sm_count_topk();
  if (sms <= 0) return cudaErrorUnknown;
  int dev = 0, max_smem = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  const long long tok_extent = c.page_table ? c.page_size : c.max_seqlen;
  CUtensorMap mk;
  {
    const cuuint64_t dims[5] = {64, (cuuint64_t)tok_extent, (cuuint64_t)(s.d_qk / 64), (cuuint64_t)s.n_k,
                                (cuuint64_t)c.num_blocks};
    const cuuint64_t strides[4] = {(cuuint64_t)c.k_stride_tok * 2, 128, (cuuint64_t)c.k_stride_head * 2,
                                   (cuuint64_t)c.k_stride_blk * 2};
    const cuuint32_t box[5] = {64, (cuuint32_t)box_tok, (cuuint32_t)(s.d_qk / 64), 1, 1};
    if (!make_tmap_bf16_sw128(&mk, c.k_cache, 5, dims, strides, box)) return cudaErrorNotSupported;
  }
  ScoreParams sp;
  sp.q = reinterpret_cast<const __nv_bfloat16*>(q);
  sp.seqlens = c.seqlens; sp.page_table = c.page_table;
  sp.page_size = c.page_size; sp.max_pages_per_seq = c.max_pages_per_seq;
  sp.num_blocks = c.num_blocks; sp.max_seqlen = c.max_seqlen;
  sp.batch = s.batch; sp.n_q = s.n_q; sp.n_k = s.n_k; sp.g_k = s.n_q / s.n_k;
  sp.groups = (sp.g_k + 7) / 8;
  const int ng = sp.groups;
  sp.box_tok = box_tok;
  sp.lpad = ((long long)(c.max_seqlen > 0 ? c.max_seqlen : 1) + kST - 1) / kST * kST;
  sp.scale_log2 = s.scale * kLog2e;
  sp.scores = reinterpret_cast<float*>(workspace);
  sp.bmax = reinterpret_cast<float*>(reinterpret_cast<char*>(workspace) +
                                     up256((size_t)s.batch * s.n_q * (size_t)sp.lpad * sizeof(float)));
  sp.dev_status = dev_status;
  const int k_tile = kST * s.d_qk * 2;
  const int fixed = 1024 + 2 * 16 * 8 + (s.batch + 1) * 4 + 64;
  int stages = (max_smem - fixed) / k_tile;
  if (stages > 6) stages = 6;
  if (stages < 2) return cudaErrorNotSupported;
  sp.stages = stages;
  const int smem = fixed + stages * k_tile;
  const long long tiles_max = (long long)s.batch * s.n_k * ((c.max_seqlen + kST - 1) / kST);
  long long grid = sms;
  if (grid > tiles_max) grid = tiles_max;
  if (grid < 1) grid = 1;

  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)score_threads(ng));
  cfg.dynamicSmemBytes = (size_t)smem;
  cudaError_t err = cudaErrorNotSupported;
  auto launch = [&](auto kernel) {
    err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (err == cudaSuccess) err = cudaLaunchKernelEx(&cfg, kernel, mk, sp);
  };
  if (s.d_qk == 128) {
    if (ng == 1) launch(decode_scores_kernel<128, 1>);
    else if (ng == 2) launch(decode_scores_kernel<128, 2>);
    else if (ng == 3) launch(decode_scores_kernel<128, 3>);
    else if (ng == 4) launch(decode_scores_kernel<128, 4>);
  } else {
    if (ng == 1) launch(decode_scores_kernel<64, 1>);
    else if (ng == 2) launch(decode_scores_kernel<64, 2>);
    else if (ng == 3) launch(decode_scores_kernel<64, 3>);
    else if (ng == 4) launch(decode_scores_kernel<64, 4>);
  }
  if (err != cudaSuccess) return err;
  count_launch();

  const size_t rows = (size_t)s.batch * s.n_q;
  AttendParams ap;
  ap.scores = sp.scores; ap.bmax = sp.bmax; ap.lpad = sp.lpad;
  ap.general_only = g_topk_general_only;
  ap.v = reinterpret_cast<const __nv_bfloat16*>(c.v_cache);
  ap.v_sb = c.v_stride_blk; ap.v_sh = c.v_stride_head; ap.v_st = c.v_stride_tok;
  ap.seqlens = c.seqlens; ap.page_table = c.page_table;
  ap.page_size = c.page_size; ap.max_pages_per_seq = c.max_pages_per_seq;
  ap.num_blocks = c.num_blocks; ap.max_seqlen = c.max_seqlen;
  ap.batch = s.batch; ap.n_q = s.n_q; ap.n_v = s.n_v; ap.d_v = s.d_v; ap.topk = topk;
  ap.out = out; ap.lse = lse; ap.out_is_f32 = s.out_dtype == DIFFQKV_F32;
  ap.dev_status = dev_status;
  ap.kept_ids = kept_ids;
  cfg.gridDim = dim3((unsigned)rows);
  cfg.blockDim = dim3(kAttendThreads);
  cfg.dynamicSmemBytes =
      (size_t)(kMaxFlag * 16 + kMaxCand + kSparseCand + 2 * kMaxFlag + kAttendWarps * s.d_v) * sizeof(float);
  err = cudaFuncSetAttribute(topk_attend_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cfg.dynamicSmemBytes);
  if (err != cudaSuccess) return err;
  err = cudaLaunchKernelEx(&cfg, topk_attend_kernel, ap);
  if (err != cudaSuccess) return err;
  count_launch();
  return cudaGetLastError();
}

}  // namespace diffqkv
