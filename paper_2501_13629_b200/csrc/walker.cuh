// Position in a flat (sequence, unit, tile) work list, shared by the persistent kernels that divide such a list over
// their blocks (the TMA decode kernel: units of query heads, 64-token tiles; the score kernel of selective V
// fetching: K heads, 128-token tiles).  `prefix[b]` is the number of tiles of all sequences before b, so sequence b
// owns flat entries [n_units * prefix[b], n_units * prefix[b + 1]), unit by unit, tile by tile.
#pragma once

namespace diffqkv {

struct FlatWalker {
  long long g;  // flat index
  int b, u, t, nt;
  __device__ void seek(long long g0, const int* prefix, int batch, int n_units) {
    g = g0;
    int lo = 0, hi = batch;  // smallest b' with n_units * prefix[b'] > g; answer b = b' - 1
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if ((long long)n_units * prefix[mid] > g0) hi = mid; else lo = mid + 1;
    }
    b = lo - 1;
    nt = prefix[b + 1] - prefix[b];
    const long long rem = g0 - (long long)n_units * prefix[b];
    u = (int)(rem / nt);
    t = (int)(rem % nt);
  }
  // the next sequence that has tiles (b == batch when there is none; nt is then 1 so that nothing divides by zero)
  __device__ void next_sequence(const int* prefix, int batch) {
    do {
      ++b;
      nt = b < batch ? prefix[b + 1] - prefix[b] : 1;
    } while (b < batch && nt == 0);
  }
  __device__ void advance(const int* prefix, int batch, int n_units) {
    ++g;
    if (++t == nt) {
      t = 0;
      if (++u == n_units) {
        u = 0;
        next_sequence(prefix, batch);
      }
    }
  }
};

}  // namespace diffqkv
