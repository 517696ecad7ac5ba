// Block-wide radix select on non-negative floats (their bit patterns order as unsigned integers).
#pragma once

#include "common.cuh"

namespace catekv {

// Finds the `need`-th largest of the n values load(0..n-1) (1 <= need <= n), with all threads of
// the block taking part.  Returns its bit pattern in `thr` and, in `need_eq`, how many of the
// entries equal to it belong to the top `need` (the rest of the top are strictly greater).
// hist: 256 shared counters; s_pair: 2 shared words.
template <class Load>
__device__ __forceinline__ void block_radix_select(Load load, int n, unsigned int need, unsigned int* hist,
                                                   unsigned int* s_pair, unsigned int& thr, unsigned int& need_eq) {
  const int tid = threadIdx.x, nthr = blockDim.x;
  unsigned int prefix = 0;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    const unsigned int pmask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    for (int c = tid; c < n; c += nthr) {
      const unsigned int v = load(c);
      if ((v & pmask) == prefix) atomicAdd(&hist[(v >> shift) & 0xffu], 1u);
    }
    __syncthreads();
    if (tid == 0) {
      unsigned int cum = 0;
      int dsel = 0;
      for (int dgt = 255; dgt >= 0; --dgt) {
        if (cum + hist[dgt] >= need) { dsel = dgt; break; }
        cum += hist[dgt];
      }
      s_pair[0] = prefix | ((unsigned int)dsel << shift);
      s_pair[1] = need - cum;
    }
    __syncthreads();
    prefix = s_pair[0];
    need = s_pair[1];
  }
  thr = prefix;
  need_eq = need;
}

}  // namespace catekv
