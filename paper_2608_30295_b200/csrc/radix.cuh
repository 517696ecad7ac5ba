// Block-wide radix select on non-negative floats (their bit patterns order as unsigned integers).
#pragma once

#include "common.cuh"

namespace catekv {

// One warp picks the radix digit that holds the `need`-th largest entry from a 256-bin histogram `h` (bins of
// larger digits first): lane L owns the 8 bins 255 - 8L .. 248 - 8L, a shuffle scan gives the count in the bins
// above a lane's, and the lane whose bins reach `need` writes the extended prefix and what is still needed
// inside the chosen bin to s_pair.  All 32 lanes must call it.
__device__ __forceinline__ void radix_pick_digit(const unsigned int* h, unsigned int need, unsigned int prefix, int shift,
                                                 unsigned int* s_pair) {
  const int lane = threadIdx.x & 31;
  unsigned int c[8], sum = 0;
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    c[e] = h[255 - (lane * 8 + e)];
    sum += c[e];
  }
  unsigned int inc = sum;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned int y = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += y;
  }
  const unsigned int before = inc - sum;
  if (before < need && need <= inc) {
    unsigned int cum = before;
    int dsel = 255 - lane * 8;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      if (cum + c[e] >= need) {
        dsel = 255 - (lane * 8 + e);
        break;
      }
      cum += c[e];
    }
    s_pair[0] = prefix | ((unsigned int)dsel << shift);
    s_pair[1] = need - cum;
  } else if (lane == 31 && inc < need) {  // fewer entries than asked for: everything is taken
    s_pair[0] = prefix;
    s_pair[1] = need - (inc - c[7]);
  }
}

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
    for (int c0 = 0; c0 < n; c0 += 4 * nthr) {  // whole warps stay in the loop: the vote below needs them
      // four independent loads in flight per thread
      unsigned int v[4];
      bool in[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int c = c0 + e * nthr + tid;
        v[e] = c < n ? load(c) : 0u;
        in[e] = c < n;
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const bool hit = in[e] && (v[e] & pmask) == prefix;
        // a warp whose lanes all fall in one bin (the common case in the top digit: scores share their exponent)
        // adds once; otherwise every hit adds for itself, the digits being spread over the bins
        const unsigned int dgt = hit ? ((v[e] >> shift) & 0xffu) : 0x100u;
        int same;
        __match_all_sync(0xffffffffu, dgt, &same);
        if (same) {
          if (hit && (threadIdx.x & 31) == 0) atomicAdd(&hist[dgt], 32u);
        } else if (hit) {
          atomicAdd(&hist[dgt], 1u);
        }
      }
    }
    __syncthreads();
    if (tid < 32) radix_pick_digit(hist, need, prefix, shift, s_pair);
    __syncthreads();
    prefix = s_pair[0];
    need = s_pair[1];
  }
  thr = prefix;
  need_eq = need;
}

}  // namespace catekv
