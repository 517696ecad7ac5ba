// Radix select on non-negative floats (their bit patterns order as unsigned integers): the digit decision
// shared by the top-k kernel and the percentile kernel.
#pragma once

#include "common.cuh"

namespace catekv {

// The digit histograms are kept in kHistCopies interleaved copies (bin d of copy c at word d * kHistCopies + c), a lane
// adds to copy lane % kHistCopies: in the first passes most entries share their top digits, and atomics on one
// address serialise.  A CTA folds its copies into a plain 256-bin histogram before anybody reads it.
constexpr int kHistCopies = 8;
__device__ __forceinline__ void radix_hist_zero(unsigned int* hcopies) {
  for (int i = threadIdx.x; i < 256 * kHistCopies; i += blockDim.x) hcopies[i] = 0;
}
__device__ __forceinline__ void radix_hist_add(unsigned int* hcopies, unsigned int digit, unsigned int count) {
  atomicAdd(&hcopies[digit * kHistCopies + (threadIdx.x & (kHistCopies - 1))], count);
}
// threads 0..255: bin tid of the folded histogram
__device__ __forceinline__ void radix_hist_fold(const unsigned int* hcopies, unsigned int* hist) {
  if (threadIdx.x < 256) {
    unsigned int t = 0;
#pragma unroll
    for (int c = 0; c < kHistCopies; ++c) t += hcopies[threadIdx.x * kHistCopies + c];
    hist[threadIdx.x] = t;
  }
}

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

}  // namespace catekv
