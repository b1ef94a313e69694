// Top-k selection and gate of one token (Eq. 3-4), shared by the router kernels so that
// equal logits give equal decisions whichever kernel produced them.
#pragma once

#include "moga_internal.cuh"

namespace moga {

// row: the token's M logits (bias already added).  Picks the k largest (strict >, so ties
// keep the lower group index), in descending order, and writes their gates:
// softmax over all M logits (MOGA_GATE_SOFTMAX_ALL) or over the k picks, max-subtracted.
__device__ __forceinline__ void select_and_gate(const float* row, int M, int k, int gate_mode,
                                                int32_t* __restrict__ gid_out,
                                                float* __restrict__ gate_out) {
  unsigned long long taken = 0ull;
  float top = 0.f, zsel = 0.f;
  float val[kMaxK];
  int sel[kMaxK];
#pragma unroll
  for (int j = 0; j < kMaxK; ++j) {
    if (j < k) {
      int best = -1;
      float bv = 0.f;
      for (int i = 0; i < M; ++i) {
        if ((taken >> i) & 1ull) continue;
        float v = row[i];
        if (best < 0 || v > bv) { best = i; bv = v; }
      }
      taken |= 1ull << best;
      sel[j] = best;
      val[j] = bv;
      if (j == 0) top = bv;
      zsel += expf(bv - top);
    }
  }
  float Z = zsel;
  if (gate_mode == MOGA_GATE_SOFTMAX_ALL) {
    Z = 0.f;
    for (int i = 0; i < M; ++i) Z += expf(row[i] - top);
  }
#pragma unroll
  for (int j = 0; j < kMaxK; ++j) {
    if (j < k) {
      gid_out[j] = sel[j];
      gate_out[j] = expf(val[j] - top) / Z;
    }
  }
}

}  // namespace moga
