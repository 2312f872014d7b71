// Small sorted candidate lists for ChooseNBestExpansions: order is (score descending, token ascending).
#pragma once
#include "tw_internal.cuh"

namespace tw {

__device__ __forceinline__ bool cand_better(float v, int k, float v2, int k2) {
  return v > v2 || (v == v2 && k < k2);
}

// Per-thread list of the best kMaxBeam (value, token) pairs seen, kept sorted in registers.
struct TopList {
  float v[kMaxBeam];
  int k[kMaxBeam];
  __device__ __forceinline__ void init() {
#pragma unroll
    for (int j = 0; j < kMaxBeam; ++j) { v[j] = -INFINITY; k[j] = 0x7fffffff; }
  }
  // value of the n-th entry (1-based n <= kMaxBeam)
  __device__ __forceinline__ float nth(int n) const {
    float r = -INFINITY;
#pragma unroll
    for (int j = 0; j < kMaxBeam; ++j) r = (j < n) ? v[j] : r;   // a select chain keeps the list in registers
    return r;
  }
  __device__ __forceinline__ void insert(float cv, int ck) {
#pragma unroll
    for (int j = 0; j < kMaxBeam; ++j) {
      if (cand_better(cv, ck, v[j], k[j])) {
        const float tv = v[j]; const int tk = k[j];
        v[j] = cv; k[j] = ck; cv = tv; ck = tk;
      }
    }
  }
  __device__ __forceinline__ void pop() {
#pragma unroll
    for (int i = 0; i < kMaxBeam - 1; ++i) { v[i] = v[i + 1]; k[i] = k[i + 1]; }
    v[kMaxBeam - 1] = -INFINITY; k[kMaxBeam - 1] = 0x7fffffff;
  }
};

// Merges the 32 lists of a warp: the best n pairs, best first, are written by lane 0 to out_v / out_k.
// Returns how many were written (pairs with value -inf are not candidates).
__device__ __forceinline__ int warp_merge_lists(TopList& l, int n, float* out_v, int* out_k) {
  const int lane = threadIdx.x & 31;
  int cnt = 0;
  for (int j = 0; j < n; ++j) {
    float bv = l.v[0]; int bk = l.k[0]; int bl = lane;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int ok = __shfl_xor_sync(0xffffffffu, bk, o);
      const int ol = __shfl_xor_sync(0xffffffffu, bl, o);
      if (cand_better(ov, ok, bv, bk)) { bv = ov; bk = ok; bl = ol; }
    }
    if (bv == -INFINITY) break;
    if (lane == 0) { out_v[j] = bv; out_k[j] = bk; }
    if (lane == bl) l.pop();
    ++cnt;
  }
  return cnt;
}

}  // namespace tw
