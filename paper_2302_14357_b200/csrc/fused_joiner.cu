// Fused joiner + softmax + Eq. 3-7 + candidate selection for TW_MODE_BF16.  The [rows, V] logits live
// only in tensor memory: a thread-block cluster of CL = V / 256 CTAs owns a tile of 128 rows, CTA c
// holding columns [256 c, 256 c + 256) of it in TMEM (two accumulator buffers, so the contraction of
// the next row tile overlaps this tile's epilogue).
//
// Per row tile, in every CTA of the cluster:
//   contraction   TMA ring -> tcgen05.mma (as in gemm_bf16.cu), z = tanh(E + Pp) W_out^T
//   epilogue A    per row: running max / sum-exp over the CTA's 256 columns, the blank logit
//   exchange      (max, sum-exp[, blank logit]) of every row to every CTA of the cluster through
//                 distributed shared memory, completion by remote mbarrier arrivals
//   scan          lse, blank log-probability, the occupancy recursion la over the S frames of a
//                 hypothesis (frames of a hypothesis are adjacent lanes of one warp): Eq. 3-5, 7
//   epilogue B    delta_nb(k) = sum_t exp(la[t] - lse[t] + z[t, k]) (Eq. 6) by a segmented warp
//                 reduction, and the hypothesis' N best tokens among this CTA's columns
// Row layout: a tile holds 4 * (32 / S) hypotheses; hypothesis j of warp quarter q sits in TMEM lanes
// 32 q + j S .. + S - 1 (one lane per frame); lanes past (32 / S) S are idle.
//
// No TMA multicast is used: every CTA fetches the A tile it shares with its cluster mates itself.
// Waits on mbarriers are bounded; the two cluster-wide hardware barriers (start, end) are reached by
// every thread of every CTA on every path.
#include "bf16_path.cuh"
#include "sm100.cuh"
#include "topn.cuh"

namespace tw {

namespace {

using namespace sm100;

constexpr int BM = 128, BK = 64, NC = 256;   // rows per tile, K per stage, columns per CTA
constexpr int kStages = 3;
constexpr int kMaxCL = 16;
constexpr int kEpiWarps = 8, kEpiThreads = 32 * kEpiWarps;
constexpr int kThreadsFused = 64 + kEpiThreads;
constexpr uint32_t kABytes = BM * BK * 2, kBBytes = NC * BK * 2;

struct FusedSmem {
  // offsets from the 1024-aligned base
  static constexpr size_t kA = 0;
  static constexpr size_t kB = kA + (size_t)kStages * kABytes;
  static constexpr size_t kXch = kB + (size_t)kStages * kBBytes;                  // float2 [2][kMaxCL][BM]
  static constexpr size_t kXchBlank = kXch + (size_t)2 * kMaxCL * BM * 8;         // float  [2][BM]
  static constexpr size_t kPart = kXchBlank + (size_t)2 * BM * 4;                 // float2 [2][BM]
  static constexpr size_t kZb = kPart + (size_t)2 * BM * 8;                       // float  [BM]
  static constexpr size_t kBias = kZb + (size_t)BM * 4;                           // float  [NC]
  static constexpr size_t kBars = kBias + (size_t)NC * 4;                         // uint64 [16]
  static constexpr size_t kTotal = kBars + 16 * 8 + 16;
};
constexpr size_t kSmemFused = FusedSmem::kTotal + 1024;

// sum over the S lanes [lane, lane + S) of x, valid in lanes whose window stays inside the warp
__device__ __forceinline__ float window_sum(float x, int S) {
  float total = 0.f, cur = x;
  int off = 0;
  for (int size = 1; size <= S; size <<= 1) {
    if (S & size) { total += __shfl_down_sync(0xffffffffu, cur, off); off += size; }
    cur += __shfl_down_sync(0xffffffffu, cur, size);
  }
  return total;
}

#include "fused_joiner_kernel.inc"

// ChooseNBestExpansions, stage 1b: merge the 2 CL sorted per-CTA lists of each hypothesis row
__global__ void merge_lists_kernel(FusedJoinerParams p, float* cand_v, int* cand_k, int* cand_n) {
  const int R = p.R_dev ? *p.R_dev : p.R_max;
  const int r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (r >= R) return;
  const int nlists = 2 * p.CL;
  const long long list = (long long)r * (2 * kMaxCL) + lane;
  const int mine = lane < nlists ? p.c2n[list] : 0;
  int pos = 0, cnt = 0;
  for (int j = 0; j < p.N; ++j) {
    float bv = (pos < mine) ? p.c2v[list * kMaxBeam + pos] : -INFINITY;
    int bk = (pos < mine) ? p.c2k[list * kMaxBeam + pos] : 0x7fffffff;
    int bl = lane;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int ok = __shfl_xor_sync(0xffffffffu, bk, o);
      const int ol = __shfl_xor_sync(0xffffffffu, bl, o);
      if (cand_better(ov, ok, bv, bk)) { bv = ov; bk = ok; bl = ol; }
    }
    if (bv == -INFINITY) break;
    if (lane == 0) { cand_v[(long long)r * kMaxBeam + j] = bv; cand_k[(long long)r * kMaxBeam + j] = bk; }
    if (lane == bl) ++pos;
    ++cnt;
  }
  if (lane == 0) cand_n[r] = cnt;
}

}  // namespace

#include "fused_joiner_host.inc"

}  // namespace tw
