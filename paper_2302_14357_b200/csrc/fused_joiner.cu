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
//                 reduction, written to device memory ([rows / S, V]: S times smaller than the logits);
//                 the rows' N best tokens are then picked by the selection kernel of scan_select.cu
// Row layout: a tile holds 4 * (32 / S) hypotheses; hypothesis j of warp quarter q sits in TMEM lanes
// 32 q + j S .. + S - 1 (one lane per frame); lanes past (32 / S) S are idle.
//
// No TMA multicast is used: every CTA fetches the A tile it shares with its cluster mates itself.
// Waits on mbarriers are bounded; the two cluster-wide hardware barriers (start, end) are reached by
// every thread of every CTA on every path.
#include "bf16_path.cuh"
#include "sm100.cuh"

namespace tw {

namespace {

using namespace sm100;

constexpr int BM = 128, BK = 64, NC = 256;   // rows per tile, K per stage, columns per CTA
constexpr int kStages = 3;
constexpr int kMaxCL = 16;
constexpr int kColGroups = 4;                // epilogue warps per TMEM lane quarter, 64 columns each
constexpr int kEpiWarps = 4 * kColGroups, kEpiThreads = 32 * kEpiWarps;
constexpr int kThreadsFused = 64 + kEpiThreads;
constexpr uint32_t kABytes = BM * BK * 2, kBBytes = NC * BK * 2;
// longer segments (S = 5, 8, 10): the sum over a hypothesis's frames goes through a per-warp staging tile in shared
// memory, 16 columns at a time (row = TMEM lane, odd pitch: conflict-free row-per-lane writes)
constexpr int kStagePitch = 17;

struct FusedSmem {
  // offsets from the 1024-aligned base
  static constexpr size_t kA = 0;
  static constexpr size_t kB = kA + (size_t)kStages * kABytes;
  static constexpr size_t kXch = kB + (size_t)kStages * kBBytes;                  // float2 [2][kMaxCL][BM]
  static constexpr size_t kXchBlank = kXch + (size_t)2 * kMaxCL * BM * 8;         // float  [2][BM]
  static constexpr size_t kPart = kXchBlank + (size_t)2 * BM * 4;                 // float2 [kColGroups][BM]
  static constexpr size_t kZb = kPart + (size_t)kColGroups * BM * 8;                       // float  [BM]
  static constexpr size_t kBias = kZb + (size_t)BM * 4;                           // float  [NC]
  static constexpr size_t kBars = kBias + (size_t)NC * 4;                         // uint64 [16]
  static constexpr size_t kStage = kBars + 16 * 8 + 16;                           // float  [kEpiWarps][32][kStagePitch]
  static constexpr size_t kTotal = kStage + (size_t)kEpiWarps * 32 * kStagePitch * 4;
};
constexpr size_t kSmemFused = FusedSmem::kTotal + 1024;

constexpr float kLog2e = 1.4426950408889634f, kLn2 = 0.6931471805599453f;
__device__ __forceinline__ float ex2f(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ float lg2f(float x) { float y; asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }

// log2(2^a + 2^b), branch-free; log 0 = -inf on either side or both
__device__ __forceinline__ float logaddexp2_fast(float a, float b) {
  const float mx = fmaxf(a, b), mn = fminf(a, b);
  const float d = (mn == -INFINITY) ? -INFINITY : mn - mx;    // (-inf) - (-inf) would be NaN
  return mx + lg2f(1.f + ex2f(d));
}

// sum over the S lanes [lane, lane + S) of x, valid in lanes whose window stays inside the warp.
// ST > 0: segment size known at compile time (plain unrolled shuffles); ST == 0: any S <= 32.
template <int ST>
__device__ __forceinline__ float window_sum(float x, int S) {
  if (ST > 0 && ST <= 4) {
    float total = x;
#pragma unroll
    for (int d = 1; d < ST; ++d) total += __shfl_down_sync(0xffffffffu, x, d);
    return total;
  }
  // doubling: windows of 1, 2, 4, ... lanes; the set bits of S pick the pieces (unrolled when S is known)
  const int SS = ST > 0 ? ST : S;
  float total = 0.f, cur = x;
  int off = 0;
#pragma unroll
  for (int size = 1; size <= 32; size <<= 1) {
    if (size > SS) break;
    if (SS & size) { total += (off == 0) ? cur : __shfl_down_sync(0xffffffffu, cur, off); off += size; }   // the first piece is the lane's own
    if (2 * size <= SS) cur += __shfl_down_sync(0xffffffffu, cur, size);
  }
  return total;
}

#include "fused_joiner_kernel.inc"

}  // namespace

#include "fused_joiner_host.inc"

}  // namespace tw
