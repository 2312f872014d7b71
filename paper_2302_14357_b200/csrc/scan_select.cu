// Softmax + Eq. 3-7 + first stage of ChooseNBestExpansions in one kernel, one CTA per hypothesis row.
// The row's S' x V raw joiner logits are read from global memory ONCE into shared memory; everything
// else (per-frame log-sum-exp, the blank recursion, delta_nb, the row's N best tokens) runs from there.
//   lse[t]   = log sum_k exp z[t, k]                          (softmax normaliser, Sec. 3.1)
//   lb[t]    = z[t, blank] - lse[t]
//   la[1]    = ld_old[1];  la[t+1] = logaddexp(la[t] + lb[t], ld_old[t+1])      (Eq. 3-5)
//   dnb[k]   = log sum_t exp(la[t] - lse[t] + z[t, k]),  k != blank             (Eq. 6)
//   dphi     = la[S'] + lb[S']                                                  (Eq. 7)
#include "topn.cuh"
#include "tw_internal.cuh"

namespace tw {

namespace {

constexpr int kT = 256;
constexpr int kGroups = 16;        // 16 groups of 16 threads: their maxima bound the N-th best value
constexpr int kSurvCap = 192;

__device__ __forceinline__ float wmax(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float wsum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__global__ void __launch_bounds__(kT) scan_select_kernel(ScanSelectArgs a) {
  extern __shared__ __align__(16) float zs[];          // [S][V] logits of this row; row 0 later holds dnb
  __shared__ float s_lse[kMaxSeg], s_w[kMaxSeg];
  __shared__ float s_gmax[kGroups];
  __shared__ float s_bound;
  __shared__ int s_nsurv;
  __shared__ float s_sv[kSurvCap];
  __shared__ int s_sk[kSurvCap];
  __shared__ float s_wv[kT / 32][kMaxBeam];
  __shared__ int s_wk[kT / 32][kMaxBeam];
  __shared__ int s_wn[kT / 32];

  const int R = a.R_dev ? *a.R_dev : a.R_max;
  const int r = blockIdx.x;
  if (r >= R) return;
  const int S = a.S, V = a.V, blank = a.blank;
  const int sl = a.row_slen ? a.row_slen[r] : S;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* z = a.z + (long long)r * S * V;

  // ---- the one pass over global memory
  if ((V & 3) == 0) {
    const int n4 = sl * V / 4;
    const float4* src = reinterpret_cast<const float4*>(z);
    float4* dst = reinterpret_cast<float4*>(zs);
    for (int i = tid; i < n4; i += kT) dst[i] = src[i];
  } else {
    for (int i = tid; i < sl * V; i += kT) zs[i] = z[i];
  }
  if (tid == 0) s_nsurv = 0;
  __syncthreads();

  // ---- per-frame log-sum-exp: one warp per frame
  for (int t = warp; t < sl; t += kT / 32) {
    const float* row = zs + t * V;
    float mx = -INFINITY;
    for (int k = lane; k < V; k += 32) mx = fmaxf(mx, row[k]);
    mx = wmax(mx);
    float s = 0.f;
    for (int k = lane; k < V; k += 32) s += expf(row[k] - mx);
    s = wsum(s);
    if (lane == 0) {
      const float lse = mx + logf(s);
      s_lse[t] = lse;
      if (a.lse_out) a.lse_out[(long long)r * S + t] = lse;
    }
  }
  __syncthreads();

  // ---- the blank recursion, carried in float64 (S' steps, values grow to hundreds of nats)
  if (tid == 0) {
    double acc = (double)a.ld_old[(long long)r * S];
    double phi = -INFINITY;
    for (int t = 0; t < sl; ++t) {
      s_w[t] = (float)acc - s_lse[t];
      if (a.la) a.la[(long long)r * S + t] = (float)acc;
      if (a.la_d) a.la_d[(long long)r * S + t] = acc;
      const double nxt = acc + ((double)zs[t * V + blank] - (double)s_lse[t]);
      if (t + 1 < sl) acc = logaddexp_d(nxt, (double)a.ld_old[(long long)r * S + t + 1]);
      else phi = nxt;
    }
    for (int t = (sl > 0 ? sl : 0); t < S; ++t) {
      if (a.la) a.la[(long long)r * S + t] = -INFINITY;
      if (a.la_d) a.la_d[(long long)r * S + t] = -INFINITY;
      if (a.lse_out) a.lse_out[(long long)r * S + t] = 0.f;
    }
    if (a.ldphi) a.ldphi[r] = (float)phi;
    if (a.ldphi_d) a.ldphi_d[r] = phi;
  }
  __syncthreads();

  // ---- delta_nb for every token; kept in shared memory (frame 0's logits are no longer needed)
  float tmax = -INFINITY;
  for (int k = tid; k < V; k += kT) {
    float out = -INFINITY;
    if (k != blank) {
      float mx = -INFINITY;
      for (int t = 0; t < sl; ++t) mx = fmaxf(mx, s_w[t] + zs[t * V + k]);
      if (mx > -INFINITY) {
        float s = 0.f;
        for (int t = 0; t < sl; ++t) s += expf(s_w[t] + zs[t * V + k] - mx);
        out = mx + logf(s);
      }
    }
    if (sl > 0) zs[k] = out;                 // only this thread ever touches column k
    if (a.ldnb) a.ldnb[(long long)r * V + k] = out;
    tmax = fmaxf(tmax, out);
  }
  if (a.cand.n == nullptr) return;
  const int N = a.cand.N;

  // ---- a lower bound of the row's N-th best value: the N-th largest of 16 group maxima (each is a
  // distinct element of the row), so everything at or above it is a small superset of the answer
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
  if ((tid & 15) == 0) s_gmax[tid >> 4] = tmax;
  __syncthreads();
  if (warp == 0) {
    const float mine = lane < kGroups ? s_gmax[lane] : -INFINITY;
    int rank = 0;
    for (int j = 0; j < kGroups; ++j) {
      const float o = __shfl_sync(0xffffffffu, mine, j);
      rank += (o > mine) || (o == mine && j < lane);
    }
    if (lane < kGroups && rank == min(N, kGroups) - 1) s_bound = (N <= kGroups) ? mine : -INFINITY;
  }
  __syncthreads();
  const float bound = s_bound;
  if (sl > 0) {
    for (int k = tid; k < V; k += kT) {
      const float v = zs[k];
      if (v >= bound && v > -INFINITY) {
        const int i = atomicAdd(&s_nsurv, 1);
        if (i < kSurvCap) { s_sv[i] = v; s_sk[i] = k; }
      }
    }
  }
  __syncthreads();
  const int ns = s_nsurv;
  if (ns <= kSurvCap) {
    // usual case: rank the few survivors directly; order (value desc, token asc)
    if (warp == 0) {
      for (int i = lane; i < ns; i += 32) {
        const float v = s_sv[i]; const int k = s_sk[i];
        int rank = 0;
        for (int j = 0; j < ns; ++j) rank += cand_better(s_sv[j], s_sk[j], v, k);
        if (rank < N) { a.cand.v[(long long)r * kMaxBeam + rank] = v; a.cand.k[(long long)r * kMaxBeam + rank] = k; }
      }
      if (lane == 0) a.cand.n[r] = min(ns, N);
    }
    return;
  }
  // ---- many ties at the bound: per-thread sorted lists, merged by warp and then across warps
  TopList best;
  best.init();
  float admit = -INFINITY;
  for (int k = tid; k < V; k += kT) {
    const float v = zs[k];
    if (v > admit) { best.insert(v, k); admit = best.nth(N); }
  }
  const int wn = warp_merge_lists(best, N, s_wv[warp], s_wk[warp]);
  if (lane == 0) s_wn[warp] = wn;
  __syncthreads();
  if (warp == 0) {
    int pos = 0, cnt = 0;
    const int mine = lane < kT / 32 ? s_wn[lane] : 0;
    for (int j = 0; j < N; ++j) {
      float bv = (pos < mine) ? s_wv[lane & 7][pos] : -INFINITY;
      int bk = (pos < mine) ? s_wk[lane & 7][pos] : 0x7fffffff;
      int bl = lane;
#pragma unroll
      for (int o = 4; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int ok = __shfl_xor_sync(0xffffffffu, bk, o);
        const int ol = __shfl_xor_sync(0xffffffffu, bl, o);
        if (cand_better(ov, ok, bv, bk)) { bv = ov; bk = ok; bl = ol; }
      }
      bv = __shfl_sync(0xffffffffu, bv, 0); bk = __shfl_sync(0xffffffffu, bk, 0); bl = __shfl_sync(0xffffffffu, bl, 0);
      if (bv == -INFINITY) break;
      if (lane == 0) { a.cand.v[(long long)r * kMaxBeam + j] = bv; a.cand.k[(long long)r * kMaxBeam + j] = bk; }
      if (lane == bl) ++pos;
      ++cnt;
    }
    if (lane == 0) a.cand.n[r] = cnt;
  }
}

}  // namespace

size_t scan_select_smem_bytes(int S, int V) { return (size_t)S * V * sizeof(float); }

bool scan_select_fits(int S, int V) { return scan_select_smem_bytes(S, V) <= (size_t)200 * 1024; }

int scan_select_setup() {
  return cudaFuncSetAttribute(scan_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) == cudaSuccess
             ? TW_OK : TW_ERR_CUDA;
}

void launch_scan_select(const ScanSelectArgs& a, cudaStream_t st) {
  if (a.R_max <= 0) return;
  scan_select_kernel<<<a.R_max, kT, scan_select_smem_bytes(a.S, a.V), st>>>(a);
}

}  // namespace tw
