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

constexpr int kMaxT = 1024;         // threads per CTA: 256 for small rows, 1024 when one CTA fills the SM
constexpr int kMaxGroups = kMaxT / 16;   // groups of 16 threads: their maxima bound the N-th best value
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

template <bool FAST>
__device__ __forceinline__ float ex(float x) { return FAST ? __expf(x) : expf(x); }
template <bool FAST>
__device__ __forceinline__ float lg(float x) { return FAST ? __logf(x) : logf(x); }

// FAST: hardware exp2/log2 approximations (bf16 mode, where the operands carry 2^-9 already)
template <bool FAST>
__global__ void __launch_bounds__(kMaxT) scan_select_kernel(ScanSelectArgs a) {
  extern __shared__ __align__(16) float zs[];          // [S][V] logits of this row; row 0 later holds dnb
  __shared__ float s_lse[kMaxSeg], s_w[kMaxSeg];
  __shared__ float s_gmax[kMaxGroups];
  __shared__ float s_bound;
  __shared__ int s_nsurv;
  __shared__ float s_sv[kSurvCap];
  __shared__ int s_sk[kSurvCap];
  __shared__ float s_wv[kMaxT / 32][kMaxBeam];
  __shared__ int s_wk[kMaxT / 32][kMaxBeam];
  __shared__ int s_wn[kMaxT / 32];

  pdl_wait();
  pdl_trigger();
  const int R = a.R_dev ? *a.R_dev : a.R_max;
  const int r = blockIdx.x;
  if (r >= R) return;
  const int S = a.S, V = a.V, blank = a.blank;
  const int sl = a.dnb_in ? 1 : (a.row_slen ? min(max(a.row_slen[r], 0), S) : S);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int kT = blockDim.x, nwarps = kT >> 5;
  const int gshift = kT >= 256 ? 4 : 3, ngroups = kT >> gshift;   // groups of 16 threads (8 in a 128-thread CTA): at least 16 groups
  const float* z = a.z + (long long)r * S * V;

  float tmax = -INFINITY;
  if (a.dnb_in != nullptr) {
    // selection only: the row of delta_nb values is given
    const float* src = a.dnb_in + (long long)r * V;
    if ((V & 3) == 0) {
      for (int k = tid * 4; k < V; k += kT * 4) {
        float4 v = *reinterpret_cast<const float4*>(src + k);
        if (a.dnb_linear) {                                // order is the same as that of the logs
          v.x = v.x > 0.f ? v.x : -INFINITY; v.y = v.y > 0.f ? v.y : -INFINITY;
          v.z = v.z > 0.f ? v.z : -INFINITY; v.w = v.w > 0.f ? v.w : -INFINITY;
        }
        *reinterpret_cast<float4*>(zs + k) = v;
        tmax = fmaxf(fmaxf(tmax, fmaxf(v.x, v.y)), fmaxf(v.z, v.w));
      }
    } else {
      for (int k = tid; k < V; k += kT) {
        float v = src[k];
        if (a.dnb_linear) v = v > 0.f ? v : -INFINITY;
        zs[k] = v; tmax = fmaxf(tmax, v);
      }
    }
    if (tid == 0) s_nsurv = 0;
    __syncthreads();
  } else {
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
  for (int t = warp; t < sl; t += nwarps) {
    const float* row = zs + t * V;
    float mx = -INFINITY;
    for (int k = lane; k < V; k += 32) mx = fmaxf(mx, row[k]);
    mx = wmax(mx);
    float s = 0.f;
    for (int k = lane; k < V; k += 32) s += ex<FAST>(row[k] - mx);
    s = wsum(s);
    if (lane == 0) {
      const float lse = mx + lg<FAST>(s);
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
  for (int k = tid; k < V; k += kT) {
    float out = -INFINITY;
    if (k != blank) {
      float mx = -INFINITY;
      for (int t = 0; t < sl; ++t) mx = fmaxf(mx, s_w[t] + zs[t * V + k]);
      if (mx > -INFINITY) {
        float s = 0.f;
        for (int t = 0; t < sl; ++t) s += ex<FAST>(s_w[t] + zs[t * V + k] - mx);
        out = mx + lg<FAST>(s);
      }
    }
    if (sl > 0) zs[k] = out;                 // only this thread ever touches column k
    if (a.ldnb) a.ldnb[(long long)r * V + k] = out;
    tmax = fmaxf(tmax, out);
  }
  }
  if (a.cand.n == nullptr) return;
  const int N = a.cand.N;

  // ---- a lower bound of the row's N-th best value: the N-th largest of 16 group maxima (each is a
  // distinct element of the row), so everything at or above it is a small superset of the answer
  for (int o = (1 << gshift) >> 1; o > 0; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
  if ((tid & ((1 << gshift) - 1)) == 0) s_gmax[tid >> gshift] = tmax;
  __syncthreads();
  if (warp == 0) {
    for (int g = lane; g < ngroups; g += 32) {
      const float mine = s_gmax[g];
      int rank = 0;
      for (int j = 0; j < ngroups; ++j) {
        const float o = s_gmax[j];
        rank += (o > mine) || (o == mine && j < g);
      }
      if (rank == N - 1) s_bound = mine;       // N <= 16 <= ngroups: exactly one group has this rank
    }
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
        if (rank < N) {
          a.cand.v[(long long)r * kMaxBeam + rank] = a.dnb_linear ? __logf(v) : v;
          a.cand.k[(long long)r * kMaxBeam + rank] = k;
        }
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
    const int mine = lane < nwarps ? s_wn[lane] : 0;
    for (int j = 0; j < N; ++j) {
      float bv = (pos < mine) ? s_wv[lane][pos] : -INFINITY;
      int bk = (pos < mine) ? s_wk[lane][pos] : 0x7fffffff;
      int bl = lane;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int ok = __shfl_xor_sync(0xffffffffu, bk, o);
        const int ol = __shfl_xor_sync(0xffffffffu, bl, o);
        if (cand_better(ov, ok, bv, bk)) { bv = ov; bk = ok; bl = ol; }
      }
      bv = __shfl_sync(0xffffffffu, bv, 0); bk = __shfl_sync(0xffffffffu, bk, 0); bl = __shfl_sync(0xffffffffu, bl, 0);
      if (bv == -INFINITY) break;
      if (lane == 0) { a.cand.v[(long long)r * kMaxBeam + j] = a.dnb_linear ? __logf(bv) : bv; a.cand.k[(long long)r * kMaxBeam + j] = bk; }
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
  cudaError_t e1 = cudaFuncSetAttribute(scan_select_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  cudaError_t e2 = cudaFuncSetAttribute(scan_select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
  return (e1 == cudaSuccess && e2 == cudaSuccess) ? TW_OK : TW_ERR_CUDA;
}

void launch_scan_select(const ScanSelectArgs& a, bool fast_math, cudaStream_t st) {
  if (a.R_max <= 0) return;
  const size_t smem = a.dnb_in ? scan_select_smem_bytes(1, a.V) : scan_select_smem_bytes(a.S, a.V);
  // a row that takes most of an SM's shared memory runs alone there: give it the whole SM's threads
  // selection from a short row (delta_nb given): 128-thread CTAs, so that a whole batch of rows is resident at once
  const int threads = smem > 96 * 1024 ? 1024 : (smem > 48 * 1024 ? 512 : ((a.dnb_in && smem <= 16 * 1024) ? 128 : 256));
  if (fast_math) launch_pdl(scan_select_kernel<true>, dim3(a.R_max), dim3(threads), smem, st, a);
  else launch_pdl(scan_select_kernel<false>, dim3(a.R_max), dim3(threads), smem, st, a);
}

}  // namespace tw
