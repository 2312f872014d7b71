// fp32 (TW_MODE_F32) stage kernels: SIMT GEMM, joiner contraction, log-softmax, Eq. 3-7.
// This is the accuracy path: plain FFMA accumulation and libm tanhf/expf/logf, no fast-math.
#include "topn.cuh"
#include "tw_internal.cuh"

namespace tw {

namespace {

constexpr int BM = 64, BN = 64, BK = 16, LDS = BM + 4;

struct GemmParams {
  GemmOperand op[2];
  GemmOut out;
  const int* M_dev;
  int M_max, N;
  // joiner mode
  JoinerRows jr;
  const float* W_out;
  const float* b_out;
  float* z;
};

__device__ __forceinline__ void load4(const float* p, int k, int K, bool valid, float v[4]) {
  if (!valid) { v[0] = v[1] = v[2] = v[3] = 0.f; return; }
  if (k + 3 < K && ((reinterpret_cast<uintptr_t>(p + k) & 15) == 0)) {
    float4 q = *reinterpret_cast<const float4*>(p + k);
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
  } else {
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = (k + i < K) ? p[k + i] : 0.f;
  }
}

// MODE 0: plain / gathered rows, one or two operand pairs.  MODE 1: joiner rows, A = tanh(E + Pp).
template <int MODE>
__global__ void __launch_bounds__(256) gemm_f32_kernel(GemmParams p) {
  __shared__ __align__(16) float As[BK][LDS];
  __shared__ __align__(16) float Bs[BK][LDS];

  int M;
  if (MODE == 1) {
    int R = p.jr.R_dev ? *p.jr.R_dev : p.jr.R_max;
    M = R * p.jr.S;
  } else {
    M = p.M_dev ? *p.M_dev : p.M_max;
  }
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  if (m0 >= M) return;
  const int N = (MODE == 1) ? p.jr.V : p.N;

  const int tid = threadIdx.x;
  const int lrow = tid >> 2, kq = (tid & 3) * 4;
  const int tx = tid & 15, ty = tid >> 4;

  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  const int nops = (MODE == 1) ? 1 : (p.op[1].K > 0 ? 2 : 1);
  for (int o = 0; o < nops; ++o) {
    const float* arow = nullptr;   // MODE 0: A row; MODE 1: E row
    const float* prow = nullptr;   // MODE 1: Pp row
    bool avalid = false;
    const int m = m0 + lrow;
    int K;
    const float* Bmat;
    long long ldB;
    if (MODE == 1) {
      K = p.jr.J; Bmat = p.W_out; ldB = p.jr.J;
      if (m < M) {
        int r = m / p.jr.S, t = m - r * p.jr.S;
        int sl = p.jr.row_slen ? p.jr.row_slen[r] : p.jr.S;
        if (t < sl) {
          avalid = true;
          arow = p.jr.E + (long long)(p.jr.row_e0[r] + t) * K;
          prow = p.jr.Pp + (long long)(p.jr.row_p ? p.jr.row_p[r] : r) * K;
        }
      }
    } else {
      const GemmOperand& op = p.op[o];
      K = op.K; Bmat = op.B; ldB = op.ldB;
      if (m < M) {
        avalid = true;
        arow = op.A + (long long)(op.idx ? op.idx[m] : m) * op.ldA;
      }
    }
    const int n = n0 + lrow;
    const bool bvalid = n < N;
    const float* brow = Bmat + (long long)(bvalid ? n : 0) * ldB;

    for (int k0 = 0; k0 < K; k0 += BK) {
      float a[4], b[4];
      load4(arow, k0 + kq, K, avalid, a);
      if (MODE == 1) {
        float q[4];
        load4(prow, k0 + kq, K, avalid, q);
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = (avalid && k0 + kq + i < K) ? (p.jr.act == TW_ACT_RELU ? fmaxf(a[i] + q[i], 0.f) : tanhf(a[i] + q[i])) : 0.f;
      }
      load4(brow, k0 + kq, K, bvalid, b);
#pragma unroll
      for (int i = 0; i < 4; ++i) { As[kq + i][lrow] = a[i]; Bs[kq + i][lrow] = b[i]; }
      __syncthreads();
#pragma unroll
      for (int k = 0; k < BK; ++k) {
        float4 av = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
        float4 bv = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
        float aa[4] = {av.x, av.y, av.z, av.w}, bb[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(aa[i], bb[j], acc[i][j]);
      }
      __syncthreads();
    }
  }

#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= M) continue;
    float* crow;
    const float* bias;
    if (MODE == 1) {
      int r = m / p.jr.S, t = m - r * p.jr.S;
      int sl = p.jr.row_slen ? p.jr.row_slen[r] : p.jr.S;
      if (t >= sl) continue;
      crow = p.z + (long long)m * N;
      bias = p.b_out;
    } else {
      crow = p.out.C + (long long)(p.out.oidx ? p.out.oidx[m] : m) * p.out.ldC;
      bias = p.out.bias;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n < N) crow[n] = acc[i][j] + (bias ? bias[n] : 0.f);
    }
  }
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__global__ void __launch_bounds__(256) log_softmax_kernel(JoinerRows jr, int blank, float* z) {
  __shared__ float red[8];
  __shared__ float bcast;
  const int R = jr.R_dev ? *jr.R_dev : jr.R_max;
  const int m = blockIdx.x;
  const int r = m / jr.S, t = m - r * jr.S;
  if (r >= R) return;
  float* row = z + (long long)m * jr.V;
  const int sl = jr.row_slen ? jr.row_slen[r] : jr.S;
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  if (t >= sl) {
    for (int k = tid; k < jr.V; k += 256) row[k] = (k == blank) ? 0.f : -INFINITY;
    return;
  }
  const bool hat = jr.hat != 0;
  float mx = -INFINITY;
  for (int k = tid; k < jr.V; k += 256) if (!hat || k != blank) mx = fmaxf(mx, row[k]);
  mx = warp_max(mx);
  if (lane == 0) red[w] = mx;
  __syncthreads();
  if (tid == 0) { float v = red[0]; for (int i = 1; i < 8; ++i) v = fmaxf(v, red[i]); bcast = v; }
  __syncthreads();
  mx = bcast;
  float s = 0.f;
  for (int k = tid; k < jr.V; k += 256) if (!hat || k != blank) s += expf(row[k] - mx);
  s = warp_sum(s);
  __syncthreads();
  if (lane == 0) red[w] = s;
  __syncthreads();
  if (tid == 0) { float v = 0.f; for (int i = 0; i < 8; ++i) v += red[i]; bcast = mx + logf(v); }
  __syncthreads();
  const float lse = bcast;
  if (!hat) {
    for (int k = tid; k < jr.V; k += 256) row[k] = row[k] - lse;
    return;
  }
  // factorised output: log sigmoid(zb), log(1 - sigmoid(zb)) without cancellation
  const float zb = row[blank];
  __syncthreads();                               // every thread has read the blank logit before it is overwritten
  const float sp = (zb >= 0.f) ? log1pf(expf(-zb)) : -zb + log1pf(expf(zb));     // softplus(-zb)
  const float log_pb = -sp, log_rest = -sp - zb;
  const bool skip = log_pb > jr.log_tau;         // blank thresholding: the label part is left out
  if (skip && tid == 0 && jr.skipped != nullptr) atomicAdd(jr.skipped, 1ull);
  for (int k = tid; k < jr.V; k += 256)
    row[k] = (k == blank) ? log_pb : (skip ? -INFINITY : row[k] - lse + log_rest);
}

// One CTA per hypothesis row.  Eq. 3-7 through the occupancy recursion
//   la[1] = ld_old[1];  la[t+1] = logaddexp(la[t] + lb[t], ld_old[t+1]),  lb[t] = log J(t, blank)
//   log d(k, t) = la[t] + log J(t, k);  delta_nb(k) = sum_t d(k, t);  delta_phi = la[S'] + lb[S'].
__global__ void __launch_bounds__(256) expand_f32_kernel(const float* __restrict__ logp,
                                                         const float* __restrict__ ld_old,
                                                         const int* row_slen, const int* R_dev,
                                                         int R_max, int S, int V, int blank,
                                                         float* ldphi, float* ldnb, float* la_out,
                                                         double* ldphi_d, double* la_d, CandOut cand) {
  __shared__ float la[kMaxSeg];
  __shared__ float s_wv[8][kMaxBeam];
  __shared__ int s_wk[8][kMaxBeam];
  __shared__ int s_wn[8];
  const int R = R_dev ? *R_dev : R_max;
  const int r = blockIdx.x;
  if (r >= R) return;
  const int sl = row_slen ? min(max(row_slen[r], 0), S) : S;   // a caller's value outside [0, S] must not index past the row
  const float* lp = logp + (long long)r * S * V;
  if (threadIdx.x == 0) {
    // the recursion is S steps long and its values grow to hundreds of nats: carry it in float64
    double a = (double)ld_old[(long long)r * S];
    double phi = -INFINITY;
    for (int t = 0; t < sl; ++t) {
      la[t] = (float)a;
      if (la_d) la_d[(long long)r * S + t] = a;
      const double nxt = a + (double)lp[(long long)t * V + blank];   // -inf + finite stays -inf
      if (t + 1 < sl) a = logaddexp_d(nxt, (double)ld_old[(long long)r * S + t + 1]);
      else phi = nxt;
    }
    for (int t = (sl > 0 ? sl : 0); t < S; ++t) {
      la[t] = -INFINITY;
      if (la_d) la_d[(long long)r * S + t] = -INFINITY;
    }
    ldphi[r] = (float)phi;
    if (ldphi_d) ldphi_d[r] = phi;
  }
  __syncthreads();
  if (threadIdx.x < S) la_out[(long long)r * S + threadIdx.x] = la[threadIdx.x];
  TopList best;
  best.init();
  float admit = -INFINITY;
  for (int k = threadIdx.x; k < V; k += blockDim.x) {
    float out = -INFINITY;
    if (k != blank) {
      float mx = -INFINITY;
      for (int t = 0; t < sl; ++t) mx = fmaxf(mx, la[t] + lp[(long long)t * V + k]);
      if (mx > -INFINITY) {
        float s = 0.f;
        for (int t = 0; t < sl; ++t) s += expf(la[t] + lp[(long long)t * V + k] - mx);
        out = mx + logf(s);
      }
    }
    if (ldnb) ldnb[(long long)r * V + k] = out;
    if (cand.n && out > admit) {          // the blank column is -inf and never a candidate
      best.insert(out, k);
      admit = best.nth(cand.N);
    }
  }
  if (cand.n == nullptr) return;
  // ChooseNBestExpansions, first stage: this row's N best non-blank tokens
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int wn = warp_merge_lists(best, cand.N, s_wv[warp], s_wk[warp]);
  if (lane == 0) s_wn[warp] = wn;
  __syncthreads();
  if (warp == 0) {
    int pos = 0;
    const int mine = lane < 8 ? s_wn[lane] : 0;
    int cnt = 0;
    for (int j = 0; j < cand.N; ++j) {
      float bv = (pos < mine) ? s_wv[lane][pos] : -INFINITY;
      int bk = (pos < mine) ? s_wk[lane][pos] : 0x7fffffff;
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
      if (lane == 0) { cand.v[(long long)r * kMaxBeam + j] = bv; cand.k[(long long)r * kMaxBeam + j] = bk; }
      if (lane == bl) ++pos;
      ++cnt;
    }
    if (lane == 0) cand.n[r] = cnt;
  }
}

__global__ void rows_from_groups_kernel(const int* row_group, const int* seg_len, int R, int G, int S,
                                        int* row_e0, int* row_slen) {
  int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= R) return;
  int g = row_group[r];
  if (g < 0 || g >= G) { row_e0[r] = 0; row_slen[r] = 0; return; }   // no such segment: an empty row, nothing is read for it
  row_e0[r] = g * S;
  int sl = seg_len ? seg_len[g] : S;
  row_slen[r] = sl < 0 ? 0 : (sl > S ? S : sl);
}

}  // namespace

void launch_gemm_f32(const GemmOperand& op1, const GemmOperand& op2, const GemmOut& out,
                     const int* M_dev, int M_max, int N, cudaStream_t st) {
  if (M_max <= 0 || N <= 0) return;
  GemmParams p{};
  p.op[0] = op1; p.op[1] = op2; p.out = out; p.M_dev = M_dev; p.M_max = M_max; p.N = N;
  dim3 grid((N + BN - 1) / BN, (M_max + BM - 1) / BM);
  gemm_f32_kernel<0><<<grid, 256, 0, st>>>(p);
}

void launch_joiner_f32(const JoinerRows& rows, const float* W_out, const float* b_out, float* z,
                       cudaStream_t st) {
  if (rows.R_max <= 0) return;
  GemmParams p{};
  p.jr = rows; p.W_out = W_out; p.b_out = b_out; p.z = z;
  long long M_max = (long long)rows.R_max * rows.S;
  dim3 grid((rows.V + BN - 1) / BN, (unsigned)((M_max + BM - 1) / BM));
  gemm_f32_kernel<1><<<grid, 256, 0, st>>>(p);
}

void launch_log_softmax(const JoinerRows& rows, int blank, float* z, cudaStream_t st) {
  if (rows.R_max <= 0) return;
  log_softmax_kernel<<<rows.R_max * rows.S, 256, 0, st>>>(rows, blank, z);
}

void launch_expand_f32(const float* logp, const float* ld_old, const int* row_slen, const int* R_dev,
                       int R_max, int S, int V, int blank, float* ldphi, float* ldnb, float* la,
                       double* ldphi_d, double* la_d, const CandOut& cand, cudaStream_t st) {
  if (R_max <= 0) return;
  expand_f32_kernel<<<R_max, 256, 0, st>>>(logp, ld_old, row_slen, R_dev, R_max, S, V, blank, ldphi,
                                           ldnb, la, ldphi_d, la_d, cand);
}

void launch_rows_from_groups(const int* row_group, const int* seg_len, int R, int G, int S, int* row_e0,
                             int* row_slen, cudaStream_t st) {
  if (R <= 0) return;
  rows_from_groups_kernel<<<(R + 255) / 256, 256, 0, st>>>(row_group, seg_len, R, G, S, row_e0, row_slen);
}

}  // namespace tw
