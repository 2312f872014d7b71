// Elementwise kernels of the bf16 path: conversions, operand gathers and the joiner's A operand.
#include "bf16_path.cuh"

namespace tw {

namespace {

__global__ void f32_to_bf16_kernel(const float* __restrict__ src, __nv_bfloat16* __restrict__ dst, long long n) {
  long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i + 3 < n && ((reinterpret_cast<uintptr_t>(src + i) & 15) == 0)) {
    const float4 v = *reinterpret_cast<const float4*>(src + i);
    __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
    *reinterpret_cast<__nv_bfloat162*>(dst + i) = a;
    *reinterpret_cast<__nv_bfloat162*>(dst + i + 2) = b;
  } else {
    for (int j = 0; j < 4 && i + j < n; ++j) dst[i + j] = __float2bfloat16_rn(src[i + j]);
  }
}

__global__ void bf16_to_f32_kernel(const __nv_bfloat16* __restrict__ src, float* __restrict__ dst, long long n) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = __bfloat162float(src[i]);
}

__global__ void gather_concat_bf16_kernel(const float* __restrict__ src1, const int* idx1, long long ld1, int K1,
                                          const float* __restrict__ src2, const int* idx2, long long ld2, int K2,
                                          const int* n_dev, int n_max, __nv_bfloat16* __restrict__ dst) {
  const int n = n_dev ? *n_dev : n_max;
  const int r = blockIdx.x;
  if (r >= n) return;
  const int K = K1 + K2;
  const float* a = src1 + (long long)(idx1 ? idx1[r] : r) * ld1;
  const float* b = K2 > 0 ? src2 + (long long)(idx2 ? idx2[r] : r) * ld2 : nullptr;
  __nv_bfloat16* d = dst + (long long)r * K;
  for (int k = threadIdx.x; k < K; k += blockDim.x) d[k] = __float2bfloat16_rn(k < K1 ? a[k] : b[k - K1]);
}

__global__ void gather_parents_bf16_kernel(GatherParents g, const int* n_dev, int n_max) {
  pdl_wait();
  pdl_trigger();
  const int r = blockIdx.x, l = blockIdx.y;
  int n, parent;
  if (g.wl.B > 0) {
    // scan of n_new: each thread sums a contiguous run of utterances, then the runs are scanned
    __shared__ int s_run[128], s_hit[2], s_total;
    const int B = g.wl.B, per = (B + blockDim.x - 1) / blockDim.x;
    const int b0 = threadIdx.x * per, b1 = min(b0 + per, B);
    int mine = 0;
    for (int b = b0; b < b1; ++b) mine += g.wl.n_new[b];
    // exclusive scan of the 128 run sums: shuffles inside the warps, then the four warp totals
    __shared__ int s_wtot[4];
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    int inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int v = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += v; }
    if (lane == 31) s_wtot[wid] = inc;
    __syncthreads();
    int before = 0;
    for (int w = 0; w < wid; ++w) before += s_wtot[w];
    s_run[threadIdx.x] = before + inc - mine;
    if (threadIdx.x == blockDim.x - 1) s_total = before + inc;
    __syncthreads();
    n = s_total;
    if (r == 0 && l == 0 && threadIdx.x == 0) *g.wl.n_out = n;
    if (r >= n) return;
    int off = s_run[threadIdx.x];
    for (int b = b0; b < b1; ++b) {
      const int nb = g.wl.n_new[b];
      if (r >= off && r < off + nb) { s_hit[0] = b; s_hit[1] = r - off; }   // exactly one thread, one utterance
      off += nb;
    }
    __syncthreads();
    const int e = s_hit[0] * kMaxBeam + s_hit[1];
    parent = g.wl.new_par[e];
    if (l == 0 && threadIdx.x == 0) {
      g.wl.pw_new[r] = g.wl.new_slot[e];
      g.wl.pw_par[r] = parent;
      g.wl.pw_tok[r] = g.wl.new_tok[e];
    }
  } else {
    n = n_dev ? *n_dev : n_max;
    if (r >= n) return;
    parent = g.idx ? g.idx[r] : r;
  }
  const float* src = g.hc + (long long)parent * g.stride + (long long)l * 2 * g.Hd;
  __nv_bfloat16* d = g.dst[l] + (long long)r * g.ld[l] + g.off[l];
  // Hd is a multiple of 8 in bf16 mode (the operands' K must be): 8 floats in, one 16-byte store out per thread
  if (((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(d)) & 15) == 0 && (g.Hd & 7) == 0) {
    for (int k = threadIdx.x * 8; k < g.Hd; k += blockDim.x * 8) {
      const float4 a = *reinterpret_cast<const float4*>(src + k), b = *reinterpret_cast<const float4*>(src + k + 4);
      __nv_bfloat162 p0 = __floats2bfloat162_rn(a.x, a.y), p1 = __floats2bfloat162_rn(a.z, a.w);
      __nv_bfloat162 p2 = __floats2bfloat162_rn(b.x, b.y), p3 = __floats2bfloat162_rn(b.z, b.w);
      uint4 pk;
      pk.x = *reinterpret_cast<uint32_t*>(&p0); pk.y = *reinterpret_cast<uint32_t*>(&p1);
      pk.z = *reinterpret_cast<uint32_t*>(&p2); pk.w = *reinterpret_cast<uint32_t*>(&p3);
      *reinterpret_cast<uint4*>(d + k) = pk;
    }
  } else {
    for (int k = threadIdx.x * 2; k < g.Hd; k += blockDim.x * 2)
      *reinterpret_cast<__nv_bfloat162*>(d + k) = __floats2bfloat162_rn(src[k], src[k + 1]);
  }
}

__global__ void permute_cols_f32_kernel(const float* __restrict__ src, const int* __restrict__ perm, long long rows,
                                        int cols, float* __restrict__ dst) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= rows * cols) return;
  const long long r = i / cols;
  const int c = (int)(i - r * cols);
  dst[i] = src[r * cols + perm[c]];
}

__device__ __forceinline__ float tanh_fast(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// one CTA per (row, frame); the tanh error of the approximate instruction (about 2^-11) is below the
// bf16 rounding (2^-9) of the stored operand
__global__ void joiner_A_bf16_kernel(JoinerRows jr, __nv_bfloat16* __restrict__ A) {
  const int R = jr.R_dev ? *jr.R_dev : jr.R_max;
  const int m = blockIdx.x;
  const int r = m / jr.S, t = m - r * jr.S;
  if (r >= R) return;
  const int sl = jr.row_slen ? jr.row_slen[r] : jr.S;
  __nv_bfloat16* dst = A + (long long)m * jr.J;
  if (t >= sl) {
    for (int j = threadIdx.x; j < jr.J; j += blockDim.x) dst[j] = __float2bfloat16_rn(0.f);
    return;
  }
  const float* e = jr.E + (long long)(jr.row_e0[r] + t) * jr.J;
  const float* p = jr.Pp + (long long)(jr.row_p ? jr.row_p[r] : r) * jr.J;
  for (int j = threadIdx.x; j < jr.J; j += blockDim.x) dst[j] = __float2bfloat16_rn(jr.act == TW_ACT_RELU ? fmaxf(e[j] + p[j], 0.f) : tanh_fast(e[j] + p[j]));
}

}  // namespace

void launch_f32_to_bf16(const float* src, __nv_bfloat16* dst, long long n, cudaStream_t st) {
  if (n <= 0) return;
  const long long threads = (n + 3) / 4;
  f32_to_bf16_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(src, dst, n);
}

void launch_bf16_to_f32(const __nv_bfloat16* src, float* dst, long long n, cudaStream_t st) {
  if (n > 0) bf16_to_f32_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(src, dst, n);
}

void launch_gather_concat_bf16(const float* src1, const int* idx1, long long ld1, int K1, const float* src2,
                               const int* idx2, long long ld2, int K2, const int* n_dev, int n_max,
                               __nv_bfloat16* dst, cudaStream_t st) {
  if (n_max <= 0) return;
  gather_concat_bf16_kernel<<<n_max, 256, 0, st>>>(src1, idx1, ld1, K1, src2, idx2, ld2, K2, n_dev, n_max, dst);
}

void launch_gather_parents_bf16(const GatherParents& g, const int* n_dev, int n_max, cudaStream_t st) {
  if (n_max <= 0 || g.L <= 0) return;
  launch_pdl(gather_parents_bf16_kernel, dim3(n_max, g.L), dim3(128), 0, st, g, n_dev, n_max);
}

void launch_permute_cols_f32(const float* src, const int* perm, long long rows, int cols, float* dst, cudaStream_t st) {
  const long long n = rows * cols;
  if (n > 0) permute_cols_f32_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(src, perm, rows, cols, dst);
}

void launch_joiner_A_bf16(const JoinerRows& rows, __nv_bfloat16* A, cudaStream_t st) {
  if (rows.R_max <= 0) return;
  joiner_A_bf16_kernel<<<rows.R_max * rows.S, 256, 0, st>>>(rows, A);
}

}  // namespace tw
