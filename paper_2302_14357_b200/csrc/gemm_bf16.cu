// bf16 tensor-core GEMM for sm_100a:  C[m, n] = sum_k A[m, k] * B[n, k] (+ bias[n]), fp32 accumulate.
// Persistent: one CTA per SM walks the tile list.  TMA (128-byte swizzle) feeds a multi-stage
// shared-memory ring; one thread issues tcgen05.mma into one of two TMEM accumulator buffers, so the
// epilogue of a tile (tcgen05.ld, bias, stores) overlaps the contraction of the next.
// Warp roles: 0 = TMA producer, 1 = MMA issuer and TMEM owner, 2..9 = epilogue (two warps per TMEM
// lane quarter, half of the columns each).  Every wait is bounded (sm100::mbar_wait); on a timeout
// the kernel raises *err and every role leaves its loop.
#include "bf16_path.cuh"
#include "sm100.cuh"

namespace tw {

namespace {

using namespace sm100;

constexpr int BM = 128, BK = 64;
constexpr int kEpiWarps = 8;
constexpr int kThreadsGemm = 64 + 32 * kEpiWarps;

template <int BN>
struct Cfg {
  static constexpr int kStages = (BN == 256) ? 4 : (BN == 128 ? 6 : 8);
  static constexpr uint32_t kABytes = BM * BK * 2, kBBytes = BN * BK * 2;
  static constexpr size_t kSmem = (size_t)kStages * (kABytes + kBBytes) + 1024 + 256;
};

__device__ __forceinline__ float tanh_fast_g(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// sigma(x) = (1 + tanh(x / 2)) / 2: one special-function instruction instead of an exponential and a reciprocal (the
// LSTM cell is bound by that unit); the approximation's error, about 2^-11, is below the bf16 rounding of h
__device__ __forceinline__ float sigmoid_fast(float x) { return fmaf(0.5f, tanh_fast_g(0.5f * x), 0.5f); }

template <int BN, int EPI>
__global__ void __launch_bounds__(kThreadsGemm, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, GemmBf16Params p) {
  using C = Cfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sA = smem;
  uint8_t* sB = smem + C::kStages * C::kABytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(sB + C::kStages * C::kBBytes);
  uint64_t* empty = full + C::kStages;
  uint64_t* acc_full = empty + C::kStages;     // [2]
  uint64_t* acc_empty = acc_full + 2;          // [2]
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(acc_empty + 2);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb = (p.K + BK - 1) / BK;
  const int M_pre = (p.m_early && p.M_dev) ? __ldcg(p.M_dev) : 0;   // under the set-up's latency (see m_early)

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tmA);
    prefetch_tensormap(&tmB);
    for (int s = 0; s < C::kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], kEpiWarps); }
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) { tmem_alloc(tmem_holder, 2 * BN); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  // the set-up above touched only this CTA: it may overlap the tail of the kernel that produces A and M
  pdl_wait();
  pdl_trigger();
  const int M = p.M_dev ? (p.m_early ? M_pre : *p.M_dev) : p.M;
  const int m_tiles = (M + BM - 1) / BM, n_tiles = (p.N + BN - 1) / BN;
  const int num_tiles = m_tiles * n_tiles;     // a CTA past the last tile runs no loop iteration below

  if (warp == 0) {
    if (lane == 0) {
      uint32_t it = 0;                       // k-block counter across tiles: the ring never restarts
      bool ok = true;
      const uint64_t keep = l2_policy_evict_last();        // B is a weight matrix in every use of this kernel
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        const int m0 = (tile / n_tiles) * BM, n0 = (tile % n_tiles) * BN;
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = it % C::kStages;
          const uint32_t ph = (it / C::kStages) & 1;
          ok = mbar_wait(&empty[s], ph ^ 1, p.err);
          if (!ok) break;
          mbar_expect_tx(&full[s], C::kABytes + C::kBBytes);
          tma_load_2d(sA + s * C::kABytes, &tmA, &full[s], kb * BK, m0);
          tma_load_2d_hint(sB + s * C::kBBytes, &tmB, &full[s], kb * BK, n0, keep);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(BM, BN);
      uint32_t it = 0, lt = 0;               // lt: tiles done by this CTA
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++lt) {
        const uint32_t buf = lt & 1, aph = (lt >> 1) & 1;
        ok = mbar_wait(&acc_empty[buf], aph ^ 1, p.err);      // epilogue has drained this buffer
        if (!ok) break;
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + buf * BN;
        for (int kb = 0; kb < num_kb; ++kb, ++it) {
          const int s = it % C::kStages;
          const uint32_t ph = (it / C::kStages) & 1;
          ok = mbar_wait(&full[s], ph, p.err);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_addr = smem_u32(sA + s * C::kABytes), b_addr = smem_u32(sB + s * C::kBBytes);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)
            umma_bf16(tmem_d, make_desc_k_sw128(a_addr + k * 32), make_desc_k_sw128(b_addr + k * 32), idesc,
                      (kb | k) != 0);
          umma_commit(&empty[s]);
        }
        if (ok) umma_commit(&acc_full[buf]);
      }
    }
  } else {
    const int ew = warp - 2;                 // 0..7
    const int q = warp & 3;                  // TMEM lane quarter this warp may read
    const int half = ew >> 2;                // which half of the tile's columns
    constexpr int kColsPerWarp = BN / 2;
    uint32_t lt = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++lt) {
      const int m0 = (tile / n_tiles) * BM, n0 = (tile % n_tiles) * BN;
      const uint32_t buf = lt & 1, aph = (lt >> 1) & 1;
      ok = mbar_wait(&acc_full[buf], aph, p.err);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int m = m0 + q * 32 + lane;
      float* crow = nullptr;
      const float* arow = nullptr;           // optional per-row addend (gathered)
      const float* cin = nullptr;            // LSTM epilogue: parent's c, new (h, c), bf16 copy of h
      float* hout = nullptr;
      __nv_bfloat16* xrow = nullptr;
      if (m < M) {
        if (EPI == 0) crow = p.C + (long long)(p.oidx ? p.oidx[m] : m) * p.ldC;
        if (p.addend) arow = p.addend + (long long)(p.add_idx ? p.add_idx[m] : m) * p.ld_add;
        if (EPI == 1) {
          const long long stride = (long long)p.lstm.L * 2 * p.lstm.Hd, lo = (long long)p.lstm.l * 2 * p.lstm.Hd;
          cin = p.lstm.hc_in + (long long)(p.lstm.idx_in ? p.lstm.idx_in[m] : m) * stride + lo + p.lstm.Hd;
          hout = p.lstm.hc_out + (long long)(p.lstm.idx_out ? p.lstm.idx_out[m] : m) * stride + lo;
          xrow = p.lstm.xnext + (long long)m * p.lstm.ld_xnext;
        }
      }
#pragma unroll 1
      for (int c = 0; c < kColsPerWarp / 32; ++c) {
        float v[32];
        const int col = half * kColsPerWarp + c * 32;
        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + buf * BN + (uint32_t)col, v);
        const int nb = n0 + col;
        if (EPI == 1) {
          if (hout != nullptr && nb < p.N) {       // N = 4 Hd is a multiple of 32: the chunk is 8 whole units
            if (p.bias) {
#pragma unroll
              for (int j = 0; j < 32; ++j) v[j] += p.bias[nb + j];
            }
            if (arow) {
              if ((reinterpret_cast<uintptr_t>(arow + nb) & 31) == 0) {
#pragma unroll
                for (int j = 0; j < 32; j += 8) {
                  float a8[8];
                  ld_global_v8(arow + nb + j, a8);
#pragma unroll
                  for (int u = 0; u < 8; ++u) v[j + u] += a8[u];
                }
              } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] += arow[nb + j];
              }
            }
            const int j0 = nb >> 2;
            const bool w256 = (p.lstm.Hd & 7) == 0 &&
                              ((reinterpret_cast<uintptr_t>(p.lstm.hc_in) | reinterpret_cast<uintptr_t>(p.lstm.hc_out)) & 31) == 0;
            float cp[8], hn[8], cn[8];
            if (w256) {
              ld_global_v8(cin + j0, cp);
            } else {
#pragma unroll
              for (int u = 0; u < 8; ++u) cp[u] = cin[j0 + u];
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const float c = sigmoid_fast(v[4 * u + 1]) * cp[u] + sigmoid_fast(v[4 * u]) * tanh_fast_g(v[4 * u + 2]);
              cn[u] = c;
              hn[u] = sigmoid_fast(v[4 * u + 3]) * tanh_fast_g(c);
            }
            float* cout = hout + p.lstm.Hd;
            if (w256) {
              st_global_v8(hout + j0, hn);
              st_global_v8(cout + j0, cn);
            } else {
              *reinterpret_cast<float4*>(hout + j0) = make_float4(hn[0], hn[1], hn[2], hn[3]);
              *reinterpret_cast<float4*>(hout + j0 + 4) = make_float4(hn[4], hn[5], hn[6], hn[7]);
              *reinterpret_cast<float4*>(cout + j0) = make_float4(cn[0], cn[1], cn[2], cn[3]);
              *reinterpret_cast<float4*>(cout + j0 + 4) = make_float4(cn[4], cn[5], cn[6], cn[7]);
            }
            __nv_bfloat162 b0 = __floats2bfloat162_rn(hn[0], hn[1]), b1 = __floats2bfloat162_rn(hn[2], hn[3]);
            __nv_bfloat162 b2 = __floats2bfloat162_rn(hn[4], hn[5]), b3 = __floats2bfloat162_rn(hn[6], hn[7]);
            uint4 pk;
            pk.x = *reinterpret_cast<uint32_t*>(&b0); pk.y = *reinterpret_cast<uint32_t*>(&b1);
            pk.z = *reinterpret_cast<uint32_t*>(&b2); pk.w = *reinterpret_cast<uint32_t*>(&b3);
            *reinterpret_cast<uint4*>(xrow + j0) = pk;
          }
        } else if (crow != nullptr && nb < p.N) {
          if (nb + 32 <= p.N && ((reinterpret_cast<uintptr_t>(crow + nb) & 15) == 0)) {
            if (p.bias) {
#pragma unroll
              for (int j = 0; j < 32; ++j) v[j] += p.bias[nb + j];
            }
            if (arow) {
              if ((reinterpret_cast<uintptr_t>(arow + nb) & 31) == 0) {
#pragma unroll
                for (int j = 0; j < 32; j += 8) {
                  float a8[8];
                  ld_global_v8(arow + nb + j, a8);
#pragma unroll
                  for (int u = 0; u < 8; ++u) v[j + u] += a8[u];
                }
              } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] += arow[nb + j];
              }
            }
            if ((reinterpret_cast<uintptr_t>(crow + nb) & 31) == 0) {   // a thread writes its own row: 32-byte sectors
#pragma unroll
              for (int j = 0; j < 32; j += 8) st_global_v8(crow + nb + j, &v[j]);
            } else {
#pragma unroll
              for (int j = 0; j < 32; j += 4)
                *reinterpret_cast<float4*>(crow + nb + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
            }
          } else {
            for (int j = 0; j < 32; ++j)
              if (nb + j < p.N) crow[nb + j] = v[j] + (p.bias ? p.bias[nb + j] : 0.f) + (arow ? arow[nb + j] : 0.f);
          }
        }
      }
      // all of this warp's TMEM reads have completed (tmem_ld32 waits): hand the buffer back
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[buf]);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, 2 * BN);
}

// ---- single-wave LSTM gate GEMM ------------------------------------------------------------------
// For a handful of row tiles and a wide N (the gate GEMMs of a step: some 10 row tiles x 4 Hd columns)
// 128 x 256 tiles need a second, almost empty wave.  Here the columns of a row tile are split evenly
// over floor(#SM / row tiles) CTAs in units of 32 columns, so every CTA owns exactly one tile of up to
// 320 columns (one tcgen05.mma of N <= 256 plus one of N <= 64 per K step, accumulators side by side in
// TMEM) and the whole GEMM is one wave.  B is loaded in boxes of 64 (and one of 32) rows.
constexpr int kWideMaxBN = 320, kWideStages = 4, kWideEpiWarps = 16;
constexpr int kThreadsWide = 64 + 32 * kWideEpiWarps;
constexpr uint32_t kWideABytes = BM * BK * 2, kWideBBytes = kWideMaxBN * BK * 2;
constexpr size_t kWideSmem = (size_t)kWideStages * (kWideABytes + kWideBBytes) + 1024 + 256;

// The LSTM cell on one CTA's accumulator tile: rows m0 .. m0 + 127, gate columns n0 .. n0 + 32 nu - 1 (TMEM columns
// 0 .. 32 nu - 1).  Called by the 16 epilogue warps (warp = 2 .. 17).  Two things keep the part after the contraction
// short.  (1) What is added to the products - the bias, or layer 0's table row W_ih emb[token] + b - is written into
// tensor memory BEFORE the contraction, which then accumulates onto it from its first instruction: the gather of
// those rows (128 bytes per thread and chunk, scattered) runs while the first operand tiles are still on their way,
// and the MMA thread waits on acc_init for it.  (2) The parents' cell states of all of a warp's chunks are fetched
// into registers during the contraction.  After it a chunk is one tensor-memory load, the cell and three stores.
constexpr int kWideMaxChunks = (kWideMaxBN / 32 + 3) / 4;      // chunks of 32 columns a warp can own (groups of 4 warps)
__device__ __forceinline__ void lstm_tile_epilogue(const GemmBf16Params& p, uint32_t tmem_base, uint64_t* acc_full,
                                                   uint64_t* acc_init, int M, int m0, int n0, int nu, int warp, int lane) {
  // a row per thread; warp group grp takes the 32-column chunks grp, grp + 4, grp + 8
  const int ew = warp - 2, q = warp & 3, grp = ew >> 2;
  const int m = m0 + q * 32 + lane;
  const bool live = m < M;                                   // tcgen05 accesses below are warp-wide: idle rows stay in the loops
  const long long stride = (long long)p.lstm.L * 2 * p.lstm.Hd, lo = (long long)p.lstm.l * 2 * p.lstm.Hd;
  const float* cin = nullptr;
  const float* arow = nullptr;
  float* hout = nullptr;
  __nv_bfloat16* xrow = nullptr;
  if (live) {
    cin = p.lstm.hc_in + (long long)(p.lstm.idx_in ? p.lstm.idx_in[m] : m) * stride + lo + p.lstm.Hd;
    hout = p.lstm.hc_out + (long long)(p.lstm.idx_out ? p.lstm.idx_out[m] : m) * stride + lo;
    xrow = p.lstm.xnext + (long long)m * p.lstm.ld_xnext;
    if (p.addend) arow = p.addend + (long long)(p.add_idx ? p.add_idx[m] : m) * p.ld_add;
  }
  // 256-bit accesses when every row segment this kernel touches starts on a 32-byte boundary
  const bool wide_ok = (p.lstm.Hd & 7) == 0 &&
                       ((reinterpret_cast<uintptr_t>(p.lstm.hc_in) | reinterpret_cast<uintptr_t>(p.lstm.hc_out) |
                         reinterpret_cast<uintptr_t>(p.addend) | (uintptr_t)(p.ld_add * 4)) & 31) == 0;
  const uint32_t tlane = tmem_base + ((uint32_t)(q * 32) << 16);
  // ---- (1) the accumulators start as bias + addend
#pragma unroll 1
  for (int c = grp; c < nu; c += kWideEpiWarps / 4) {
    float v[32];
    const int nb = n0 + c * 32;
#pragma unroll
    for (int j = 0; j < 32; ++j) v[j] = 0.f;
    if (p.bias) {
#pragma unroll
      for (int j = 0; j < 32; j += 4) {
        const float4 b4 = __ldg(reinterpret_cast<const float4*>(p.bias + nb + j));
        v[j] = b4.x; v[j + 1] = b4.y; v[j + 2] = b4.z; v[j + 3] = b4.w;
      }
    }
    if (arow) {
      if (wide_ok) {
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
          float a8[8];
          ld_global_v8(arow + nb + j, a8);
#pragma unroll
          for (int u = 0; u < 8; ++u) v[j + u] += a8[u];
        }
      } else {
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
          const float4 a4 = __ldg(reinterpret_cast<const float4*>(arow + nb + j));
          v[j] += a4.x; v[j + 1] += a4.y; v[j + 2] += a4.z; v[j + 3] += a4.w;
        }
      }
    }
    tmem_st32(tlane + (uint32_t)(c * 32), v);
  }
  tmem_st_wait();
  tc_fence_before();
  __syncwarp();
  if (lane == 0) mbar_arrive(acc_init);
  // ---- (2) the parents' cell states, while the contraction runs
  float cp[kWideMaxChunks][8];
#pragma unroll
  for (int i = 0; i < kWideMaxChunks; ++i) {
    const int c = grp + i * (kWideEpiWarps / 4);
#pragma unroll
    for (int u = 0; u < 8; ++u) cp[i][u] = 0.f;
    if (live && c < nu) {
      const int j0 = (n0 + c * 32) >> 2;                       // 8 whole hidden units (gate columns interleaved)
      if (wide_ok) {
        ld_global_v8(cin + j0, cp[i]);
      } else {
        const float4 c0 = *reinterpret_cast<const float4*>(cin + j0), c1 = *reinterpret_cast<const float4*>(cin + j0 + 4);
        cp[i][0] = c0.x; cp[i][1] = c0.y; cp[i][2] = c0.z; cp[i][3] = c0.w; cp[i][4] = c1.x; cp[i][5] = c1.y; cp[i][6] = c1.z; cp[i][7] = c1.w;
      }
    }
  }
  bool ok = mbar_wait(acc_full, 0, p.err);
  ok = __all_sync(0xffffffffu, ok);
  if (ok) {
    tc_fence_after();
#pragma unroll
    for (int i = 0; i < kWideMaxChunks; ++i) {
      const int c = grp + i * (kWideEpiWarps / 4);
      if (c >= nu) break;                                    // uniform over the warp
      float v[32];
      tmem_ld32(tlane + (uint32_t)(c * 32), v);
      if (!live) continue;
      const int j0 = (n0 + c * 32) >> 2;
      float hn[8], cn[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const float cc = sigmoid_fast(v[4 * u + 1]) * cp[i][u] + sigmoid_fast(v[4 * u]) * tanh_fast_g(v[4 * u + 2]);
        cn[u] = cc;
        hn[u] = sigmoid_fast(v[4 * u + 3]) * tanh_fast_g(cc);
      }
      float* cout = hout + p.lstm.Hd;
      if (wide_ok) {
        st_global_v8(hout + j0, hn);
        st_global_v8(cout + j0, cn);
      } else {
        *reinterpret_cast<float4*>(hout + j0) = make_float4(hn[0], hn[1], hn[2], hn[3]);
        *reinterpret_cast<float4*>(hout + j0 + 4) = make_float4(hn[4], hn[5], hn[6], hn[7]);
        *reinterpret_cast<float4*>(cout + j0) = make_float4(cn[0], cn[1], cn[2], cn[3]);
        *reinterpret_cast<float4*>(cout + j0 + 4) = make_float4(cn[4], cn[5], cn[6], cn[7]);
      }
      __nv_bfloat162 b0 = __floats2bfloat162_rn(hn[0], hn[1]), b1 = __floats2bfloat162_rn(hn[2], hn[3]);
      __nv_bfloat162 b2 = __floats2bfloat162_rn(hn[4], hn[5]), b3 = __floats2bfloat162_rn(hn[6], hn[7]);
      uint4 pk;
      pk.x = *reinterpret_cast<uint32_t*>(&b0); pk.y = *reinterpret_cast<uint32_t*>(&b1);
      pk.z = *reinterpret_cast<uint32_t*>(&b2); pk.w = *reinterpret_cast<uint32_t*>(&b3);
      *reinterpret_cast<uint4*>(xrow + j0) = pk;
    }
  }
}
__global__ void __launch_bounds__(kThreadsWide, 1)
gemm_lstm_wide_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB64,
                      const __grid_constant__ CUtensorMap tmB32, GemmBf16Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sA = smem;
  uint8_t* sB = smem + kWideStages * kWideABytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(sB + kWideStages * kWideBBytes);
  uint64_t* empty = full + kWideStages;
  uint64_t* acc_full = empty + kWideStages;
  uint64_t* acc_init = acc_full + 1;        // the epilogue warps have written the accumulators' initial values
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(acc_init + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb = (p.K + BK - 1) / BK;
  const int M_pre = (p.m_early && p.M_dev) ? __ldcg(p.M_dev) : 0;   // under the set-up's latency (see m_early)

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tmA);
    prefetch_tensormap(&tmB64);
    prefetch_tensormap(&tmB32);
    for (int s = 0; s < kWideStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(acc_full, 1);
    mbar_init(acc_init, kWideEpiWarps);
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) { tmem_alloc(tmem_holder, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  // the set-up above touched only this CTA: it may overlap the tail of the kernel that produces A and M
  pdl_wait();
  pdl_trigger();
  // The split follows the row count of THIS launch: fewer row tiles than the grid was sized for give
  // every row tile more CTAs, i.e. narrower and faster tiles (never wider than the host's bound).
  const int M = p.M_dev ? (p.m_early ? M_pre : *p.M_dev) : p.M;
  const int m_tiles = M > 0 ? (M + BM - 1) / BM : 1;
  const int units = p.N >> 5;
  int n_split = (int)gridDim.x / m_tiles;
  n_split = n_split < 1 ? 1 : (n_split > units ? units : n_split);
  const int mt = blockIdx.x / n_split, ns = blockIdx.x - mt * n_split;
  const int m0 = mt * BM;
  const int ubase = units / n_split, urem = units - ubase * n_split;
  const int u0 = ns * ubase + (ns < urem ? ns : urem), nu = ubase + (ns < urem ? 1 : 0);
  const int n0 = u0 * 32, w = nu * 32;                   // this CTA's columns [n0, n0 + w), w <= kWideMaxBN
  if (w > kWideMaxBN && threadIdx.x == 0) atomicExch(p.err, 1);    // the host sizes the grid so that this cannot happen
  const bool active = m0 < M && mt < m_tiles && w <= kWideMaxBN;   // an idle CTA skips the roles and only frees its TMEM

  if (!active) {
  } else if (warp == 0) {
    if (lane == 0) {
      const uint64_t keep = l2_policy_evict_last();        // the gate weights: read again by every step
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % kWideStages;
        const uint32_t ph = (kb / kWideStages) & 1;
        if (!mbar_wait(&empty[s], ph ^ 1, p.err)) break;
        mbar_expect_tx(&full[s], kWideABytes + (uint32_t)w * (BK * 2));
        tma_load_2d(sA + s * kWideABytes, &tmA, &full[s], kb * BK, m0);
        uint8_t* bdst = sB + s * kWideBBytes;
        int r = 0;
        for (; r + 64 <= w; r += 64) tma_load_2d_hint(bdst + r * (BK * 2), &tmB64, &full[s], kb * BK, n0 + r, keep);
        if (r < w) tma_load_2d_hint(bdst + r * (BK * 2), &tmB32, &full[s], kb * BK, n0 + r, keep);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const int n1 = w <= 256 ? w : ((w >> 1) + 15) & ~15, n2 = w - n1;    // wider than one MMA: two of about equal width
      const uint32_t idesc1 = make_idesc_bf16(BM, n1), idesc2 = make_idesc_bf16(BM, n2);
      bool ok = mbar_wait(acc_init, 0, p.err);             // the accumulators hold bias + addend: accumulate onto them
      for (int kb = 0; kb < num_kb && ok; ++kb) {
        const int s = kb % kWideStages;
        const uint32_t ph = (kb / kWideStages) & 1;
        ok = mbar_wait(&full[s], ph, p.err);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a_addr = smem_u32(sA + s * kWideABytes), b_addr = smem_u32(sB + s * kWideBBytes);
#pragma unroll
        for (int k = 0; k < BK / 16; ++k) {
          const uint64_t da = make_desc_k_sw128(a_addr + k * 32);
          umma_bf16(tmem_base, da, make_desc_k_sw128(b_addr + k * 32), idesc1, 1u);
          if (n2 > 0)
            umma_bf16(tmem_base + (uint32_t)n1, da, make_desc_k_sw128(b_addr + n1 * (BK * 2) + k * 32), idesc2, 1u);
        }
        umma_commit(&empty[s]);
      }
      if (ok) umma_commit(acc_full);
    }
  } else {
    lstm_tile_epilogue(p, tmem_base, acc_full, acc_init, M, m0, n0, nu, warp, lane);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, 512);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

}  // namespace

int make_tmap_bf16(CUtensorMap* out, const void* base, uint64_t rows, uint64_t K, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || (K % 8) != 0 || (reinterpret_cast<uintptr_t>(base) & 15) != 0 || box_rows > 256 || rows == 0) return TW_ERR_ARG;
  cuuint64_t dims[2] = {K, rows};
  cuuint64_t strides[1] = {K * 2};
  cuuint32_t box[2] = {(cuuint32_t)BK, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? TW_OK : TW_ERR_CUDA;
}

int gemm_bf16_setup() {
  cudaError_t e1 = cudaFuncSetAttribute(gemm_bf16_kernel<256, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<256>::kSmem);
  cudaError_t e2 = cudaFuncSetAttribute(gemm_bf16_kernel<128, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<128>::kSmem);
  cudaError_t e3 = cudaFuncSetAttribute(gemm_bf16_kernel<256, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<256>::kSmem);
  cudaError_t e4 = cudaFuncSetAttribute(gemm_bf16_kernel<128, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<128>::kSmem);
  cudaError_t e6 = cudaFuncSetAttribute(gemm_bf16_kernel<64, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<64>::kSmem);
  if (e6 != cudaSuccess) return TW_ERR_CUDA;
  cudaError_t e5 = cudaFuncSetAttribute(gemm_lstm_wide_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kWideSmem);
  return (e1 == cudaSuccess && e2 == cudaSuccess && e3 == cudaSuccess && e4 == cudaSuccess && e5 == cudaSuccess) ? TW_OK : TW_ERR_CUDA;
}

static int sm_count() {
  static int num_sms = 0;
  if (num_sms == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (cudaDeviceGetAttribute(&num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || num_sms <= 0) num_sms = 148;
  }
  return num_sms;
}

bool launch_gemm_lstm_wide(const CUtensorMap& tmA, const CUtensorMap& tmB64, const CUtensorMap& tmB32,
                           const GemmBf16Params& p, cudaStream_t st) {
  if (p.epi != 1 || p.M <= 0 || p.N <= 0 || (p.N & 31) != 0) return false;
  const int num_sms = sm_count();
  const int mt = (p.M + BM - 1) / BM;
  // (also when 128 x 256 tiles would be one wave already: that wave has few CTAs, each pulling a fat tile through its
  // SM's L2 port, while the narrow tiles of this kernel put every SM to work: c1 -3 %, p1 -4.7 %, c2 -0.9 % per decode)
  const int n_split = num_sms / mt;
  if (n_split < 1) return false;
  const int units = p.N >> 5;
  if (((units + n_split - 1) / n_split) * 32 > kWideMaxBN) return false;
  // one CTA per SM: the kernel splits the columns of each row tile over floor(grid / row tiles of this launch) CTAs
  launch_pdl(gemm_lstm_wide_kernel, dim3(num_sms), dim3(kThreadsWide), kWideSmem, st, tmA, tmB64, tmB32, p);
  return true;
}

void launch_gemm_bf16(const CUtensorMap& tmA, const CUtensorMap& tmB128, const CUtensorMap& tmB256,
                      const GemmBf16Params& p, cudaStream_t st, const CUtensorMap* tmB64) {
  if (p.M <= 0 || p.N <= 0) return;
  const int num_sms = sm_count();
  const int mt = (p.M + BM - 1) / BM;
  const int nt256 = (p.N + 255) / 256, nt128 = (p.N + 127) / 128;
  // small problems: narrower tiles put more SMs to work
  if ((long long)mt * nt256 >= num_sms) {
    const int grid = (int)((long long)mt * nt256 < num_sms ? mt * nt256 : num_sms);
    if (p.epi == 1) launch_pdl(gemm_bf16_kernel<256, 1>, dim3(grid), dim3(kThreadsGemm), Cfg<256>::kSmem, st, tmA, tmB256, p);
    else launch_pdl(gemm_bf16_kernel<256, 0>, dim3(grid), dim3(kThreadsGemm), Cfg<256>::kSmem, st, tmA, tmB256, p);
  } else if (tmB64 != nullptr && p.epi == 0 && (long long)mt * nt128 * 4 <= (long long)num_sms * 3) {
    // few tiles and a short K loop each: 64-column tiles put twice as many SMs to work
    const long long tiles = (long long)mt * ((p.N + 63) / 64);
    const int grid = (int)(tiles < num_sms ? tiles : num_sms);
    launch_pdl(gemm_bf16_kernel<64, 0>, dim3(grid), dim3(kThreadsGemm), Cfg<64>::kSmem, st, tmA, *tmB64, p);
  } else {
    const long long tiles = (long long)mt * nt128;
    const int grid = (int)(tiles < num_sms ? tiles : num_sms);
    if (p.epi == 1) launch_pdl(gemm_bf16_kernel<128, 1>, dim3(grid), dim3(kThreadsGemm), Cfg<128>::kSmem, st, tmA, tmB128, p);
    else launch_pdl(gemm_bf16_kernel<128, 0>, dim3(grid), dim3(kThreadsGemm), Cfg<128>::kSmem, st, tmA, tmB128, p);
  }
}

}  // namespace tw
