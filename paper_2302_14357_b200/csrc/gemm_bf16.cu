// bf16 tensor-core GEMM for sm_100a:  C[m, n] = sum_k A[m, k] * B[n, k] (+ bias[n]), fp32 accumulate.
// TMA (128-byte swizzle) feeds a multi-stage shared-memory ring; one thread issues tcgen05.mma into a
// TMEM accumulator; four warps read the accumulator back with tcgen05.ld and write the tile.
// Warp roles: 0 = TMA producer, 1 = MMA issuer and TMEM owner, 2..5 = epilogue (one TMEM lane quarter
// each).  Every wait is bounded (sm100::mbar_wait); on a timeout the kernel raises *err and exits.
#include "bf16_path.cuh"
#include "sm100.cuh"

namespace tw {

namespace {

using namespace sm100;

constexpr int BM = 128, BK = 64;

template <int BN>
struct Cfg {
  static constexpr int kStages = (BN == 256) ? 4 : 6;
  static constexpr uint32_t kABytes = BM * BK * 2, kBBytes = BN * BK * 2;
  static constexpr size_t kSmem = (size_t)kStages * (kABytes + kBBytes) + 1024 + 256;
};

template <int BN>
__global__ void __launch_bounds__(192, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, GemmBf16Params p) {
  using C = Cfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* sA = smem;
  uint8_t* sB = smem + C::kStages * C::kABytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(sB + C::kStages * C::kBBytes);
  uint64_t* empty = full + C::kStages;
  uint64_t* accum = empty + C::kStages;
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(accum + 1);

  const int M = p.M_dev ? *p.M_dev : p.M;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  if (m0 >= M) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb = (p.K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    prefetch_tensormap(&tmA);
    prefetch_tensormap(&tmB);
    for (int s = 0; s < C::kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(accum, 1);
    fence_barrier_init();
    fence_proxy_async_smem();
  }
  if (warp == 1) { tmem_alloc(tmem_holder, BN); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  if (warp == 0) {
    if (lane == 0) {
      for (int kb = 0; kb < num_kb; ++kb) {
        const int s = kb % C::kStages;
        const uint32_t ph = (kb / C::kStages) & 1;
        if (!mbar_wait(&empty[s], ph ^ 1, p.err)) break;
        mbar_expect_tx(&full[s], C::kABytes + C::kBBytes);
        tma_load_2d(sA + s * C::kABytes, &tmA, &full[s], kb * BK, m0);
        tma_load_2d(sB + s * C::kBBytes, &tmB, &full[s], kb * BK, n0);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(BM, BN);
      bool ok = true;
      for (int kb = 0; kb < num_kb && ok; ++kb) {
        const int s = kb % C::kStages;
        const uint32_t ph = (kb / C::kStages) & 1;
        ok = mbar_wait(&full[s], ph, p.err);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a_addr = smem_u32(sA + s * C::kABytes), b_addr = smem_u32(sB + s * C::kBBytes);
#pragma unroll
        for (int k = 0; k < BK / 16; ++k)
          umma_bf16(tmem_base, make_desc_k_sw128(a_addr + k * 32), make_desc_k_sw128(b_addr + k * 32), idesc,
                    (kb | k) != 0);
        umma_commit(&empty[s]);
      }
      umma_commit(accum);
    }
  } else {
    const int q = warp & 3;
    const int m = m0 + q * 32 + lane;
    bool ok = mbar_wait(accum, 0, p.err);
    ok = __all_sync(0xffffffffu, ok);
    tc_fence_after();
    if (ok) {
      float* crow = nullptr;
      if (m < M) crow = p.C + (long long)(p.oidx ? p.oidx[m] : m) * p.ldC;
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        float v[32];
        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * 32), v);
        const int nb = n0 + c * 32;
        if (crow != nullptr && nb < p.N) {
          if (nb + 32 <= p.N && ((reinterpret_cast<uintptr_t>(crow + nb) & 15) == 0)) {
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              float4 o;
              o.x = v[j] + (p.bias ? p.bias[nb + j] : 0.f);
              o.y = v[j + 1] + (p.bias ? p.bias[nb + j + 1] : 0.f);
              o.z = v[j + 2] + (p.bias ? p.bias[nb + j + 2] : 0.f);
              o.w = v[j + 3] + (p.bias ? p.bias[nb + j + 3] : 0.f);
              *reinterpret_cast<float4*>(crow + nb + j) = o;
            }
          } else {
            for (int j = 0; j < 32; ++j)
              if (nb + j < p.N) crow[nb + j] = v[j] + (p.bias ? p.bias[nb + j] : 0.f);
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, BN);
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
  cudaError_t e1 = cudaFuncSetAttribute(gemm_bf16_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<256>::kSmem);
  cudaError_t e2 = cudaFuncSetAttribute(gemm_bf16_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<128>::kSmem);
  return (e1 == cudaSuccess && e2 == cudaSuccess) ? TW_OK : TW_ERR_CUDA;
}

void launch_gemm_bf16(const CUtensorMap& tmA, const CUtensorMap& tmB128, const CUtensorMap& tmB256,
                      const GemmBf16Params& p, cudaStream_t st) {
  if (p.M <= 0 || p.N <= 0) return;
  const int mt = (p.M + BM - 1) / BM;
  const int nt256 = (p.N + 255) / 256;
  // small problems: narrower tiles put more SMs to work
  if ((long long)mt * nt256 >= 148) {
    dim3 grid(nt256, mt);
    gemm_bf16_kernel<256><<<grid, 192, Cfg<256>::kSmem, st>>>(tmA, tmB256, p);
  } else {
    dim3 grid((p.N + 127) / 128, mt);
    gemm_bf16_kernel<128><<<grid, 192, Cfg<128>::kSmem, st>>>(tmA, tmB128, p);
  }
}

}  // namespace tw
