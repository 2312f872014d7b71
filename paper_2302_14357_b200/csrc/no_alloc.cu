// tw_joiner_expand_noalloc: the joiner + softmax + Eq. 3-7 stage for callers that must not allocate
// device memory.  Its scratch (the log J tensor and two small row tables) lives in a fixed array that
// is part of the library image, so the call needs no handle, no workspace and no cudaMalloc.
#include <mutex>

#include "tw_internal.cuh"

namespace {

constexpr long long kScratchFloats = TW_NOALLOC_MAX_ELEMS;   // R * S * V of log J
constexpr int kMaxRows = TW_NOALLOC_MAX_ROWS;
constexpr int kMaxDevices = 64;

// [0, kScratchFloats): log J;  then kMaxRows ints of first-frame rows;  then kMaxRows ints of lengths.
static __device__ __align__(256) float g_noalloc_scratch[kScratchFloats + 2 * kMaxRows];

std::mutex g_mu;
float* g_scratch_addr[kMaxDevices] = {};

// The array's name is only a host-side handle; the device address has to be asked for, once per
// device, with that device current.
int scratch_for_current_device(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return TW_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return TW_ERR_CUDA;
    g_scratch_addr[dev] = static_cast<float*>(p);
  }
  *out = g_scratch_addr[dev];
  return TW_OK;
}

}  // namespace

extern "C" int tw_joiner_expand_noalloc(const float* W_out, const float* b_out, int32_t J, int32_t V,
                                        int32_t S, int32_t blank, int32_t joiner_act, const float* E_seg, const float* Pp,
                                        const int32_t* row_group, const int32_t* seg_len,
                                        const float* ld_old, int32_t G, int32_t R, float* out_ldphi,
                                        float* out_ldnb, float* out_la, void* stream) {
  using namespace tw;
  if (!W_out || !b_out || !E_seg || !Pp || !row_group || !ld_old || !out_ldphi || !out_ldnb || !out_la)
    return TW_ERR_ARG;
  if (J < 1 || V < 2 || S < 1 || S > TW_MAX_SEGMENT || blank < 0 || blank >= V || G < 0 || R < 0)
    return TW_ERR_ARG;
  if (joiner_act != TW_ACT_TANH && joiner_act != TW_ACT_RELU) return TW_ERR_ARG;
  if (R > kMaxRows || (long long)R * S * V > kScratchFloats) return TW_ERR_LIMIT;
  if (R == 0) return TW_OK;
  float* scratch = nullptr;
  int s = scratch_for_current_device(&scratch);
  if (s != TW_OK) return s;
  float* logp = scratch;
  int* row_e0 = reinterpret_cast<int*>(scratch + kScratchFloats);
  int* row_slen = row_e0 + kMaxRows;
  cudaStream_t st = (cudaStream_t)stream;
  // every element of the scratch that is read below is written first by this call, so nothing left by
  // an earlier call can leak in and nothing needs clearing
  launch_rows_from_groups(row_group, seg_len, R, G, S, row_e0, row_slen, st);
  JoinerRows jr{};
  jr.E = E_seg; jr.row_e0 = row_e0; jr.Pp = Pp; jr.row_p = nullptr; jr.row_slen = row_slen;
  jr.R_dev = nullptr; jr.R_max = R; jr.S = S; jr.J = J; jr.V = V; jr.act = joiner_act;
  launch_joiner_f32(jr, W_out, b_out, logp, st);
  launch_log_softmax(jr, blank, logp, st);
  launch_expand_f32(logp, ld_old, row_slen, nullptr, R, S, V, blank, out_ldphi, out_ldnb, out_la, nullptr,
                    nullptr, CandOut{}, st);
  return cudaGetLastError() == cudaSuccess ? TW_OK : TW_ERR_CUDA;
}
