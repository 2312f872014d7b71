// C ABI of libtw: handle life-cycle, the decode driver and the separately callable stages.
#include <new>
#include <vector>
#include <stdio.h>
#include <string.h>
#include <math.h>

#include "tw_handle.cuh"

using namespace tw;

namespace {

#define TW_CUDA(h, expr)                                   \
  do {                                                     \
    cudaError_t e_ = (expr);                               \
    if (e_ != cudaSuccess) {                               \
      if (h) (h)->last_cuda = (int)e_;                     \
      return (e_ == cudaErrorMemoryAllocation) ? TW_ERR_ALLOC : TW_ERR_CUDA; \
    }                                                      \
  } while (0)

template <typename T>
int dev_alloc(tw_handle* h, T** p, size_t count) {
  void* q = nullptr;
  if (count == 0) count = 1;
  cudaError_t e = cudaMalloc(&q, count * sizeof(T));
  if (e != cudaSuccess) { h->last_cuda = (int)e; *p = nullptr; return TW_ERR_ALLOC; }
  h->dev_allocs.push_back(q);
  *p = static_cast<T*>(q);
  return TW_OK;
}

#define TW_TRY(expr) do { int s_ = (expr); if (s_ != TW_OK) return s_; } while (0)

// float32 copy of a caller's tensor of the model's element type (bf16 -> float32 is exact)
int copy_weight(tw_handle* h, float** dst, const void* src, size_t count) {
  TW_TRY(dev_alloc(h, dst, count));
  if (h->dtype == TW_BF16) launch_bf16_to_f32(static_cast<const __nv_bfloat16*>(src), *dst, (long long)count, 0);
  else TW_CUDA(h, cudaMemcpy(*dst, src, count * sizeof(float), cudaMemcpyDeviceToDevice));
  return TW_OK;
}

// Encoder frames of the caller's element type -> what the projection GEMM of this mode reads: the bf16 operand
// buffer (TW_MODE_BF16) or float32 frames (TW_MODE_F32; the caller's own buffer when it is float32 already).
const float* stage_frames(tw_handle* h, const void* enc, long long n, cudaStream_t st) {
  if (h->mode == TW_MODE_BF16) {
    if (h->dtype == TW_BF16) cudaMemcpyAsync(h->bf.enc.ptr, enc, (size_t)n * 2, cudaMemcpyDeviceToDevice, st);
    else launch_f32_to_bf16(static_cast<const float*>(enc), h->bf.enc.ptr, n, st);
    return nullptr;
  }
  if (h->dtype == TW_BF16) {
    launch_bf16_to_f32(static_cast<const __nv_bfloat16*>(enc), h->enc_f32, n, st);
    return h->enc_f32;
  }
  return static_cast<const float*>(enc);
}

// fp32 -> bf16 copy of a [rows, K] matrix with its tensor maps
int make_bf16_mat(tw_handle* h, Bf16Mat* m, const float* src, long long rows, long long K, bool as_A, bool as_B) {
  m->rows = rows; m->K = K;
  TW_TRY(dev_alloc(h, &m->ptr, (size_t)(rows * K)));
  if (src) launch_f32_to_bf16(src, m->ptr, rows * K, 0);
  else TW_CUDA(h, cudaMemset(m->ptr, 0, (size_t)(rows * K) * sizeof(__nv_bfloat16)));
  if (as_A) TW_TRY(make_tmap_bf16(&m->as_A, m->ptr, rows, K, 128));
  if (as_B) {
    TW_TRY(make_tmap_bf16(&m->as_B128, m->ptr, rows, K, 128));
    TW_TRY(make_tmap_bf16(&m->as_B256, m->ptr, rows, K, 256));
    TW_TRY(make_tmap_bf16(&m->as_B64, m->ptr, rows, K, 64));
    TW_TRY(make_tmap_bf16(&m->as_B32, m->ptr, rows, K, 32));
  }
  return TW_OK;
}

void gemm_bf16(tw_handle* h, const Bf16Mat& A, const Bf16Mat& B, const int* M_dev, int M, float* C, const int* oidx,
               long long ldC, const float* bias, cudaStream_t st, const float* addend = nullptr,
               const int* add_idx = nullptr, long long ld_add = 0, int m_early = 0) {
  GemmBf16Params p{M_dev, M, (int)B.rows, (int)A.K, C, oidx, ldC, bias, h->bf.err};
  p.addend = addend; p.add_idx = add_idx; p.ld_add = ld_add; p.m_early = m_early;
  launch_gemm_bf16(A.as_A, B.as_B128, B.as_B256, p, st, &B.as_B64);
}

// UpdatePredictorOutput for n hypotheses: one predictor step on tok[i] from the state at row
// (idx_in ? idx_in[i] : i) of hc_in, written to row (idx_out ? idx_out[i] : i) of hc_out; the projected
// output W_p g goes to row (idx_out ? idx_out[i] : i) of Pp_out.  State rows are [L][2][Hd].
void enqueue_predictor(tw_handle* h, const int* tok, const float* hc_in, const int* idx_in, float* hc_out,
                       const int* idx_out, float* Pp_out, const int* n_dev, int n_max, cudaStream_t st,
                       int* launches, const WorkListBuild* wl = nullptr, bool gathered = false) {
  GemmOperand none{};
  if (h->pred_kind == TW_PRED_STATELESS) {
    GemmOperand a{h->emb, tok, h->emb_dim, h->W_p, h->P, h->P};
    GemmOut o{Pp_out, idx_out, h->J, nullptr};
    launch_gemm_f32(a, none, o, n_dev, n_max, h->J, st);
    *launches += 1;
    return;
  }
  const int L = h->L, Hd = h->Hd;
  const long long stride = (long long)L * 2 * Hd;
  if (h->mode == TW_MODE_BF16) {
    // parents' h of every layer -> the recurrent halves of the layers' A operands (one launch)
    GatherParents g{};
    g.hc = hc_in; g.idx = idx_in; g.stride = stride; g.L = L; g.Hd = Hd;
    for (int l = 0; l < L; ++l) { g.dst[l] = h->bf.X[l].ptr; g.ld[l] = (int)h->bf.X[l].K; g.off[l] = (l == 0) ? 0 : Hd; }
    if (wl) g.wl = *wl;                       // the gather kernel builds tok / idx_in / idx_out / *n_dev first
    if (!gathered) launch_gather_parents_bf16(g, n_dev, n_max, st);   // gathered: hyp_step_kernel did both already
    // gate GEMMs with the LSTM cell in the epilogue; each writes the next GEMM's input half as bf16
    for (int l = 0; l < L; ++l) {
      GemmBf16Params p{n_dev, n_max, 4 * Hd, (int)h->bf.X[l].K, nullptr, nullptr, 0, nullptr, h->bf.err};
      if (l == 0) { p.addend = h->bf.EmbProj; p.add_idx = tok; p.ld_add = 4 * Hd; }   // W_ih[0] emb[tok] + b[0]: a table row
      else p.bias = h->bf.bias_perm[l];
      p.epi = 1;
      p.m_early = l > 0;                      // the row count is older than the layer below, which runs ahead of this one
      p.lstm = LstmEpi{hc_in, idx_in, hc_out, idx_out, L, l, Hd,
                       (l + 1 < L) ? h->bf.X[l + 1].ptr : h->bf.Htop.ptr, (l + 1 < L) ? 2LL * Hd : (long long)Hd};
      if (!launch_gemm_lstm_wide(h->bf.X[l].as_A, h->bf.W_cat[l].as_B64, h->bf.W_cat[l].as_B32, p, st))
        launch_gemm_bf16(h->bf.X[l].as_A, h->bf.W_cat[l].as_B128, h->bf.W_cat[l].as_B256, p, st);
    }
    gemm_bf16(h, h->bf.Htop, h->bf.W_p, n_dev, n_max, Pp_out, idx_out, h->J, nullptr, st, nullptr, nullptr, 0, /*m_early=*/1);
    *launches += L + (gathered ? 1 : 2);
    return;
  }
  for (int l = 0; l < L; ++l) {
    const float* x = (l == 0) ? h->emb : hc_out + (long long)(l - 1) * 2 * Hd;
    const int* xi = (l == 0) ? tok : idx_out;
    const long long xld = (l == 0) ? h->emb_dim : stride;
    const int xk = (l == 0) ? h->emb_dim : Hd;
    const float* hp = hc_in + (long long)l * 2 * Hd;
    GemmOperand xo{x, xi, xld, h->W_ih[l], xk, xk};
    GemmOperand ro{hp, idx_in, stride, h->W_hh[l], Hd, Hd};
    GemmOut o{h->gates, nullptr, 4 * Hd, h->b_l[l]};
    launch_gemm_f32(xo, ro, o, n_dev, n_max, 4 * Hd, st);
    // pointwise: c' = sigma(f) c + sigma(i) tanh(g), h' = sigma(o) tanh(c')
    launch_lstm_pointwise(h->gates, idx_out, idx_in, n_dev, n_max, hc_in, hc_out, L, l, Hd, st);
    *launches += 2;
  }
  const float* top = hc_out + (long long)(L - 1) * 2 * Hd;
  GemmOperand to{top, idx_out, stride, h->W_p, h->P, h->P};
  GemmOut o{Pp_out, idx_out, h->J, nullptr};
  launch_gemm_f32(to, none, o, n_dev, n_max, h->J, st);
  *launches += 1;
}

int enqueue_predictor_plain(tw_handle* h, const int* tokens, const float* state_in, int R,
                            float* state_out, float* out_Pp, cudaStream_t st, int* launches) {
  enqueue_predictor(h, tokens, state_in, nullptr, state_out, nullptr, out_Pp, nullptr, R, st, launches);
  return TW_OK;
}

// UpdatePredictorOutput for the work list the compaction kernel built (new slot, parent slot, token).
// build_list: the compaction kernel did not run; the gather kernel derives the work list from the per-utterance
// lists of new hypotheses itself (bf16 mode)
void enqueue_predictor_slots(tw_handle* h, cudaStream_t st, int* launches, bool build_list = false, int B = 0) {
  if (h->pred_kind == TW_PRED_STATELESS) return;   // the joiner reads W_p emb[last token] from a table
  const HypState& hs = h->hs;
  WorkListBuild wl{};
  if (build_list) {
    wl.B = B; wl.n_new = hs.n_new; wl.new_slot = hs.new_slot; wl.new_par = hs.new_par; wl.new_tok = hs.new_tok;
    wl.pw_new = hs.pw_new; wl.pw_par = hs.pw_par; wl.pw_tok = hs.pw_tok; wl.n_out = hs.scalars + kScNPred;
  }
  const bool gathered = build_list && h->hs_fused.inline_gather != 0;
  enqueue_predictor(h, hs.pw_tok, hs.slot_hc, hs.pw_par, hs.slot_hc, hs.pw_new, hs.slot_Pp,
                    hs.scalars + kScNPred, h->R_max, st, launches, build_list && !gathered ? &wl : nullptr, gathered);
}

// E = enc W_e^T for `rows` frames
void enqueue_project(tw_handle* h, const void* enc, int rows, float* E, cudaStream_t st, int* launches) {
  const float* enc32 = stage_frames(h, enc, (long long)rows * h->D_enc, st);
  if (h->mode == TW_MODE_BF16) {
    gemm_bf16(h, h->bf.enc, h->bf.W_e, nullptr, rows, E, nullptr, h->J, nullptr, st);
    *launches += 2;
  } else {
    GemmOperand a{enc32, nullptr, h->D_enc, h->W_e, h->D_enc, h->D_enc};
    GemmOperand none{};
    GemmOut o{E, nullptr, h->J, nullptr};
    launch_gemm_f32(a, none, o, nullptr, rows, h->J, st);
    *launches += 1;
  }
}

// bf16 mode set-up: operand copies, tensor maps, activation buffers
int build_bf16(tw_handle* h) {
  if ((h->D_enc % 8) || (h->J % 8) || (h->P % 8) || (h->emb_dim % 8) || (h->Hd % 8)) return TW_ERR_ARG;
  TW_TRY(gemm_bf16_setup());
  TW_TRY(dev_alloc(h, &h->bf.err, (size_t)1));
  TW_CUDA(h, cudaMemset(h->bf.err, 0, sizeof(int)));
  TW_TRY(make_bf16_mat(h, &h->bf.W_e, h->W_e, h->J, h->D_enc, false, true));
  TW_TRY(make_bf16_mat(h, &h->bf.W_out, h->W_out, h->V, h->J, false, true));
  TW_TRY(make_bf16_mat(h, &h->bf.enc, nullptr, (long long)h->max_batch * h->max_T, h->D_enc, true, false));
  TW_TRY(make_bf16_mat(h, &h->bf.A_join, nullptr, (long long)h->R_max * h->S, h->J, true, false));
  if (h->pred_kind == TW_PRED_LSTM) {
    TW_TRY(make_bf16_mat(h, &h->bf.W_p, h->W_p, h->J, h->P, false, true));
    TW_TRY(make_bf16_mat(h, &h->bf.Htop, nullptr, h->R_max, h->Hd, true, false));
    // Gate GEMM outputs are interleaved by hidden unit (column 4 j + g = gate g of unit j) so that the
    // LSTM cell can run in the GEMM epilogue: weight rows, biases and the table are permuted once here.
    const int G4 = 4 * h->Hd;
    std::vector<int> perm(G4);
    for (int j = 0; j < h->Hd; ++j)
      for (int g = 0; g < 4; ++g) perm[4 * j + g] = g * h->Hd + j;
    int* perm_dev = nullptr;
    TW_TRY(dev_alloc(h, &perm_dev, (size_t)G4));
    TW_CUDA(h, cudaMemcpy(perm_dev, perm.data(), G4 * sizeof(int), cudaMemcpyHostToDevice));
    {
      // EmbProj[k] = W_ih[0] emb[k] + b[0]  (fp32 products of the stored weights, exact inputs), columns permuted
      float* tmp = nullptr;
      TW_CUDA(h, cudaMalloc((void**)&tmp, (size_t)h->V * G4 * sizeof(float)));
      TW_TRY(dev_alloc(h, &h->bf.EmbProj, (size_t)h->V * G4));
      GemmOperand a{h->emb, nullptr, h->emb_dim, h->W_ih[0], h->emb_dim, h->emb_dim};
      GemmOperand none{};
      GemmOut o{tmp, nullptr, G4, h->b_l[0]};
      launch_gemm_f32(a, none, o, nullptr, h->V, G4, 0);
      launch_permute_cols_f32(tmp, perm_dev, h->V, G4, h->bf.EmbProj, 0);
      TW_CUDA(h, cudaDeviceSynchronize());
      cudaFree(tmp);
      TW_TRY(make_bf16_mat(h, &h->bf.W_cat[0], nullptr, G4, h->Hd, false, true));
      launch_gather_concat_bf16(h->W_hh[0], perm_dev, h->Hd, h->Hd, nullptr, nullptr, 0, 0, nullptr, G4, h->bf.W_cat[0].ptr, 0);
      TW_TRY(make_bf16_mat(h, &h->bf.X[0], nullptr, h->R_max, h->Hd, true, false));
    }
    for (int l = 1; l < h->L; ++l) {
      TW_TRY(make_bf16_mat(h, &h->bf.W_cat[l], nullptr, G4, 2 * h->Hd, false, true));
      launch_gather_concat_bf16(h->W_ih[l], perm_dev, h->Hd, h->Hd, h->W_hh[l], perm_dev, h->Hd, h->Hd, nullptr, G4,
                                h->bf.W_cat[l].ptr, 0);
      TW_TRY(make_bf16_mat(h, &h->bf.X[l], nullptr, h->R_max, 2 * h->Hd, true, false));
      TW_TRY(dev_alloc(h, &h->bf.bias_perm[l], (size_t)G4));
      launch_permute_cols_f32(h->b_l[l], perm_dev, 1, G4, h->bf.bias_perm[l], 0);
    }
  }
  // fused joiner: needs S frames of a hypothesis inside one warp and V split into 256-column CTAs
  h->bf.Vp = (h->V + 255) / 256 * 256;
  if (fused_joiner_eligible(h->S, h->bf.Vp, h->J)) {
    h->bf.CL = h->bf.Vp / 256;
    int s = fused_joiner_setup(h->bf.CL, h->S, &h->bf.max_clusters);
    if (s == TW_OK) {
      if (h->bf.Vp == h->V) {
        h->bf.W_out_pad = h->bf.W_out; h->bf.bias_pad = h->b_out; h->bf.ldnb_pad = h->hs.ldnb;
      } else {
        TW_TRY(make_bf16_mat(h, &h->bf.W_out_pad, nullptr, h->bf.Vp, h->J, false, true));      // zero rows
        launch_f32_to_bf16(h->W_out, h->bf.W_out_pad.ptr, (long long)h->V * h->J, 0);
        std::vector<float> bias((size_t)h->bf.Vp, -1e30f);
        TW_CUDA(h, cudaMemcpy(bias.data(), h->b_out, (size_t)h->V * sizeof(float), cudaMemcpyDeviceToHost));
        TW_TRY(dev_alloc(h, &h->bf.bias_pad, (size_t)h->bf.Vp));
        TW_CUDA(h, cudaMemcpy(h->bf.bias_pad, bias.data(), (size_t)h->bf.Vp * sizeof(float), cudaMemcpyHostToDevice));
        TW_TRY(dev_alloc(h, &h->bf.ldnb_pad, (size_t)h->R_max * h->bf.Vp));
      }
      // |z| <= max_k (|W_out[k, :]|_1 + |b_out[k]|) because |tanh| <= 1: small enough => sum exp(z) needs no max
      float* bound_dev = nullptr; float bound = 0.f;
      TW_TRY(dev_alloc(h, &bound_dev, (size_t)1));
      launch_logit_bound(h->bf.W_out.ptr, h->b_out, h->V, h->J, bound_dev, 0);
      TW_CUDA(h, cudaMemcpy(&bound, bound_dev, sizeof(float), cudaMemcpyDeviceToHost));
      h->bf.no_max = (bound <= 40.f) && h->joiner_act == TW_ACT_TANH;   // the bound needs |act| <= 1
      h->bf.zbound = bound;
      TW_TRY(make_bf16_mat(h, &h->bf.A_tiled, nullptr, fused_joiner_A_rows(h->R_max, h->S), h->J, true, false));
      TW_TRY(dev_alloc(h, &h->bf.lse, (size_t)h->R_max * h->S));
      TW_TRY(dev_alloc(h, &h->bf.dmax, (size_t)h->R_max * (h->bf.Vp / 32)));
      TW_TRY(scan_select_setup());
      h->bf.fused_ok = true;
      // default: on for the segment sizes with a specialised kernel instance; the generic instance is
      // currently slower than the staged kernels
      h->bf.fused_on = fused_joiner_specialised(h->S);
    }
  }
  h->hs.defer_rows = 0;
  h->hs.inline_gather = 0;
  h->hs.dnb_sel = nullptr;
  h->hs.dnb_max = nullptr;
  h->hs_fused = h->hs;
  h->hs_fused.logp = nullptr; h->hs_fused.lse = nullptr; h->hs_fused.ldphi_d = nullptr; h->hs_fused.la_d = nullptr;
  if (h->mode == TW_MODE_BF16 && h->bf.fused_ok) {
    h->aux_ok = cudaStreamCreateWithFlags(&h->aux_stream, cudaStreamNonBlocking) == cudaSuccess &&
                cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming) == cudaSuccess &&
                cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming) == cudaSuccess;
    if (!h->aux_ok) cudaGetLastError();
    h->hs_fused.defer_rows = h->aux_ok ? 1 : 0;
    h->hs_fused.dnb_sel = h->bf.ldnb_pad;        // the step's hyp_step_kernel picks the rows' best tokens itself
    h->hs_fused.dnb_max = fused_joiner_writes_maxima(h->S) ? h->bf.dmax : nullptr;
    h->hs_fused.V = h->bf.Vp;                    // row pitch of delta_nb there (padding columns hold 0)
    // hyp_step_kernel builds the predictor's work list and operand rows itself (HypState::inline_gather)
    if (h->hs_fused.defer_rows && h->pred_kind != TW_PRED_STATELESS) {
      h->hs_fused.inline_gather = 1;
      if ((((size_t)4 * h->Hd * sizeof(float)) & 15) == 0) {
        h->hs_fused.pf_table = reinterpret_cast<const char*>(h->bf.EmbProj);
        h->hs_fused.pf_row_bytes = 4 * h->Hd * (int)sizeof(float);
      }
      for (int l = 0; l < h->L; ++l) {
        h->hs_fused.xg_dst[l] = h->bf.X[l].ptr; h->hs_fused.xg_ld[l] = (int)h->bf.X[l].K; h->hs_fused.xg_off[l] = (l == 0) ? 0 : h->Hd;
      }
    }
  }
  TW_CUDA(h, cudaGetLastError());
  return TW_OK;
}

int build_workspace(tw_handle* h) {
  HypState& hs = h->hs;
  const int B = h->max_batch, N = h->N, S = h->S;
  hs.B = B; hs.N = N; hs.S = S; hs.V = h->V; hs.J = h->J; hs.U_cap = h->U_cap; hs.I_max = h->I_max;
  hs.blank = h->blank;
  hs.capB = N * h->I_max;
  hs.capSlot = N * (h->I_max + 1);
  hs.L = h->L; hs.Hd = h->Hd;
  hs.stateless = (h->pred_kind == TW_PRED_STATELESS);
  hs.empty_row = h->blank;
  const size_t nb = (size_t)B, nslot = nb * hs.capSlot, nB = nb * hs.capB, R = (size_t)h->R_max;
  int** per_utt[] = {&hs.len, &hs.t0, &hs.slen, &hs.nA, &hs.nB, &hs.nTop, &hs.iters, &hs.status,
                     &hs.cursor, &hs.n_new, &hs.calls, &hs.joins, &hs.row_off, &hs.new_off, &hs.avail};
  for (int** p : per_utt) TW_TRY(dev_alloc(h, p, nb));
  TW_TRY(dev_alloc(h, &hs.A_slot, nb * kMaxBeam));
  TW_TRY(dev_alloc(h, &hs.A_ls, nb * kMaxBeam));
  TW_TRY(dev_alloc(h, &hs.A_ld, nb * kMaxBeam * S));
  TW_TRY(dev_alloc(h, &hs.A_done, nb * kMaxBeam));
  hs.mono = 0;
  TW_TRY(dev_alloc(h, &hs.B_slot, nB));
  TW_TRY(dev_alloc(h, &hs.B_ls, nB));
  TW_TRY(dev_alloc(h, &hs.B_hash, nB));
  TW_TRY(dev_alloc(h, &hs.B_len, nB));
  TW_TRY(dev_alloc(h, &hs.B_top, nb * kMaxBeam));
  TW_TRY(dev_alloc(h, &hs.carry, nb * kMaxBeam));
  TW_TRY(dev_alloc(h, &hs.slot_len, nslot));
  TW_TRY(dev_alloc(h, &hs.slot_hash, nslot));
  TW_TRY(dev_alloc(h, &hs.slot_tok, nslot * h->U_cap));
  if (!hs.stateless) {
    TW_TRY(dev_alloc(h, &hs.slot_hc, nslot * hs.L * 2 * hs.Hd));
    TW_TRY(dev_alloc(h, &hs.slot_Pp, nslot * h->J));
    TW_TRY(dev_alloc(h, &h->gates, R * 4 * hs.Hd));
  }
  TW_TRY(dev_alloc(h, &hs.new_slot, nb * kMaxBeam));
  TW_TRY(dev_alloc(h, &hs.new_par, nb * kMaxBeam));
  TW_TRY(dev_alloc(h, &hs.new_tok, nb * kMaxBeam));
  TW_TRY(dev_alloc(h, &hs.new_row, nb * kMaxBeam));
  int** per_row[] = {&hs.row_b, &hs.row_e0, &hs.row_p, &hs.row_slen, &hs.pw_new, &hs.pw_par, &hs.pw_tok,
                     &h->stage_e0, &h->stage_slen};
  for (int** p : per_row) TW_TRY(dev_alloc(h, p, R));
  TW_TRY(dev_alloc(h, &hs.row_ld, R * S));
  TW_TRY(dev_alloc(h, &hs.scalars, (size_t)kScCount));
  TW_TRY(dev_alloc(h, &hs.rows_total, (size_t)3));
  TW_TRY(dev_alloc(h, &hs.ldphi, R));
  TW_TRY(dev_alloc(h, &hs.la, R * S));
  if (scan_select_fits(S, h->V)) {
    TW_TRY(scan_select_setup());
    TW_TRY(dev_alloc(h, &hs.lse, R * S));
  }
  TW_TRY(dev_alloc(h, &hs.ldphi_d, R));
  TW_TRY(dev_alloc(h, &hs.cand_v, R * kMaxBeam));
  TW_TRY(dev_alloc(h, &hs.cand_k, R * kMaxBeam));
  TW_TRY(dev_alloc(h, &hs.cand_n, R));
  TW_TRY(dev_alloc(h, &hs.la_d, R * S));
  TW_TRY(dev_alloc(h, &hs.ldnb, R * h->V));
  TW_TRY(dev_alloc(h, &hs.logp, R * S * h->V));
  TW_TRY(dev_alloc(h, &h->E, (nb * h->max_T + 1) * h->J));   // + one dump row for frames a streamed chunk does not hold
  if (h->mode == TW_MODE_F32 && h->dtype == TW_BF16) TW_TRY(dev_alloc(h, &h->enc_f32, nb * h->max_T * h->D_enc));
  TW_TRY(dev_alloc(h, &h->stream_oidx, nb * h->max_T));
  TW_TRY(dev_alloc(h, &h->zero_len, nb));
  TW_CUDA(h, cudaMemset(h->zero_len, 0, nb * sizeof(int)));
  TW_CUDA(h, cudaMemset(hs.scalars, 0, kScCount * sizeof(int)));
  TW_CUDA(h, cudaMemset(hs.rows_total, 0, 3 * sizeof(long long)));
  TW_CUDA(h, cudaHostAlloc((void**)&h->host_flag, (kScCount + 4) * sizeof(long long), cudaHostAllocDefault));
  return TW_OK;
}

int init_impl(tw_handle* h, const tw_model* m, const tw_config* c) {
  h->D_enc = m->D_enc; h->P = m->P; h->J = m->J; h->V = m->V; h->blank = m->blank;
  h->pred_kind = m->pred_kind; h->emb_dim = m->emb_dim; h->joiner_act = m->joiner_act;
  h->dtype = m->dtype; h->esize = m->dtype == TW_BF16 ? 2 : 4;
  h->hat = m->joiner_norm == TW_NORM_HAT ? 1 : 0;
  h->L = (m->pred_kind == TW_PRED_LSTM) ? m->lstm_layers : 0;
  h->Hd = (m->pred_kind == TW_PRED_LSTM) ? m->lstm_hidden : 0;
  h->N = c->N; h->S = c->S; h->mode = c->mode; h->max_batch = c->max_batch; h->max_T = c->max_T;
  h->I_max = c->max_iters_per_segment > 0 ? c->max_iters_per_segment : 4 * c->S + 16;
  h->U_cap = c->max_tokens > 0 ? c->max_tokens : 512;
  h->R_max = h->max_batch * h->N;

  TW_TRY(copy_weight(h, &h->W_e, m->W_e, (size_t)h->J * h->D_enc));
  TW_TRY(copy_weight(h, &h->W_p, m->W_p, (size_t)h->J * h->P));
  TW_TRY(copy_weight(h, &h->W_out, m->W_out, (size_t)h->V * h->J));
  TW_TRY(copy_weight(h, &h->b_out, m->b_out, (size_t)h->V));
  TW_TRY(copy_weight(h, &h->emb, m->emb, (size_t)h->V * h->emb_dim));
  for (int l = 0; l < h->L; ++l) {
    const int in = (l == 0) ? h->emb_dim : h->Hd;
    TW_TRY(copy_weight(h, &h->W_ih[l], m->host_lstm_W_ih[l], (size_t)4 * h->Hd * in));
    TW_TRY(copy_weight(h, &h->W_hh[l], m->host_lstm_W_hh[l], (size_t)4 * h->Hd * h->Hd));
    TW_TRY(copy_weight(h, &h->b_l[l], m->host_lstm_b[l], (size_t)4 * h->Hd));
  }
  TW_TRY(build_workspace(h));
  if (h->mode == TW_MODE_BF16) TW_TRY(build_bf16(h));

  int launches = 0;
  GemmOperand none{};
  float* init_out = nullptr;                 // InitPredictor's output as given by the caller (Sec. 3.2), float32
  if (m->pred_init_out) TW_TRY(copy_weight(h, &init_out, m->pred_init_out, (size_t)h->P));
  if (h->pred_kind == TW_PRED_STATELESS) {
    // W_p emb[k] for every token: the joiner rows index this table by their last token.  A given initial output
    // gets a row of its own after the vocabulary's, which serves the empty prefix.
    TW_TRY(dev_alloc(h, &h->PpTab, (size_t)(h->V + 1) * h->J));
    GemmOperand a{h->emb, nullptr, h->emb_dim, h->W_p, h->P, h->P};
    GemmOut o{h->PpTab, nullptr, h->J, nullptr};
    launch_gemm_f32(a, none, o, nullptr, h->V, h->J, 0);
    if (init_out) {
      GemmOperand a1{init_out, nullptr, h->P, h->W_p, h->P, h->P};
      GemmOut o1{h->PpTab + (size_t)h->V * h->J, nullptr, h->J, nullptr};
      launch_gemm_f32(a1, none, o1, nullptr, 1, h->J, 0);
      h->hs.empty_row = h->hs_fused.empty_row = h->V;
    }
  } else {
    const size_t nhc = (size_t)h->L * 2 * h->Hd;
    TW_TRY(dev_alloc(h, &h->init_Pp, (size_t)h->J));
    if (m->pred_init_state || init_out) {
      // the caller's initial state; zeros without one; the output defaults to the top layer's h
      if (m->pred_init_state) TW_TRY(copy_weight(h, &h->init_hc, m->pred_init_state, nhc));
      else { TW_TRY(dev_alloc(h, &h->init_hc, nhc)); TW_CUDA(h, cudaMemset(h->init_hc, 0, nhc * sizeof(float))); }
      const float* out = init_out ? init_out : h->init_hc + (size_t)(h->L - 1) * 2 * h->Hd;
      GemmOperand a1{out, nullptr, h->P, h->W_p, h->P, h->P};
      GemmOut o1{h->init_Pp, nullptr, h->J, nullptr};
      launch_gemm_f32(a1, none, o1, nullptr, 1, h->J, 0);
    } else {
      // one step on the blank token from an all-zero state
      float* zero = nullptr; int* tok = nullptr;
      TW_TRY(dev_alloc(h, &zero, nhc));
      TW_TRY(dev_alloc(h, &tok, (size_t)1));
      TW_TRY(dev_alloc(h, &h->init_hc, nhc));
      TW_CUDA(h, cudaMemset(zero, 0, nhc * sizeof(float)));
      TW_CUDA(h, cudaMemcpy(tok, &h->blank, sizeof(int), cudaMemcpyHostToDevice));
      TW_TRY(enqueue_predictor_plain(h, tok, zero, 1, h->init_hc, h->init_Pp, 0, &launches));
    }
    h->hs.init_hc = h->hs_fused.init_hc = h->init_hc; h->hs.init_Pp = h->hs_fused.init_Pp = h->init_Pp;
  }
  TW_CUDA(h, cudaGetLastError());
  TW_CUDA(h, cudaDeviceSynchronize());
  return TW_OK;
}

}  // namespace

namespace tw {
void enqueue_joiner_logits(tw_handle* h, const JoinerRows& rows, float* logp, cudaStream_t st, int* launches);
void enqueue_scan(tw_handle* h, const JoinerRows& rows, const float* ld_old, float* logp, float* ldphi,
                  float* ldnb, float* la, double* ldphi_d, double* la_d, const CandOut& cand, cudaStream_t st,
                  int* launches);
void enqueue_joiner_expand_f32(tw_handle* h, const JoinerRows& rows, const float* ld_old, float* logp,
                               float* ldphi, float* ldnb, float* la, double* ldphi_d, double* la_d,
                               const CandOut& cand, cudaStream_t st, int* launches) {
  enqueue_joiner_logits(h, rows, logp, st, launches);
  enqueue_scan(h, rows, ld_old, logp, ldphi, ldnb, la, ldphi_d, la_d, cand, st, launches);
}

// softmax, Eq. 3-7 and the rows' candidates from the raw logits in `logp`
void enqueue_scan(tw_handle* h, const JoinerRows& rows, const float* ld_old, float* logp, float* ldphi,
                  float* ldnb, float* la, double* ldphi_d, double* la_d, const CandOut& cand, cudaStream_t st,
                  int* launches) {
  if (h->hs.lse != nullptr && !h->hat) {
    ScanSelectArgs a{logp, ld_old, rows.row_slen, rows.R_dev, rows.R_max, rows.S, rows.V, h->blank,
                     h->hs.lse, ldphi, ldnb, la, ldphi_d, la_d, cand};
    launch_scan_select(a, h->mode == TW_MODE_BF16, st);
    *launches += 1;
  } else {
    launch_log_softmax(rows, h->blank, logp, st);        // factorised output and blank thresholding included (rows.hat)
    launch_expand_f32(logp, ld_old, rows.row_slen, rows.R_dev, rows.R_max, rows.S, rows.V, h->blank, ldphi,
                      ldnb, la, ldphi_d, la_d, cand, st);
    *launches += 2;
  }
}

// Fused path: joiner, softmax, Eq. 3-7 and per-row candidates with the logits kept in tensor memory
int enqueue_joiner_fused(tw_handle* h, const JoinerRows& rows, const float* ld_old, float* ldphi, float* ldnb,
                         float* la, const CandOut& cand, cudaStream_t st, int* launches, StageMarkFn mark_fn,
                         bool plain_first, int utt_B, int* clear_word) {
  {
    PdlScope first(plain_first ? false : g_pdl_on);
    if (utt_B > 0) launch_joiner_A_tiled_utt(rows, h->hs.row_off, h->hs.nA, utt_B, h->bf.A_tiled.ptr, st);
    else {
      // a small model's weights stay in L2 between two steps by themselves; a large one's W_out is asked for again
      const long long wbytes = (long long)h->bf.W_out_pad.rows * h->bf.W_out_pad.K * 2;
      launch_joiner_A_tiled(rows, h->bf.A_tiled.ptr, st, wbytes >= (4ll << 20) ? h->bf.W_out_pad.ptr : nullptr, wbytes);
    }
  }
  if (mark_fn) mark_fn(h, 3, st);       // operand preparation is booked with the elementwise stages
  if (ldnb == nullptr) ldnb = h->bf.ldnb_pad;   // a caller's buffer has V columns: only with an unpadded vocabulary
  FusedJoinerParams fp{};
  fp.R_dev = rows.R_dev; fp.R_max = rows.R_max; fp.S = rows.S; fp.V = h->bf.Vp; fp.K = rows.J; fp.blank = h->blank;
  fp.CL = h->bf.CL; fp.no_max = h->bf.no_max ? 1 : 0; fp.zbound = h->bf.zbound; fp.bias = h->bf.bias_pad; fp.ld_old = ld_old; fp.row_slen = rows.row_slen;
  fp.ldphi = ldphi; fp.la = la; fp.lse = h->bf.lse; fp.ldnb = ldnb; fp.err = h->bf.err; fp.clear_word = clear_word;
  fp.dmax = (ldnb == h->bf.ldnb_pad && fused_joiner_writes_maxima(rows.S)) ? h->bf.dmax : nullptr;   // the chunk maxima belong to the handle's own delta_nb buffer
  fp.early_w = utt_B > 0 ? 0 : 1;       // (measured: beside the per-utterance operand kernel the early loads cost 6 % at c2, S = 10)
  fp.hat = rows.hat; fp.log2_tau = rows.log_tau * 1.4426950408889634f; fp.skipped = rows.skipped;
  TW_TRY(launch_fused_joiner(h->bf.A_tiled.as_A, h->bf.W_out_pad.as_B256, fp, h->bf.max_clusters, st));
  if (mark_fn) mark_fn(h, 2, st);       // the fused kernel alone
  *launches += 2;
  if (cand.n != nullptr) {      // ChooseNBestExpansions, first stage: the rows' N best tokens
    ScanSelectArgs a{};
    a.R_dev = rows.R_dev; a.R_max = rows.R_max; a.S = rows.S; a.V = h->bf.Vp; a.blank = h->blank;
    a.cand = cand; a.dnb_in = ldnb; a.dnb_linear = 1;
    launch_scan_select(a, true, st);
    *launches += 1;
  }
  return TW_OK;
}

// z[(r, t), :] = W_out tanh(E + Pp) + b_out into `logp` (rows of padding frames hold no result)
void enqueue_joiner_logits(tw_handle* h, const JoinerRows& rows, float* logp, cudaStream_t st, int* launches) {
  if (h->mode == TW_MODE_BF16) {
    launch_joiner_A_bf16(rows, h->bf.A_join.ptr, st);
    const int* M_dev = rows.R_dev ? h->hs.scalars + kScM : nullptr;
    gemm_bf16(h, h->bf.A_join, h->bf.W_out, M_dev, rows.R_max * rows.S, logp, nullptr, rows.V, h->b_out, st);
    *launches += 2;
  } else {
    launch_joiner_f32(rows, h->W_out, h->b_out, logp, st);
    *launches += 1;
  }
}
}  // namespace tw

extern "C" {

int tw_init(const tw_model* m, const tw_config* c, tw_handle** out) {
  if (out) *out = nullptr;
  if (!m || !c || !out) return TW_ERR_ARG;
  if (!m->W_e || !m->W_p || !m->W_out || !m->b_out || !m->emb) return TW_ERR_ARG;
  if (m->D_enc < 1 || m->P < 1 || m->J < 1 || m->V < 2 || m->emb_dim < 1) return TW_ERR_ARG;
  if (m->blank < 0 || m->blank >= m->V) return TW_ERR_ARG;
  if (m->joiner_act != TW_ACT_TANH && m->joiner_act != TW_ACT_RELU) return TW_ERR_ARG;
  if (m->dtype != TW_F32 && m->dtype != TW_BF16) return TW_ERR_ARG;
  if (m->joiner_norm != TW_NORM_SOFTMAX && m->joiner_norm != TW_NORM_HAT) return TW_ERR_ARG;
  if (c->N < 1 || c->N > TW_MAX_BEAM || c->S < 1 || c->S > TW_MAX_SEGMENT) return TW_ERR_ARG;
  if (m->V - 1 < c->N) return TW_ERR_ARG;
  if (c->max_batch < 1 || c->max_T < 1 || c->max_iters_per_segment < 0 || c->max_tokens < 0) return TW_ERR_ARG;
  if (c->mode != TW_MODE_F32 && c->mode != TW_MODE_BF16) return TW_ERR_ARG;
  if (m->pred_kind == TW_PRED_STATELESS) {
    if (m->P != m->emb_dim) return TW_ERR_ARG;
  } else if (m->pred_kind == TW_PRED_LSTM) {
    if (m->lstm_layers < 1 || m->lstm_layers > kMaxLayers || m->lstm_hidden < 1) return TW_ERR_ARG;
    if (m->P != m->lstm_hidden) return TW_ERR_ARG;
    if (!m->host_lstm_W_ih || !m->host_lstm_W_hh || !m->host_lstm_b) return TW_ERR_ARG;
    for (int l = 0; l < m->lstm_layers; ++l)
      if (!m->host_lstm_W_ih[l] || !m->host_lstm_W_hh[l] || !m->host_lstm_b[l]) return TW_ERR_ARG;
  } else {
    return TW_ERR_ARG;
  }
  if ((long long)c->max_batch * c->max_T * (long long)m->J >= (1ll << 40)) return TW_ERR_ARG;
  if ((long long)c->max_batch * c->max_T >= (1ll << 31)) return TW_ERR_ARG;
  tw_handle* h = new (std::nothrow) tw_handle();
  if (!h) return TW_ERR_ALLOC;
  int s = init_impl(h, m, c);
  if (s != TW_OK) { tw_destroy(h); return s; }
  // two lanes of half the batch each (tw_decode overlaps them); a failure here only disables lanes
  if (c->max_batch >= 256) {
    tw_config half = *c;
    half.max_batch = (c->max_batch + 1) / 2;
    for (int k = 0; k < 2; ++k) {
      tw_handle* l = new (std::nothrow) tw_handle();
      if (!l) break;
      l->is_lane = true;
      if (init_impl(l, m, &half) != TW_OK) { tw_destroy(l); break; }
      h->lane[k] = l;
    }
    if (!h->lane[1] && h->lane[0]) { tw_destroy(h->lane[0]); h->lane[0] = nullptr; }
  }
  *out = h;
  return TW_OK;
}

int tw_destroy(tw_handle* h) {
  if (!h) return TW_ERR_ARG;
  for (int k = 0; k < 2; ++k)
    if (h->lane[k]) { tw_destroy(h->lane[k]); h->lane[k] = nullptr; }
  cudaDeviceSynchronize();
  for (void* p : h->dev_allocs) cudaFree(p);
  for (cudaEvent_t e : h->events) cudaEventDestroy(e);
  if (h->graph_exec) cudaGraphExecDestroy(h->graph_exec);
  if (h->ev_order) cudaEventDestroy(h->ev_order);
  if (h->ev_poll) cudaEventDestroy(h->ev_poll);
  for (cudaEvent_t e : h->ev_chunk) if (e) cudaEventDestroy(e);
  if (h->copy_stream) cudaStreamDestroy(h->copy_stream);
  if (h->ev_fork) cudaEventDestroy(h->ev_fork);
  if (h->ev_join) cudaEventDestroy(h->ev_join);
  if (h->aux_stream) cudaStreamDestroy(h->aux_stream);
  if (h->own_stream) cudaStreamDestroy(h->own_stream);
  if (h->host_flag) cudaFreeHost(h->host_flag);
  delete h;
  return TW_OK;
}

int tw_max_tokens(const tw_handle* h) { return h ? h->U_cap : -1; }
int tw_last_cuda_error(const tw_handle* h) { return h ? h->last_cuda : 0; }

int tw_set_fused(tw_handle* h, int on) {
  if (!h) return TW_ERR_ARG;
  if (on && !h->bf.fused_ok) return TW_ERR_STATE;
  h->bf.fused_on = on != 0;
  return TW_OK;
}

int tw_set_monotonic(tw_handle* h, int on) {
  if (!h) return TW_ERR_ARG;
  if (h->stream_B > 0) return TW_ERR_STATE;        // not in the middle of a streaming session
  tw_handle* all[3] = {h, h->lane[0], h->lane[1]};
  for (tw_handle* x : all) {
    if (!x) continue;
    x->hs.mono = x->hs_fused.mono = on ? 1 : 0;
    // a captured step graph holds the kernels' arguments by value: capture again with the new setting
    if (x->graph_exec) { cudaGraphExecDestroy(x->graph_exec); x->graph_exec = nullptr; }
  }
  return TW_OK;
}

int tw_set_inline_gather(tw_handle* h, int on) {
  if (!h) return TW_ERR_ARG;
  if (h->stream_B > 0) return TW_ERR_STATE;
  tw_handle* all[3] = {h, h->lane[0], h->lane[1]};
  for (tw_handle* x : all) {
    if (!x) continue;
    // the operand rows' addresses were filled in by tw_init whenever the fused decode path with an LSTM predictor exists
    const bool can = x->mode == TW_MODE_BF16 && x->bf.fused_ok && x->hs_fused.defer_rows && x->pred_kind != TW_PRED_STATELESS;
    if (on && !can) return TW_ERR_STATE;
    if (can) x->hs_fused.inline_gather = on ? 1 : 0;
    if (x->graph_exec) { cudaGraphExecDestroy(x->graph_exec); x->graph_exec = nullptr; }   // captured arguments are by value
  }
  return TW_OK;
}

int tw_set_blank_threshold(tw_handle* h, float threshold) {
  if (!h) return TW_ERR_ARG;
  if (!(threshold >= 0.f && threshold <= 1.f)) return TW_ERR_ARG;
  if (!h->hat || h->stream_B > 0) return TW_ERR_STATE;
  tw_handle* all[3] = {h, h->lane[0], h->lane[1]};
  for (tw_handle* x : all) {
    if (!x) continue;
    x->log_tau = threshold > 0.f ? logf(threshold) : -INFINITY;
    if (x->graph_exec) { cudaGraphExecDestroy(x->graph_exec); x->graph_exec = nullptr; }   // captured arguments are by value
  }
  return TW_OK;
}

int tw_set_lanes(tw_handle* h, int on) {
  if (!h) return TW_ERR_ARG;
  h->lanes_on = on != 0;
  return TW_OK;
}

int tw_set_graph(tw_handle* h, int on) {
  if (!h) return TW_ERR_ARG;
  h->graph_on = on != 0;
  return TW_OK;
}

int tw_set_profiling(tw_handle* h, int on) {
  if (!h) return TW_ERR_ARG;
  h->profiling = on != 0;
  h->stats.ns_joiner = h->stats.ns_scan = h->stats.joiner_launches = 0;   // the stage calls add to these while it is on
  return TW_OK;
}

int tw_get_stats(const tw_handle* h, tw_stats* out) {
  if (!h || !out) return TW_ERR_ARG;
  *out = h->stats;
  out->fused_clusters = h->bf.fused_ok ? h->bf.max_clusters : 0;
  out->fused_on = (h->mode == TW_MODE_BF16 && h->bf.fused_on) ? 1 : 0;
  return TW_OK;
}

const char* tw_strerror(int s) {
  switch (s) {
    case TW_OK: return "ok";
    case TW_ERR_ARG: return "invalid argument";
    case TW_ERR_ALLOC: return "allocation failed";
    case TW_ERR_CUDA: return "CUDA call failed";
    case TW_ERR_LIMIT: return "safety cap hit (inner iterations per segment or token capacity)";
    case TW_ERR_STATE: return "call not valid for this handle";
    case TW_ERR_TIMEOUT: return "bounded device-side wait gave up";
    default: return "unknown status";
  }
}

}  // extern "C"

namespace {
enum Stage { kStStart = -1, kStPrologue = 0, kStPredictor, kStJoiner, kStScan, kStHyp, kStCount };

// Profiling: records an event that closes stage `stage` (the time since the previous mark is its).
void mark(tw_handle* h, int stage, cudaStream_t st) {
  if (!h->profiling) return;
  const size_t i = h->marks.size();
  if (i >= h->events.size()) {
    cudaEvent_t e;
    if (cudaEventCreate(&e) != cudaSuccess) { h->profiling = false; return; }
    h->events.push_back(e);
  }
  cudaEventRecord(h->events[i], st);
  h->marks.push_back(stage);
}

}  // namespace

#include "tw_api_stages.inc"
#include "tw_api_decode.inc"
#include "tw_api_stream.inc"
