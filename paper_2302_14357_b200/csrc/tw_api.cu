// C ABI of libtw: handle life-cycle, the decode driver and the separately callable stages.
#include <new>
#include <stdio.h>
#include <string.h>

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

int copy_weight(tw_handle* h, float** dst, const float* src, size_t count) {
  TW_TRY(dev_alloc(h, dst, count));
  TW_CUDA(h, cudaMemcpy(*dst, src, count * sizeof(float), cudaMemcpyDeviceToDevice));
  return TW_OK;
}

// One predictor step on plain arrays (see tw_predictor_step).
int enqueue_predictor_plain(tw_handle* h, const int* tokens, const float* state_in, int R,
                            float* state_out, float* out_Pp, cudaStream_t st, int* launches) {
  if (h->pred_kind == TW_PRED_STATELESS) {
    GemmOperand a{h->emb, tokens, h->emb_dim, h->W_p, h->P, h->P};
    GemmOperand none{};
    GemmOut o{out_Pp, nullptr, h->J, nullptr};
    launch_gemm_f32(a, none, o, nullptr, R, h->J, st);
    *launches += 1;
    return TW_OK;
  }
  const int L = h->L, Hd = h->Hd;
  const long long stride = (long long)L * 2 * Hd;
  for (int l = 0; l < L; ++l) {
    GemmOperand x = (l == 0) ? GemmOperand{h->emb, tokens, h->emb_dim, h->W_ih[0], h->emb_dim, h->emb_dim}
                             : GemmOperand{state_out + (long long)(l - 1) * 2 * Hd, nullptr, stride, h->W_ih[l], Hd, Hd};
    GemmOperand r{state_in + (long long)l * 2 * Hd, nullptr, stride, h->W_hh[l], Hd, Hd};
    GemmOut o{h->gates, nullptr, 4 * Hd, h->b_l[l]};
    launch_gemm_f32(x, r, o, nullptr, R, 4 * Hd, st);
    launch_lstm_pointwise_plain(h->gates, state_in, state_out, R, L, l, Hd, st);
    *launches += 2;
  }
  GemmOperand top{state_out + (long long)(L - 1) * 2 * Hd, nullptr, stride, h->W_p, h->P, h->P};
  GemmOperand none{};
  GemmOut o{out_Pp, nullptr, h->J, nullptr};
  launch_gemm_f32(top, none, o, nullptr, R, h->J, st);
  *launches += 1;
  return TW_OK;
}

// UpdatePredictorOutput for the work list the compaction kernel built (new slot, parent slot, token).
void enqueue_predictor_slots(tw_handle* h, cudaStream_t st, int* launches) {
  if (h->pred_kind == TW_PRED_STATELESS) return;   // the joiner reads W_p emb[last token] from a table
  const HypState& hs = h->hs;
  const int L = h->L, Hd = h->Hd;
  const long long stride = (long long)L * 2 * Hd;
  const int* n_dev = hs.scalars + kScNPred;
  for (int l = 0; l < L; ++l) {
    GemmOperand x = (l == 0) ? GemmOperand{h->emb, hs.pw_tok, h->emb_dim, h->W_ih[0], h->emb_dim, h->emb_dim}
                             : GemmOperand{hs.slot_hc + (long long)(l - 1) * 2 * Hd, hs.pw_new, stride, h->W_ih[l], Hd, Hd};
    GemmOperand r{hs.slot_hc + (long long)l * 2 * Hd, hs.pw_par, stride, h->W_hh[l], Hd, Hd};
    GemmOut o{h->gates, nullptr, 4 * Hd, h->b_l[l]};
    launch_gemm_f32(x, r, o, n_dev, h->R_max, 4 * Hd, st);
    launch_lstm_pointwise_slots(h->gates, hs.pw_new, hs.pw_par, n_dev, h->R_max, hs.slot_hc, L, l, Hd, st);
    *launches += 2;
  }
  GemmOperand top{hs.slot_hc + (long long)(L - 1) * 2 * Hd, hs.pw_new, stride, h->W_p, h->P, h->P};
  GemmOperand none{};
  GemmOut o{hs.slot_Pp, hs.pw_new, h->J, nullptr};
  launch_gemm_f32(top, none, o, n_dev, h->R_max, h->J, st);
  *launches += 1;
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
  const size_t nb = (size_t)B, nslot = nb * hs.capSlot, nB = nb * hs.capB, R = (size_t)h->R_max;
  int** per_utt[] = {&hs.len, &hs.t0, &hs.slen, &hs.nA, &hs.nB, &hs.nTop, &hs.iters, &hs.status,
                     &hs.cursor, &hs.n_new, &hs.calls, &hs.joins, &hs.row_off};
  for (int** p : per_utt) TW_TRY(dev_alloc(h, p, nb));
  TW_TRY(dev_alloc(h, &hs.A_slot, nb * kMaxBeam));
  TW_TRY(dev_alloc(h, &hs.A_ls, nb * kMaxBeam));
  TW_TRY(dev_alloc(h, &hs.A_ld, nb * kMaxBeam * S));
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
  int** per_row[] = {&hs.row_b, &hs.row_e0, &hs.row_p, &hs.row_slen, &hs.pw_new, &hs.pw_par, &hs.pw_tok,
                     &h->stage_e0, &h->stage_slen};
  for (int** p : per_row) TW_TRY(dev_alloc(h, p, R));
  TW_TRY(dev_alloc(h, &hs.row_ld, R * S));
  TW_TRY(dev_alloc(h, &hs.scalars, (size_t)kScCount));
  TW_TRY(dev_alloc(h, &hs.rows_total, (size_t)2));
  TW_TRY(dev_alloc(h, &hs.ldphi, R));
  TW_TRY(dev_alloc(h, &hs.la, R * S));
  TW_TRY(dev_alloc(h, &hs.ldphi_d, R));
  TW_TRY(dev_alloc(h, &hs.la_d, R * S));
  TW_TRY(dev_alloc(h, &hs.ldnb, R * h->V));
  TW_TRY(dev_alloc(h, &hs.logp, R * S * h->V));
  TW_TRY(dev_alloc(h, &h->E, nb * h->max_T * h->J));
  TW_CUDA(h, cudaMemset(hs.scalars, 0, kScCount * sizeof(int)));
  TW_CUDA(h, cudaMemset(hs.rows_total, 0, 2 * sizeof(long long)));
  TW_CUDA(h, cudaHostAlloc((void**)&h->host_flag, (kScCount + 4) * sizeof(long long), cudaHostAllocDefault));
  return TW_OK;
}

int init_impl(tw_handle* h, const tw_model* m, const tw_config* c) {
  h->D_enc = m->D_enc; h->P = m->P; h->J = m->J; h->V = m->V; h->blank = m->blank;
  h->pred_kind = m->pred_kind; h->emb_dim = m->emb_dim;
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

  int launches = 0;
  if (h->pred_kind == TW_PRED_STATELESS) {
    // W_p emb[k] for every token: the joiner rows index this table by their last token
    TW_TRY(dev_alloc(h, &h->PpTab, (size_t)h->V * h->J));
    GemmOperand a{h->emb, nullptr, h->emb_dim, h->W_p, h->P, h->P};
    GemmOperand none{};
    GemmOut o{h->PpTab, nullptr, h->J, nullptr};
    launch_gemm_f32(a, none, o, nullptr, h->V, h->J, 0);
  } else {
    // InitPredictor(): one step on the blank token from an all-zero state
    const size_t nhc = (size_t)h->L * 2 * h->Hd;
    float* zero = nullptr; int* tok = nullptr;
    TW_TRY(dev_alloc(h, &zero, nhc));
    TW_TRY(dev_alloc(h, &tok, (size_t)1));
    TW_TRY(dev_alloc(h, &h->init_hc, nhc));
    TW_TRY(dev_alloc(h, &h->init_Pp, (size_t)h->J));
    TW_CUDA(h, cudaMemset(zero, 0, nhc * sizeof(float)));
    TW_CUDA(h, cudaMemcpy(tok, &h->blank, sizeof(int), cudaMemcpyHostToDevice));
    TW_TRY(enqueue_predictor_plain(h, tok, zero, 1, h->init_hc, h->init_Pp, 0, &launches));
    h->hs.init_hc = h->init_hc; h->hs.init_Pp = h->init_Pp;
  }
  TW_CUDA(h, cudaGetLastError());
  TW_CUDA(h, cudaDeviceSynchronize());
  return TW_OK;
}

}  // namespace

namespace tw {
void enqueue_joiner_expand_f32(tw_handle* h, const JoinerRows& rows, const float* ld_old, float* logp,
                               float* ldphi, float* ldnb, float* la, double* ldphi_d, double* la_d,
                               cudaStream_t st, int* launches) {
  launch_joiner_f32(rows, h->W_out, h->b_out, logp, st);
  launch_log_softmax(rows, h->blank, logp, st);
  launch_expand_f32(logp, ld_old, rows.row_slen, rows.R_dev, rows.R_max, rows.S, rows.V, h->blank, ldphi,
                    ldnb, la, ldphi_d, la_d, st);
  *launches += 3;
}
}  // namespace tw

extern "C" {

int tw_init(const tw_model* m, const tw_config* c, tw_handle** out) {
  if (out) *out = nullptr;
  if (!m || !c || !out) return TW_ERR_ARG;
  if (!m->W_e || !m->W_p || !m->W_out || !m->b_out || !m->emb) return TW_ERR_ARG;
  if (m->D_enc < 1 || m->P < 1 || m->J < 1 || m->V < 2 || m->emb_dim < 1) return TW_ERR_ARG;
  if (m->blank < 0 || m->blank >= m->V) return TW_ERR_ARG;
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
  *out = h;
  return TW_OK;
}

int tw_destroy(tw_handle* h) {
  if (!h) return TW_ERR_ARG;
  cudaDeviceSynchronize();
  for (void* p : h->dev_allocs) cudaFree(p);
  for (cudaEvent_t e : h->events) cudaEventDestroy(e);
  if (h->host_flag) cudaFreeHost(h->host_flag);
  delete h;
  return TW_OK;
}

int tw_max_tokens(const tw_handle* h) { return h ? h->U_cap : -1; }
int tw_last_cuda_error(const tw_handle* h) { return h ? h->last_cuda : 0; }

int tw_set_profiling(tw_handle* h, int on) {
  if (!h) return TW_ERR_ARG;
  h->profiling = on != 0;
  return TW_OK;
}

int tw_get_stats(const tw_handle* h, tw_stats* out) {
  if (!h || !out) return TW_ERR_ARG;
  *out = h->stats;
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

#include "tw_api_stages.inc"
#include "tw_api_decode.inc"
