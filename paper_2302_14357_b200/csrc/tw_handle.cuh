// The decoder handle behind the C ABI.
#pragma once
#include <vector>

#include "bf16_path.cuh"
#include "tw_internal.cuh"

struct tw_handle {
  // model dimensions and search parameters
  int D_enc = 0, P = 0, J = 0, V = 0, blank = 0;
  int pred_kind = 0, emb_dim = 0, L = 0, Hd = 0, joiner_act = 0;
  int hat = 0;                // TW_NORM_HAT model: factorised output
  float log_tau = 0.f;        // log of the blank threshold (0: nothing is skipped)
  int dtype = 0;              // element type of the caller's weights and encoder frames (TW_F32 / TW_BF16)
  size_t esize = 4;           // its size in bytes
  float* enc_f32 = nullptr;   // TW_MODE_F32 with bf16 frames: their float32 copy [max_batch * max_T, D_enc]
  int N = 0, S = 0, mode = 0, max_batch = 0, max_T = 0, I_max = 0, U_cap = 0;
  int R_max = 0;

  // fp32 weights on the device
  float *W_e = nullptr, *W_p = nullptr, *W_out = nullptr, *b_out = nullptr, *emb = nullptr;
  float *W_ih[tw::kMaxLayers] = {}, *W_hh[tw::kMaxLayers] = {}, *b_l[tw::kMaxLayers] = {};
  float* PpTab = nullptr;     // stateless predictor: W_p emb[k] for every token k, [V, J]
  float* init_hc = nullptr;   // InitPredictor state [L][2][Hd]
  float* init_Pp = nullptr;   // and its projected output [J]

  tw::HypState hs{};
  tw::HypState hs_fused{};    // same arrays, but log J is not materialised (fused joiner path)
  float* E = nullptr;         // projected encoder frames [max_batch * max_T, J]
  float* gates = nullptr;     // LSTM gate pre-activations [R_max, 4 Hd]
  int *stage_e0 = nullptr, *stage_slen = nullptr;   // [R_max] scratch of the stage entry points
  int* stream_oidx = nullptr;   // [max_batch * max_T] destination rows of a pushed chunk's frames
  int* zero_len = nullptr;      // [max_batch] zeros
  int stream_B = 0;             // utterances of the open streaming session (0: none)

  // TW_MODE_BF16: bf16 copies of the GEMM operands with their tensor maps
  struct {
    tw::Bf16Mat W_e, W_out, W_p, W_cat[tw::kMaxLayers];   // W_cat[0] = W_hh[0] [4Hd, Hd]; W_cat[l>0] = [W_ih[l] | W_hh[l]] [4Hd, 2Hd]
    tw::Bf16Mat enc;                                      // [max_batch * max_T, D_enc]
    tw::Bf16Mat A_join;                                   // [R_max * S, J]  tanh(E + Pp)
    tw::Bf16Mat X[tw::kMaxLayers];                        // LSTM layer inputs: [R_max, Hd] (layer 0: parent h) or [R_max, 2Hd]
    tw::Bf16Mat Htop;                                     // [R_max, Hd]
    float* bias_perm[tw::kMaxLayers] = {};   // LSTM biases in the interleaved gate order (layers > 0)
    float* EmbProj = nullptr;   // [V, 4Hd] = emb W_ih[0]^T + b[0]: layer 0's input half, one row per token
    int* err = nullptr;                                   // device error word of the bounded waits
    // fused joiner + softmax + Eq. 3-7 + selection (logits stay in tensor memory)
    bool fused_ok = false, fused_on = false, no_max = false;
    float zbound = 0.f;                                   // bound of |logit| behind no_max
    int CL = 0, max_clusters = 0;
    // The fused kernel splits the vocabulary into 256-column CTAs.  A vocabulary that is not a multiple of 256 is
    // padded for it: Vp columns, the added rows of W_out zero and their bias -1e30 (probability 0, never a
    // candidate).  Vp == V: the padded objects below are the plain ones.
    int Vp = 0;
    tw::Bf16Mat W_out_pad;
    float* bias_pad = nullptr;
    float* ldnb_pad = nullptr;                            // [R_max, Vp]
    float* dmax = nullptr;                                // [R_max, Vp / 32] chunk maxima of delta_nb (fused decode path)
    tw::Bf16Mat A_tiled;                                  // A operand in the fused kernel's tile layout
    float* lse = nullptr;                                 // [R_max, S]
  } bf;

  // staging of tw_decode_host (allocated on first use)
  char* st_enc = nullptr; int* st_len = nullptr; int* st_tok = nullptr; int* st_lens = nullptr;
  // tw_decode_host uploads the frames in a few time chunks on copy_stream and decodes chunk k (as a streaming
  // session) while chunk k + 1 is still on its way
  static constexpr int kHostChunks = 2;
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_chunk[kHostChunks] = {nullptr, nullptr};
  int* st_chunk_lens = nullptr;                         // [kHostChunks][max_batch]
  double* st_scores = nullptr; int* st_status = nullptr;

  int* host_flag = nullptr;   // pinned copy of the device scalars

  // The step body (kStepsPerGraph device steps) is captured once per (B, T, joiner path) into a CUDA
  // graph and replayed; it runs on a stream of the handle's own because the caller's may be the legacy
  // default stream, which cannot be captured.
  bool graph_on = true, graph_failed = false;
  cudaStream_t own_stream = nullptr;
  cudaEvent_t ev_order = nullptr;
  cudaGraphExec_t graph_exec = nullptr;
  int graph_B = -1, graph_T = -1, graph_fused = -1, graph_launches = 0;
  cudaEvent_t ev_poll = nullptr;
  // side branch of a decode step: the kernel that completes the new hypotheses' frame distributions and
  // writes the rows' row_ld runs on aux_stream beside the next pass's predictor kernels (fork after the
  // compaction kernel, join before the joiner's operand kernel)
  cudaStream_t aux_stream = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  bool aux_ok = false, aux_pending = false;

  // state of the decode in flight (decode_begin .. decode_end)
  struct Run {
    int B = 0, T = 0;
    int32_t* out_tokens = nullptr; int32_t* out_lens = nullptr; double* out_scores = nullptr; int32_t* out_status = nullptr;
    cudaStream_t st = nullptr;
    bool use_graph = false, active = false;
    long long issued = 0, max_steps = 0;
    int launches = 0;
  } run;

  // two internal decoders for half of max_batch each (see tw_decode); null for small handles
  tw_handle* lane[2] = {nullptr, nullptr};
  bool lanes_on = true, is_lane = false;

  // optional per-stage timing of tw_decode (tw_set_profiling): pooled events and the stage each closes
  bool profiling = false;
  std::vector<cudaEvent_t> events;
  std::vector<int> marks;

  std::vector<void*> dev_allocs;
  tw_stats stats{};
  int last_cuda = 0;
};

namespace tw {
// stages shared by tw_decode and the stage entry points
void enqueue_joiner_logits(tw_handle* h, const JoinerRows& rows, float* logp, cudaStream_t st, int* launches);
// mark_fn (optional) is called with stage 3 after the operand kernel and stage 2 after the fused kernel
typedef void (*StageMarkFn)(tw_handle*, int, cudaStream_t);
int enqueue_joiner_fused(tw_handle* h, const JoinerRows& rows, const float* ld_old, float* ldphi, float* ldnb,
                         float* la, const CandOut& cand, cudaStream_t st, int* launches, StageMarkFn mark_fn = nullptr,
                         bool plain_first = false,    // plain_first: the operand kernel is launched with plain stream ordering
                         int utt_B = 0,               // utt_B > 0: the rows are a decode step's (hs.row_off, hs.nA of utt_B utterances)
                         int* clear_word = nullptr);  // a device word the fused kernel clears (FusedJoinerParams::clear_word)
void enqueue_scan(tw_handle* h, const JoinerRows& rows, const float* ld_old, float* logp, float* ldphi,
                  float* ldnb, float* la, double* ldphi_d, double* la_d, const CandOut& cand, cudaStream_t st,
                  int* launches);
void enqueue_joiner_expand_f32(tw_handle* h, const JoinerRows& rows, const float* ld_old, float* logp,
                               float* ldphi, float* ldnb, float* la, double* ldphi_d, double* la_d,
                               const CandOut& cand, cudaStream_t st, int* launches);
}

