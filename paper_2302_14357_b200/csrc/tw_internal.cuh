// Internal declarations shared by the translation units of libtw.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <math.h>

#include "../../include/tw.h"

namespace tw {

constexpr int kMaxBeam = TW_MAX_BEAM;
constexpr int kMaxSeg = TW_MAX_SEGMENT;
constexpr int kMaxLayers = 4;

// ---------------------------------------------------------------------------------------------
// Programmatic dependent launch.  The kernels of a decode step run back to back on one stream, each
// reading what the previous one wrote.  Launched with launch_pdl, a kernel may be scheduled while its
// predecessor is still running (once every CTA of the predecessor has called pdl_trigger or exited), so
// its set-up (barriers, tensor memory, tensor-map prefetch) overlaps the predecessor's tail.  The rules
// every kernel launched this way follows: (1) every thread calls pdl_wait before it reads or writes
// global memory that another kernel of the stream writes or reads, and every CTA calls it on every path
// (a kernel that finished without waiting would release ITS successor too early); (2) nothing before
// pdl_wait has a side effect outside the CTA.  pdl_wait returns at once in a kernel launched normally.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Host-side switch of the calling thread: while false, launch_pdl launches normally.  Two decoders that share
// the GPU on two streams keep it off: an early-scheduled CTA that only waits would hold an SM the other
// stream's kernels could use.
inline thread_local bool g_pdl_on = true;
struct PdlScope {
  bool saved;
  explicit PdlScope(bool on) : saved(g_pdl_on) { g_pdl_on = on; }
  ~PdlScope() { g_pdl_on = saved; }
};

template <typename... P, typename... A>
inline cudaError_t launch_pdl(void (*kern)(P...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, A&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = g_pdl_on ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<P>(args)...);
}

// ---------------------------------------------------------------------------------------------
// numerics helpers (accurate libm versions: the fp32 mode must track an fp64 reference to ~1e-6)
__device__ __forceinline__ float logaddexp_f(float a, float b) {
  if (a == -INFINITY) return b;
  if (b == -INFINITY) return a;
  float m = fmaxf(a, b);
  return m + log1pf(expf(-fabsf(a - b)));
}
__device__ __forceinline__ double logaddexp_d(double a, double b) {
  if (a == -INFINITY) return b;
  if (b == -INFINITY) return a;
  double m = fmax(a, b);
  return m + log1p(exp(-fabs(a - b)));
}

// ---------------------------------------------------------------------------------------------
// SIMT fp32 GEMM  C[m, n] = sum_k A[m, k] * B[n, k] (+ second operand pair) (+ bias[n])
struct GemmOperand {
  const float* A;     // rows of length K; row m starts at A + (idx ? idx[m] : m) * ldA
  const int* idx;     // optional row gather
  long long ldA;
  const float* B;     // [N, K] row-major, leading dimension ldB
  long long ldB;
  int K;
};

struct GemmOut {
  float* C;           // row m written at C + (oidx ? oidx[m] : m) * ldC
  const int* oidx;
  long long ldC;
  const float* bias;  // optional [N]
};

// M may come from device memory (M_dev != nullptr): CTAs beyond it exit.
void launch_gemm_f32(const GemmOperand& op1, const GemmOperand& op2, const GemmOut& out,
                     const int* M_dev, int M_max, int N, cudaStream_t st);

// Joiner rows: hypothesis row r covers frames E[row_e0[r] + t], t < row_slen[r], and the projected
// predictor output Pp[row_p[r]].
struct JoinerRows {
  const float* E;        // [*, J]
  const int* row_e0;     // [R] first frame row of each hypothesis row
  const float* Pp;       // [*, J]
  const int* row_p;      // [R] row into Pp (nullptr: identity)
  const int* row_slen;   // [R] valid frames (nullptr: S)
  const int* R_dev;      // device row count (nullptr: use R_max)
  int R_max, S, J, V;
  int act;               // TW_ACT_TANH / TW_ACT_RELU
  // Factorised output (TW_NORM_HAT): p(blank) = sigmoid(z_blank), the rest shared out by a softmax over the other
  // tokens; a (row, frame) with log p(blank) > log_tau keeps its blank probability only (blank thresholding) and
  // is counted in *skipped.  hat == 0: plain softmax, the two other fields are not read.
  int hat = 0;
  float log_tau = 0.f;
  unsigned long long* skipped = nullptr;
};
// z[(r,t), k] = sum_j tanh(E[e0[r]+t, j] + Pp[p[r], j]) * W_out[k, j] + b_out[k]; rows of padding
// frames (t >= slen) are left untouched.
void launch_joiner_f32(const JoinerRows& rows, const float* W_out, const float* b_out, float* z,
                       cudaStream_t st);
// in place: z[(r,t), :] -> log softmax; padding frames get (0 at blank, -inf elsewhere)
void launch_log_softmax(const JoinerRows& rows, int blank, float* z, cudaStream_t st);
// Per-row candidates of ChooseNBestExpansions: the row's best N non-blank tokens, best first
// (score descending, then token ascending).  v, k are [R][kMaxBeam]; n[r] is how many are valid.
struct CandOut {
  float* v; int* k; int* n; int N;
};
// Eq. 3-7 from materialised log J; ldnb may be nullptr when only the candidates are wanted, and
// cand.n may be nullptr when they are not
void launch_expand_f32(const float* logp, const float* ld_old, const int* row_slen, const int* R_dev,
                       int R_max, int S, int V, int blank, float* ldphi, float* ldnb, float* la,
                       double* ldphi_d, double* la_d, const CandOut& cand,
                       cudaStream_t st);   // float64 copies optional
// Softmax + Eq. 3-7 + per-row candidates from RAW logits z [R, S, V] read once into shared memory
// (scan_select.cu).  Every output pointer is optional.
struct ScanSelectArgs {
  const float* z; const float* ld_old; const int* row_slen; const int* R_dev;
  int R_max, S, V, blank;
  float* lse_out;      // [R, S] softmax normalisers: log J(t, k) = z[t, k] - lse[t]
  float *ldphi, *ldnb, *la; double *ldphi_d, *la_d;
  CandOut cand;
  const float* dnb_in = nullptr;   // when set: [R, V] delta_nb values are given and only the selection runs
  int dnb_linear = 0;              // dnb_in holds probabilities (0 = none), candidates are returned as logs
};
bool scan_select_fits(int S, int V);   // the row's S x V logits fit in shared memory
int scan_select_setup();
void launch_scan_select(const ScanSelectArgs& a, bool fast_math, cudaStream_t st);
// helper for the stage entry points: row_e0[r] = row_group[r] * S, row_slen[r] = seg_len[row_group[r]] clamped to
// [0, S]; a row whose group is outside [0, G) becomes an empty row (length 0)
void launch_rows_from_groups(const int* row_group, const int* seg_len, int R, int G, int S, int* row_e0,
                             int* row_slen, cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// Hypothesis state of a batch (structure of arrays in one device workspace).
enum Scalar { kScR = 0, kScNPred = 1, kScActive = 2, kScSteps = 3, kScM = 4, kScCount = 8 };   // kScM = R * S

struct HypState {
  int B, N, S, V, J, U_cap, I_max, blank;
  int capB;      // capacity of list B per utterance = N * I_max
  int capSlot;   // hypothesis slots per utterance = N * (I_max + 1)
  int L, Hd;     // LSTM layers / hidden (0 for the stateless predictor)
  int stateless;
  int empty_row;   // stateless predictor: row of the projected-output table that serves the empty token prefix
  // per utterance [B]
  int *len, *t0, *slen, *nA, *nB, *nTop, *iters, *status, *cursor, *n_new, *calls, *joins;
  int* avail;    // streaming: frames pushed so far (len is the part of them that may be decoded now)
  // list A: [B][kMaxBeam]
  int* A_slot; double* A_ls; double* A_ld;   // A_ld [B][kMaxBeam][S]
  // Monotonic variant (every output consumes a frame): a token emitted at frame t leaves its hypothesis at
  // frame t + 1, so A_ld is filled one entry later and A_done [B][kMaxBeam] holds the mass that has left the
  // segment (emitted at its last frame), which joins delta_phi.  mono == 0: A_done is unused.
  double* A_done; int mono;
  // defer_rows != 0: compact_kernel only numbers the rows and builds the predictor's work list; the row tables,
  // row_ld and the clearing of n_new are left to the kernel that completes the new hypotheses' frame
  // distributions, which then runs beside the predictor kernels of the next pass
  int defer_rows;
  // dnb_sel != nullptr: delta_nb [R][V] as plain probability ratios (0: no candidate); hyp_step_kernel then picks
  // every row's N best tokens itself instead of reading cand_v / cand_k / cand_n
  const float* dnb_sel;
  // with dnb_sel: optional [R][V / 32] largest value of every 32-column chunk of a row, written by the kernel that wrote
  // delta_nb; the selection then reads these first and only the few chunks that can hold one of the N best after them
  const float* dnb_max;
  // list B of Algorithm 1 (hypotheses finished for this segment): [B][capB]
  int* B_slot; double* B_ls; unsigned long long* B_hash; int* B_len;
  int* B_top;    // [B][kMaxBeam] indices into list B of its best entries, best first
  int* carry;    // [B][kMaxBeam] slots held by hypotheses carried over from earlier segments
  // hypothesis slots: [B][capSlot]
  int* slot_len; unsigned long long* slot_hash; int* slot_tok;  // slot_tok [..][U_cap]
  float* slot_hc;   // [B*capSlot][L][2][Hd]   (LSTM predictor only)
  float* slot_Pp;   // [B*capSlot][J]          (LSTM predictor only)
  // new hypotheses of the current step, per utterance: [B][kMaxBeam] (global slot ids)
  int *new_slot, *new_par, *new_tok, *new_row;   // new_row: joiner row of the parent
  // compacted rows of the current step: [B*N]
  int *row_b, *row_e0, *row_p, *row_slen; float* row_ld;   // row_ld [R][S]
  int *row_off, *new_off;     // [B] first row / first work-list entry of each utterance
  // compacted predictor work list: [B*N]
  int *pw_new, *pw_par, *pw_tok;
  int* scalars;           // [kScCount] device scalars
  long long* rows_total;  // [2]: sum over steps of rows R, and of rows x their segment's frames
  // stage outputs of the current step
  float *ldphi, *la, *ldnb, *logp;
  float* lse;   // [R][S]; when set, logp holds raw logits and log J = logp - lse
  double *ldphi_d, *la_d;   // float64 copies of ldphi / la (nullptr: use the float32 ones)
  float* cand_v; int* cand_k; int* cand_n;   // per-row expansion candidates [R][kMaxBeam], [R]
  // InitPredictor result (LSTM only): [L][2][Hd], [J]
  const float* init_hc; const float* init_Pp;
  // inline_gather != 0 (fused bf16 decode with an LSTM predictor): hyp_step_kernel appends its new hypotheses to
  // the predictor's work list itself (entries claimed by an atomic add on scalars[kScNPred], which the joiner
  // kernel of the same pass cleared after the predictor kernels had read it) and writes their parents' h as bf16
  // into the gate GEMMs' operand rows xg_dst[l] (row pitch xg_ld[l], column offset xg_off[l], in elements), so
  // that no gather kernel runs between it and the first gate GEMM.  The order of the list's entries varies
  // from run to run; no result depends on it (every entry is computed on its own).
  int inline_gather;
  void* xg_dst[kMaxLayers]; int xg_ld[kMaxLayers]; int xg_off[kMaxLayers];
  // With inline_gather: the first gate GEMM adds a row of this table per new hypothesis ([V] rows of pf_row_bytes, a
  // table far larger than L2) and every layer reads the parent's cell state; hyp_step_kernel, which is the first to
  // know tokens and parents, asks for both in L2 so that the GEMM's epilogue threads do not each wait on DRAM.
  const char* pf_table; int pf_row_bytes;
};

void launch_hyp_init(const HypState& hs, const int* lengths, int B, int T, cudaStream_t st);
void launch_hyp_step(const HypState& hs, int B, cudaStream_t st);
void launch_compact(const HypState& hs, int B, int T, cudaStream_t st);
// Streaming.  stream_rows: destination row in E of every frame of a pushed chunk [B, Tc] (frames past
// chunk_lens[b] or past max_T go to `dump_row`); stream_advance: avail += chunk_lens (clamped to max_T,
// flagging TW_ERR_LIMIT), len = whole segments of avail (all of avail when closing), and a turn-over
// for every utterance that was waiting for frames.
void launch_stream_rows(const HypState& hs, const int* chunk_lens, int B, int Tc, int max_T, int dump_row,
                        int* oidx, cudaStream_t st);
void launch_stream_advance(const HypState& hs, const int* chunk_lens, int B, int max_T, int closing,
                           cudaStream_t st);
void launch_finish(const HypState& hs, int B, int* out_tokens, int* out_lens, double* out_scores,
                   int* out_status, cudaStream_t st);

// LSTM pointwise: gates [n, 4Hd] + c of row (idx_in ? idx_in[i] : i) of hc_in -> (h, c) of layer l in row
// (idx_out ? idx_out[i] : i) of hc_out; state rows are [L][2][Hd]
void launch_lstm_pointwise(const float* gates, const int* idx_out, const int* idx_in, const int* n_dev,
                           int n_max, const float* hc_in, float* hc_out, int L, int l, int Hd, cudaStream_t st);

}  // namespace tw
