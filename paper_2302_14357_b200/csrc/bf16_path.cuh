// TW_MODE_BF16: bf16 operands on the tcgen05 tensor cores, fp32 accumulation and fp32 epilogues.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>

#include "tw_internal.cuh"

namespace tw {

// LSTM cell epilogue of a gate GEMM whose output columns are interleaved by unit (column 4 j + g is
// gate g of hidden unit j, gates in the order input, forget, cell, output):
//   c' = sigma(f) c + sigma(i) tanh(g),  h' = sigma(o) tanh(c')
// c is read from state row (idx_in ? idx_in[m] : m) of hc_in, (h', c') are written to state row
// (idx_out ? idx_out[m] : m) of hc_out (rows are [L][2][Hd]), and h' also goes, as bf16, to row m of
// xnext (the next GEMM's A operand).
struct LstmEpi {
  const float* hc_in; const int* idx_in; float* hc_out; const int* idx_out;
  int L, l, Hd;
  __nv_bfloat16* xnext; long long ld_xnext;
};

struct GemmBf16Params {
  const int* M_dev;   // device row count (nullptr: use M); CTAs beyond it exit
  int M, N, K;        // M is the maximum when M_dev is given
  float* C;           // row m written at C + (oidx ? oidx[m] : m) * ldC
  const int* oidx;
  long long ldC;
  const float* bias;  // optional [N]
  int* err;           // device error word, raised by a wait that gave up
  const float* addend = nullptr;   // optional: row m also gets addend[(add_idx ? add_idx[m] : m) * ld_add + n]
  const int* add_idx = nullptr;
  long long ld_add = 0;
  int epi = 0;        // 0: store C (+ bias, + addend); 1: LSTM cell (C is not written)
  int m_early = 0;    // 1: *M_dev was written before the kernel launched ahead of this one began (not by that kernel):
                      // it is read during the set-up, ahead of the wait for that kernel
  LstmEpi lstm = {};
};

// 2-D bf16 tensor map over a row-major [rows, K] matrix, box = 64 x box_rows, 128-byte swizzle.
// Requires K % 8 == 0 and a 16-byte aligned base.
int make_tmap_bf16(CUtensorMap* out, const void* base, uint64_t rows, uint64_t K, uint32_t box_rows);
int gemm_bf16_setup();
// tmB128 / tmB256: maps of the same B matrix with 128- and 256-row boxes
// tmB64 (optional): a map with 64-row boxes, used for small problems without an epilogue fusion
void launch_gemm_bf16(const CUtensorMap& tmA, const CUtensorMap& tmB128, const CUtensorMap& tmB256,
                      const GemmBf16Params& p, cudaStream_t st, const CUtensorMap* tmB64 = nullptr);

// LSTM gate GEMM (epi == 1) as a single wave of one tile per CTA when 128 x 256 tiles would need a second,
// nearly empty wave; returns false (nothing launched) when the shape does not call for it.
// tmB64 / tmB32: maps of B with 64- and 32-row boxes
bool launch_gemm_lstm_wide(const CUtensorMap& tmA, const CUtensorMap& tmB64, const CUtensorMap& tmB32,
                           const GemmBf16Params& p, cudaStream_t st);

// A bf16 matrix with its tensor maps
struct Bf16Mat {
  __nv_bfloat16* ptr = nullptr;
  long long rows = 0, K = 0;
  CUtensorMap as_A;            // box 128 rows
  CUtensorMap as_B128, as_B256;
  CUtensorMap as_B64, as_B32;
};

// elementwise helpers ---------------------------------------------------------------------------
void launch_f32_to_bf16(const float* src, __nv_bfloat16* dst, long long n, cudaStream_t st);
void launch_bf16_to_f32(const __nv_bfloat16* src, float* dst, long long n, cudaStream_t st);   // exact
// dst[r, 0:K1] = src1 row (idx1 ? idx1[r] : r), dst[r, K1:K1+K2] = src2 row (idx2 ? idx2[r] : r)
void launch_gather_concat_bf16(const float* src1, const int* idx1, long long ld1, int K1, const float* src2,
                               const int* idx2, long long ld2, int K2, const int* n_dev, int n_max,
                               __nv_bfloat16* dst, cudaStream_t st);
// X[l][r, off_l : off_l + Hd] = bf16(h of layer l in state row (idx ? idx[r] : r)), for every layer at once
// Optional: the kernel first builds the predictor's work list itself.  Entry r is the i-th new hypothesis of
// utterance b, where r = (sum of n_new over the utterances before b) + i; every CTA finds its (b, i) by a scan
// of n_new (B values), the CTAs of layer 0 write entry r of pw_new / pw_par / pw_tok, and CTA (0, 0) writes the
// list's length to n_out.  B == 0: the list exists already (idx, n_dev).
struct WorkListBuild {
  int B;
  const int* n_new; const int* new_slot; const int* new_par; const int* new_tok;   // [B], [B][kMaxBeam] x 3
  int* pw_new; int* pw_par; int* pw_tok; int* n_out;
};
struct GatherParents {
  const float* hc; const int* idx; long long stride;   // state rows [L][2][Hd]
  int L, Hd;
  __nv_bfloat16* dst[kMaxLayers]; int ld[kMaxLayers]; int off[kMaxLayers];
  WorkListBuild wl;
};
void launch_gather_parents_bf16(const GatherParents& g, const int* n_dev, int n_max, cudaStream_t st);
// dst[r, c] = src[r, perm[c]]  (fp32, rows x cols)
void launch_permute_cols_f32(const float* src, const int* perm, long long rows, int cols, float* dst, cudaStream_t st);
// joiner A operand: A[(r, t), j] = tanh(E[e0[r]+t, j] + Pp[p[r], j]) as bf16; zero rows for padding frames
void launch_joiner_A_bf16(const JoinerRows& rows, __nv_bfloat16* A, cudaStream_t st);


// ---- fused joiner + softmax + Eq. 3-7 + candidate selection (fused_joiner.cu) ------------------
struct FusedJoinerParams {
  const int* R_dev; int R_max;       // hypothesis rows (device count optional; written before the operand kernel ahead of this
                                     // one was launched, and not by it: the kernel reads it ahead of its wait)
  int S, V, K, blank, CL;            // CL = V / 256 CTAs per cluster; K = J
  int no_max;                        // logits are bounded by zbound (at most 40): softmax sums need no maximum search
  float zbound;                      // max_k (|W_out[k, :]|_1 + |b_out[k]|) >= |z| (tanh joiner); used when no_max
  const float* bias;                 // b_out [V]
  const float* ld_old;               // [R][S]
  const int* row_slen;               // [R] (nullptr: S)
  float* ldphi; float* la; float* lse;   // [R], [R][S], [R][S]
  float* ldnb;                       // [R][V] delta_nb as a probability ratio, NOT its log (0 at the blank column)
  float* dmax;                       // optional [R][V / 32]: the largest delta_nb of every 32-column chunk of every row
                                     // (written by the instances that sum over frames with shuffles: fused_joiner_writes_maxima)
  int* err;
  int hat;                           // factorised output (JoinerRows::hat); log2_tau = log2 of the blank threshold
  float log2_tau;
  unsigned long long* skipped;       // optional counter of the (row, frame) pairs blank thresholding left out
  int* clear_word;                   // optional: one device word the kernel sets to 0 once its predecessors have finished
  int early_w;                       // 1: the W_out tiles of the first ring stages are asked for ahead of the wait for the operand kernel
};
bool fused_joiner_eligible(int S, int V, int J);
bool fused_joiner_specialised(int S);
bool fused_joiner_writes_maxima(int S);   // the instance for this segment size fills FusedJoinerParams::dmax   // a kernel instance with this segment size compiled in exists
long long fused_joiner_A_rows(int R_max, int S);      // rows of the tile-layout A operand
int fused_joiner_setup(int CL, int S, int* max_clusters);
// max_k (sum_j |W_out[k, j]| + |b_out[k]|): bound of |z| since |tanh| <= 1; written to *out (device)
void launch_logit_bound(const __nv_bfloat16* W, const float* bias, int V, int J, float* out, cudaStream_t st);
// dst[r, k] = log src[r * ld_src + k] (log 0 = -inf) for r < R, k < V; dst rows have V columns (dst may be src when
// ld_src == V)
void launch_log_rows(const float* src, long long ld_src, float* dst, int R, int V, cudaStream_t st);
// pf_base / pf_bytes (optional): a constant matrix the kernel asks into L2 for its successor (16-byte aligned)
void launch_joiner_A_tiled(const JoinerRows& rows, __nv_bfloat16* A, cudaStream_t st, const void* pf_base = nullptr,
                           long long pf_bytes = 0);
// the same for the rows of a decode step (utterance b's rows are row_off[b] .. + nA[b] - 1, all on one segment)
void launch_joiner_A_tiled_utt(const JoinerRows& rows, const int* row_off, const int* nA, int B, __nv_bfloat16* A,
                               cudaStream_t st);
int launch_fused_joiner(const CUtensorMap& tmA, const CUtensorMap& tmB256, const FusedJoinerParams& p,
                        int max_clusters, cudaStream_t st);
// adds log J(t, parent row, token) to A_ld of the hypotheses created in this step
void launch_survivor_ld(const HypState& hs, int B, int T, const __nv_bfloat16* A, const __nv_bfloat16* W, const float* bias,
                        const float* lse, cudaStream_t st);

}  // namespace tw
