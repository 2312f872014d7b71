/*
 * libtw: token-wise beam search for RNN-T (Algorithm 1 of "A Token-Wise Beam
 * Search Algorithm for RNN-T") on one NVIDIA B200 (sm_100a).
 *
 * C ABI.  Conventions that hold for every call unless a comment says otherwise:
 *   - pointers are DEVICE pointers; a name starting with host_ is a HOST pointer;
 *   - matrices are dense, row-major, float32; int arrays are int32; the model's weights and the encoder frames
 *     are float32 or bfloat16 as tw_model::dtype says (those parameters are `const void*`);
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream);
 *     work is enqueued on it and the call returns without synchronising, except
 *     where stated;
 *   - the caller owns every buffer it passes; the library owns the handle and
 *     its workspace from tw_init to tw_destroy;
 *   - every function returns a tw_status; nothing throws, nothing aborts.  A
 *     failed argument check enqueues no work.
 *   - scores are natural-log probabilities; log 0 is -infinity.
 *   - a handle must not be used from two host threads at once, and two calls on
 *     one handle must not overlap on the GPU (they share its workspace).
 *
 * Notation (paper, Sec. 3): T encoder frames, V vocabulary size including the
 * blank symbol, N beam size, S segment size, J joiner hidden width, P predictor
 * output width, H <= N live hypotheses of an utterance (list A of Algorithm 1),
 * R = sum of H over the utterances of a batch ("rows").
 */
#ifndef TW_H_
#define TW_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tw_handle tw_handle;

typedef enum {
  TW_OK = 0,
  TW_ERR_ARG = 1,    /* null pointer, size out of range, inconsistent shapes           */
  TW_ERR_ALLOC = 2,  /* device or host allocation failed                                */
  TW_ERR_CUDA = 3,   /* a CUDA call failed; tw_last_cuda_error() has the code           */
  TW_ERR_LIMIT = 4,  /* a safety cap was hit (per-utterance: see tw_decode out_status)  */
  TW_ERR_STATE = 5,  /* call not valid for this handle (e.g. stage needs another mode)  */
  TW_ERR_TIMEOUT = 6 /* a bounded device-side wait gave up; results are not valid       */
} tw_status;

enum { TW_MODE_F32 = 0, TW_MODE_BF16 = 1 };   /* arithmetic of the decoder (tw_config::mode)                   */
enum { TW_F32 = 0, TW_BF16 = 1 };             /* element type of the caller's weights and frames (tw_model::dtype) */
enum { TW_PRED_STATELESS = 0, TW_PRED_LSTM = 1 };
enum { TW_ACT_TANH = 0, TW_ACT_RELU = 1 };   /* joiner hidden nonlinearity */
enum { TW_NORM_SOFTMAX = 0, TW_NORM_HAT = 1 }; /* how the joiner's logits become probabilities (tw_model::joiner_norm) */

#define TW_MAX_BEAM 16     /* N <= 16 */
#define TW_MAX_SEGMENT 64  /* S <= 64 */

/*
 * The RNN-T pieces the search calls (Sec. 3.1).
 *   joiner:    z(t,u,.) = W_out . act(W_e h_t + W_p g_u) + b_out,  J = softmax(z); act = tanh, or ReLU
 *              (TW_ACT_RELU is the joiner of the models in Sec. 4.1)
 *   predictor: stateless  g = emb[last token]         (P == emb_dim; empty prefix -> emb[blank])
 *              LSTM       lstm_layers stacked cells, gate order (input, forget, cell, output),
 *                         one bias per layer, g = top layer's h   (P == lstm_hidden);
 *                         InitPredictor(): see pred_init_* below.
 * dtype says what the weight pointers, pred_init_* and every encoder-frame argument of this handle point to:
 * TW_F32 (float32) or TW_BF16 (bfloat16, 2 bytes per element).  It is independent of tw_config::mode: the
 * library keeps float32 copies for its float32 kernels and, in TW_MODE_BF16, bfloat16 copies for the tensor
 * cores (exact if the values are bfloat16-representable, as they are when dtype is TW_BF16).  The per-layer
 * pointer tables are HOST arrays of device pointers.  Nothing passed here is referenced after tw_init returns.
 *
 * InitPredictor() (Sec. 3.2: the predictor's initial state is a learned quantity, initialised like a weight).
 * Both fields are optional; with both NULL the initial state is one predictor step on the blank token from an
 * all-zero state (LSTM) or the blank token's embedding (stateless).
 *   pred_init_state  [lstm_layers, 2, lstm_hidden]  per layer h then c (LSTM only; NULL: zeros when
 *                    pred_init_out is given)
 *   pred_init_out    [P]  the predictor output of the empty token prefix (NULL with a state given: the top
 *                    layer's h)
 */
typedef struct {
  int32_t D_enc, P, J, V, blank;
  int32_t pred_kind, emb_dim, lstm_layers, lstm_hidden;
  int32_t joiner_act; /* TW_ACT_TANH or TW_ACT_RELU */
  int32_t dtype;      /* TW_F32 or TW_BF16 */
  int32_t joiner_norm; /* TW_NORM_SOFTMAX: J = softmax(z) (Sec. 3.1).  TW_NORM_HAT: the factorised output that blank
                          thresholding needs (Sec. 2): p(blank) = sigmoid(z_blank), and p(k) = (1 - p(blank)) *
                          softmax over the non-blank tokens; row `blank` of W_out is then the blank head */
  const void* W_e;   /* [J, D_enc] */
  const void* W_p;   /* [J, P]     */
  const void* W_out; /* [V, J]     */
  const void* b_out; /* [V]        */
  const void* emb;   /* [V, emb_dim] */
  const void* const* host_lstm_W_ih; /* [lstm_layers] -> [4*Hd, in]  (in = emb_dim, then Hd) */
  const void* const* host_lstm_W_hh; /* [lstm_layers] -> [4*Hd, Hd] */
  const void* const* host_lstm_b;    /* [lstm_layers] -> [4*Hd]     */
  const void* pred_init_state;       /* optional, see above */
  const void* pred_init_out;         /* optional, see above */
} tw_model;

/*
 * Search parameters (Algorithm 1 inputs N and S) and capacities.
 *   max_iters_per_segment: safety cap on passes of the inner loop per segment; the paper relies on
 *     the threshold alone.  When an utterance hits it the rest of its list A is dropped for that
 *     segment and its status becomes TW_ERR_LIMIT.  0 selects 4*S + 16.
 *   max_tokens: capacity of a hypothesis' token sequence (U_cap).  An expansion that would exceed
 *     it is dropped and the utterance's status becomes TW_ERR_LIMIT.  0 selects 512.
 */
typedef struct {
  int32_t N, S, mode;
  int32_t max_batch, max_T;
  int32_t max_iters_per_segment;
  int32_t max_tokens;
} tw_config;

/* Counters of the last tw_decode (Sec. 4.2: Calls/Frame = calls/frames, Joins/Frame = joins/frames). */
typedef struct {
  int64_t frames;        /* sum of utterance lengths                                  */
  int64_t calls;         /* sum over utterances of inner-loop passes (joiner calls)   */
  int64_t joins;         /* sum over passes of the frames in that pass' segment       */
  int64_t steps;         /* batched device steps that did work (one step = one pass for every live utterance) */
  int64_t rows;          /* sum over steps of live hypothesis rows R                  */
  int64_t kernel_launches; /* kernels enqueued by the last tw_decode                  */
  int64_t limit_hits;    /* utterances whose status is TW_ERR_LIMIT                   */
  int64_t joiner_frame_rows; /* sum over steps of (rows x frames of their segment) = joiner GEMM rows M */
  /* device time per stage in nanoseconds, summed over the decode; zero unless tw_set_profiling(h, 1) */
  int64_t ns_prologue;   /* E = enc W_e^T and list initialisation                      */
  int64_t ns_predictor;  /* UpdatePredictorOutput                                      */
  int64_t ns_joiner;     /* the joiner kernel alone: contraction, or the fused contraction + softmax + Eq. 3-7 */
  int64_t ns_scan;       /* separate softmax / Eq. 3-7 / selection kernels and the joiner's operand kernel */
  int64_t ns_hyp;        /* AddAndMerge, threshold, N-best expansions, compaction      */
  int64_t joiner_launches; /* launches summed in ns_joiner                             */
  int64_t fused_clusters;  /* clusters the fused joiner keeps resident (0: fused path unavailable) */
  int64_t fused_on;        /* 1 if tw_decode takes the fused joiner path                          */
  int64_t frame_rows_skipped; /* of joiner_frame_rows, the (row, frame) pairs blank thresholding left out */
} tw_stats;

/* Builds a decoder: copies (and in bf16 mode converts) the weights, runs InitPredictor, allocates
 * the workspace for max_batch utterances of up to max_T frames.  Synchronises the device.
 * Errors: TW_ERR_ARG for null pointers, N not in [1, TW_MAX_BEAM], S not in [1, TW_MAX_SEGMENT],
 * V - 1 < N (fewer non-blank tokens than the beam), blank outside [0, V), P inconsistent with the
 * predictor; TW_ERR_ALLOC / TW_ERR_CUDA otherwise.  *out is NULL on failure.  The library reads no environment
 * variable: every switch is a call on the handle. */
int tw_init(const tw_model* host_model, const tw_config* host_cfg, tw_handle** out);
int tw_destroy(tw_handle* h);

/*
 * Algorithm 1 for a batch of B utterances, each decoded independently.
 *   enc      [B, T, D_enc]  encoder output (computed beforehand, Sec. 3.2), elements of the model's dtype;
 *                           frames at or past lengths[b] are ignored
 *   lengths  [B]            0 <= lengths[b] <= T (values outside are clamped and flagged TW_ERR_ARG
 *                           in out_status[b])
 *   out_tokens [B, N, U_cap] N best token sequences, best first, padded with -1
 *   out_lens   [B, N]        their lengths; -1 for an unused slot (fewer than N hypotheses)
 *   out_scores [B, N]        float64 log p, descending; -inf for an unused slot
 *   out_status [B]           TW_OK, TW_ERR_LIMIT or TW_ERR_ARG per utterance
 * Every step of the inner loop (joiner over the segment, softmax, Eq. 3-7, AddAndMerge, threshold,
 * N-best expansions, predictor update) runs on the device; the host only enqueues batches of steps
 * and polls one completion word between batches.  The call synchronises `stream` before returning.
 * Returns TW_ERR_LIMIT if any utterance hit a cap (outputs are still valid for the others),
 * TW_ERR_ARG if B > max_batch, T > max_T or a pointer is null.
 */
int tw_decode(tw_handle* h, const void* enc, const int32_t* lengths, int32_t B, int32_t T,
              int32_t* out_tokens, int32_t* out_lens, double* out_scores, int32_t* out_status,
              void* stream);

/* Same as tw_decode with HOST buffers: copies the inputs to the device, decodes, copies the four
 * outputs back; synchronises before returning.  For batches decoded in one piece and T >= 16 S the
 * frames are uploaded in two time chunks (the first sixteenth, then the rest) on a stream of the handle's own
 * (ordered after `stream`) and the first chunk is decoded, as a streaming push, while the second is on its way; the result is
 * the same as tw_decode's.  Pinned host memory is what makes the upload asynchronous.  Must not be
 * called while a streaming session is open on the handle. */
int tw_decode_host(tw_handle* h, const void* host_enc, const int32_t* host_lengths, int32_t B,
                   int32_t T, int32_t* host_out_tokens, int32_t* host_out_lens,
                   double* host_out_scores, int32_t* host_out_status, void* stream);

/*
 * Streaming (Sec. 3.2: the encoder output may arrive segment by segment, and the chunk size used for
 * the encoder need not equal the decoding segment size S).  One session per handle at a time; the beam
 * state (list B, hypotheses, predictor states) stays on the device between calls.
 *   tw_stream_open   starts a session of B utterances with no frames.
 *   tw_stream_push   appends chunk_lens[b] <= Tc frames of enc_chunk [B, Tc, D_enc] to utterance b and
 *                    decodes every whole segment of S frames that is now available; frames short of a
 *                    segment wait for the next push.  At most max_T frames per utterance in total
 *                    (more are dropped and the utterance reports TW_ERR_LIMIT).
 *   tw_stream_nbest  the current N best of every utterance (outputs as in tw_decode).
 *   tw_stream_close  decodes the frames short of a segment as a last, shorter one and returns the final
 *                    N best; tw_get_stats then covers the whole session.
 * After tw_stream_close the result is exactly that of tw_decode on the concatenated frames.
 * All four synchronise before returning.  TW_ERR_STATE without an open session.
 */
int tw_stream_open(tw_handle* h, int32_t B, void* stream);
int tw_stream_push(tw_handle* h, const void* enc_chunk, const int32_t* chunk_lens, int32_t Tc, void* stream);
int tw_stream_nbest(tw_handle* h, int32_t* out_tokens, int32_t* out_lens, double* out_scores,
                    int32_t* out_status, void* stream);
int tw_stream_close(tw_handle* h, int32_t* out_tokens, int32_t* out_lens, double* out_scores,
                    int32_t* out_status, void* stream);

/* U_cap of this handle (row length of out_tokens). */
int tw_max_tokens(const tw_handle* h);

/*
 * Encoder half of the joiner's first layer, E = enc . W_e^T, computed once per frame
 * (Sec. 3.1 joiner; the split of the first layer is exact algebra).
 *   enc [rows, D_enc] (the model's dtype) -> out_E [rows, J] float32
 */
int tw_project_encoder(tw_handle* h, const void* enc, int32_t rows, float* out_E, void* stream);

/*
 * J = Softmax(Joiner(seg, pred)) of Algorithm 1 for R hypothesis rows, in log space.
 *   E_seg     [G, S, J]  projected frames of G segments (see tw_project_encoder)
 *   Pp        [R, J]     projected predictor outputs W_p g of the R rows
 *   row_group [R]        segment index g of each row, 0 <= g < G
 *   seg_len   [G]        valid frames of each segment, 1 <= seg_len[g] <= S (NULL: all S)
 *   out_logp  [R, S, V]  log J(t, r, k); for a frame t >= seg_len the row is the pass-through
 *                        pattern (0 at blank, -inf elsewhere), which leaves Eq. 3-7 unchanged
 * Errors: TW_ERR_ARG for null pointers or R, G < 0.  R == 0 is a no-op.
 */
int tw_joiner_segment(tw_handle* h, const float* E_seg, const float* Pp, const int32_t* row_group,
                      const int32_t* seg_len, int32_t G, int32_t R, float* out_logp, void* stream);

/*
 * Eq. 3-7 for R rows from materialised log-probabilities.
 *   logp        [R, S, V]  log J
 *   ld_old      [R, S]     log d_old: log-probability that the row's last token was emitted at
 *                          frame t (Eq. 2); -inf allowed.  Any common offset per row carries
 *                          through to the outputs, so callers may pass values relative to the
 *                          row's score.
 *   seg_len_row [R]        valid frames per row (NULL: all S)
 *   out_ldphi   [R]        log delta_phi (Eq. 7)
 *   out_ldnb    [R, V]     log delta_nb(k) (Eq. 6); -inf at the blank column
 *   out_la      [R, S]     log a(t) = log sum_{t1<=t} d_old(t1) Bl(t1, t), so that Eq. 5 reads
 *                          log d(k, t) = out_la[t] + logp[t, k]; -inf for t >= seg_len
 */
int tw_expand(tw_handle* h, const float* logp, const float* ld_old, const int32_t* seg_len_row,
              int32_t R, float* out_ldphi, float* out_ldnb, float* out_la, void* stream);

/*
 * Joiner, softmax and Eq. 3-7 in one call, without handing log J to the caller (the path tw_decode
 * takes).  Arguments as in tw_joiner_segment and tw_expand; ld_old is [R, S] and seg_len is per
 * segment.  R must not exceed max_batch * N.  In TW_MODE_F32 this runs the two stages above through
 * the handle's own log J buffer.
 */
int tw_joiner_expand(tw_handle* h, const float* E_seg, const float* Pp, const int32_t* row_group,
                     const int32_t* seg_len, const float* ld_old, int32_t G, int32_t R,
                     float* out_ldphi, float* out_ldnb, float* out_la, void* stream);

/*
 * UpdatePredictorOutput (Algorithm 1) for R hypotheses at once: one predictor step on `tokens[r]`
 * from the parent's recurrent state.
 *   tokens    [R]
 *   state_in  [R, L, 2, Hd]  per layer h then c (ignored for the stateless predictor; may be NULL)
 *   state_out [R, L, 2, Hd]  (may be NULL for the stateless predictor)
 *   out_Pp    [R, J]         W_p g for the joiner
 * InitPredictor corresponds to tokens = blank with an all-zero state_in.
 * R must not exceed max_batch * N.
 */
int tw_predictor_step(tw_handle* h, const int32_t* tokens, const float* state_in, int32_t R,
                      float* state_out, float* out_Pp, void* stream);

/*
 * Joiner, softmax and Eq. 3-7 for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging of tw_joiner_expand, not another operation.)
 *
 * Who needs it: a process whose GPU memory already belongs to someone else's allocator, for instance
 * an inference server that reserved all of HBM for its own pool at start-up, or a latency-critical
 * loop in which a cudaMalloc / cudaFree would stall every stream of the device.  Such a caller cannot
 * afford tw_init, which allocates a workspace.  This call takes no handle: the caller passes the two
 * joiner weights it needs as ordinary inputs, and the intermediate log J tensor is kept in a fixed
 * array inside the library image (about 16 MiB per GPU that loads the library, held until the
 * process exits).  The call itself never calls cudaMalloc, cudaFree or any allocating routine.
 *
 *   W_out [V, J], b_out [V]   joiner output layer (float32, device)
 *   joiner_act                TW_ACT_TANH or TW_ACT_RELU: the joiner's hidden nonlinearity (a handle carries it in
 *                             its model; here it has to be said)
 *   the remaining arguments are those of tw_joiner_expand, computed in float32
 * Limits: R <= TW_NOALLOC_MAX_ROWS and R * S * V <= TW_NOALLOC_MAX_ELEMS; a larger request returns
 * TW_ERR_LIMIT and enqueues nothing.  Other bad arguments return TW_ERR_ARG.
 * The first call on each device looks up the device address of the fixed array (with that device
 * current); make that first call outside any stream capture.
 * All calls on a device share the one array, which keeps whatever the previous call left in it.
 * Nothing in it has to start at zero: each call overwrites every element it later reads.  Two calls
 * that overlap on the GPU (different streams, or different host threads) race on the array and give
 * wrong results; serialise them.
 */
#define TW_NOALLOC_MAX_ROWS 4096
#define TW_NOALLOC_MAX_ELEMS (4 * 1024 * 1024)
int tw_joiner_expand_noalloc(const float* W_out, const float* b_out, int32_t J, int32_t V, int32_t S,
                             int32_t blank, int32_t joiner_act, const float* E_seg, const float* Pp,
                             const int32_t* row_group, const int32_t* seg_len, const float* ld_old,
                             int32_t G, int32_t R, float* out_ldphi, float* out_ldnb, float* out_la,
                             void* stream);

/* TW_MODE_BF16 only: switches between the fused joiner (joiner, softmax and Eq. 3-7 in one kernel, logits
 * kept in tensor memory; available when S <= 32 and V <= 4096, a vocabulary that is not a multiple of 256
 * being padded internally with columns of probability 0; the default for S in {1..5, 8, 10}) and the
 * staged kernels that pass the logits through device memory.  Both compute the same quantities.
 * TW_ERR_STATE if the fused kernel is not available for this handle. */
int tw_set_fused(tw_handle* h, int on);

/* tw_decode replays its step body (16 device steps) as a CUDA graph, captured once per batch shape, on
 * a stream of the handle's own that is ordered after `stream`; tw_set_graph(h, 0) makes it enqueue the
 * kernels one by one on `stream` instead (as it also does while profiling is on).  Default: on. */
int tw_set_graph(tw_handle* h, int on);

/* A handle with max_batch >= 256 also holds two internal decoders for half the batch each; tw_decode then
 * splits a batch of 256 or more utterances in two halves and advances them concurrently on two streams
 * (utterances are independent), which overlaps one half's small kernels with the other half's GEMMs.
 * tw_set_lanes(h, 0) decodes the batch in one piece.  Default: on.  Off while profiling is on. */
int tw_set_lanes(tw_handle* h, int on);

/* TW_MODE_BF16 with the fused joiner and an LSTM predictor: by default the hypothesis-step kernel of a decode step also
 * builds the predictor's work list and writes the parents' recurrent states into the gate GEMMs' operand rows;
 * tw_set_inline_gather(h, 0) leaves both to a kernel of their own (one more launch per step, a work list in a fixed
 * order).  Both give the same N-best.  TW_ERR_STATE if the handle has no such path, or while a streaming session is open. */
int tw_set_inline_gather(tw_handle* h, int on);

/* Blank thresholding (Sec. 2 and Sec. 5 name it as a way to skip joiner work that adds to the gains of Algorithm 1;
 * the paper prints no equations for it).  Only for a TW_NORM_HAT model, whose blank probability comes from a head of
 * its own.  A (hypothesis, frame) pair whose blank probability exceeds `threshold` contributes that blank probability
 * only: its non-blank terms drop out of Eq. 4-6.  threshold = 1 (the default) skips nothing, threshold = 0 skips every
 * pair.  tw_stats::frame_rows_skipped counts the skipped pairs of a decode.  TW_MODE_F32 and the staged TW_MODE_BF16
 * kernels drop the terms after the contraction; the fused kernel masks them in its epilogue (its tile layout keeps a
 * lane per frame, so the contraction's row count does not shrink).  TW_ERR_STATE for a softmax model or while a
 * streaming session is open, TW_ERR_ARG for a threshold outside [0, 1]. */
int tw_set_blank_threshold(tw_handle* h, float threshold);

/* Monotonic RNN-T variant (Sec. 2 and Sec. 5 name it as an adjustment of Algorithm 1; the paper prints no
 * equations for it).  Every output, blank or token, consumes one frame, so at most one token is emitted
 * per frame.  In Eq. 4-5 a token emitted at frame t2 leaves its hypothesis at frame t2 + 1, and a
 * hypothesis that emits at the segment's last frame has left the segment: its mass is added to Eq. 7's
 * delta_phi.  Eq. 3 and Eq. 6 are unchanged.  on != 0 selects the variant for later tw_decode and
 * tw_stream_open calls on this handle; TW_ERR_STATE while a streaming session is open.  Default: off. */
int tw_set_monotonic(tw_handle* h, int on);

/* Per-stage device timing of tw_decode with CUDA events on the decode stream (adds two event records
 * per stage per step); off by default.  While it is on, tw_joiner_expand on the fused path also times its two
 * kernels: each call synchronises `stream` and ADDS the operand kernel's device time to ns_scan, the fused
 * kernel's to ns_joiner and 1 to joiner_launches (tw_get_stats).  Every call of tw_set_profiling clears those
 * three counters. */
int tw_set_profiling(tw_handle* h, int on);
int tw_get_stats(const tw_handle* h, tw_stats* host_out);
int tw_last_cuda_error(const tw_handle* h); /* cudaError_t of the last failed CUDA call, 0 if none */
const char* tw_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* TW_H_ */
