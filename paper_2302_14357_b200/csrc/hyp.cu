// Hypothesis management of Algorithm 1 on the device: lists A and B, AddAndMerge, the N-th score
// threshold, N-best expansions with the strict '>' filter, segment turn-over, N-best read-out.
// One CTA owns one utterance; utterances advance independently of each other (an utterance whose
// list A runs empty moves to its next segment at once, it does not wait for the batch).
//
// Scores are carried in float64: a hypothesis' log-probability reaches thousands of nats, where
// float32 spacing (1.2e-4 at 2048) is coarser than the accuracy the stage kernels deliver.  The
// stage kernels work on values relative to the row's score, which stay small.
#include "tw_internal.cuh"

namespace tw {

namespace {

constexpr int kThreads = 256;
constexpr unsigned long long kHashSeed = 0x9E3779B97F4A7C15ull;

__device__ __forceinline__ unsigned long long hash_push(unsigned long long h, int tok) {
  unsigned long long x = h * 0x100000001B3ull + (unsigned long long)(tok + 1);
  x ^= x >> 33; x *= 0xFF51AFD7ED558CCDull;
  x ^= x >> 33; x *= 0xC4CEB9FE1A85EC53ull;
  x ^= x >> 33;
  return x;
}

__device__ __forceinline__ int block_min_int(int v, int* scratch) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = min(v, __shfl_xor_sync(0xffffffffu, v, o));
  __syncthreads();
  if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
  __syncthreads();
  int r = scratch[0];
#pragma unroll
  for (int i = 1; i < kThreads / 32; ++i) r = min(r, scratch[i]);
  return r;
}

// Starts the next segment of utterance b: A = ChooseNBest(B), B = [], t += S, d = (s, 0, ..., 0).
// Precondition: list A is empty and frames remain.  Called by the whole CTA.
__device__ void turn_over(const HypState& hs, int b) {
  __shared__ int s_n;
  __syncthreads();
  if (threadIdx.x == 0) {
    const int n = hs.nTop[b];
    const int t0 = hs.t0[b] + hs.slen[b];
    hs.t0[b] = t0;
    hs.slen[b] = min(hs.S, hs.len[b] - t0);
    for (int i = 0; i < kMaxBeam; ++i) {
      if (i < n) {
        const int e = hs.B_top[b * kMaxBeam + i];
        const int slot = hs.B_slot[(long long)b * hs.capB + e];
        hs.A_slot[b * kMaxBeam + i] = slot;
        hs.A_ls[b * kMaxBeam + i] = hs.B_ls[(long long)b * hs.capB + e];
        hs.carry[b * kMaxBeam + i] = slot;
      } else {
        hs.carry[b * kMaxBeam + i] = -1;
      }
    }
    hs.nA[b] = n;
    hs.nB[b] = 0;
    hs.nTop[b] = 0;
    hs.iters[b] = 0;
    s_n = n;
  }
  __syncthreads();
  const int n = s_n;
  for (int i = threadIdx.x; i < n * hs.S; i += blockDim.x) {
    const int a = i / hs.S, t = i - a * hs.S;
    hs.A_ld[((long long)b * kMaxBeam + a) * hs.S + t] = (t == 0) ? hs.A_ls[b * kMaxBeam + a] : -INFINITY;
  }
}

__global__ void __launch_bounds__(kThreads) hyp_init_kernel(HypState hs, const int* lengths, int T) {
  const int b = blockIdx.x;
  const long long gs = (long long)b * hs.capSlot;   // slot 0 holds the empty hypothesis
  if (threadIdx.x == 0) {
    int len = lengths[b], st = TW_OK;
    if (len < 0) { len = 0; st = TW_ERR_ARG; }
    if (len > T) { len = T; st = TW_ERR_ARG; }
    hs.len[b] = len; hs.status[b] = st;
    hs.calls[b] = 0; hs.joins[b] = 0; hs.iters[b] = 0; hs.cursor[b] = 0; hs.n_new[b] = 0;
    hs.t0[b] = 0; hs.slen[b] = 0; hs.nA[b] = 0;
    hs.slot_len[gs] = 0; hs.slot_hash[gs] = kHashSeed;
    // B = [([], 1, InitPredictor(), Null)]
    hs.B_slot[(long long)b * hs.capB] = 0;
    hs.B_ls[(long long)b * hs.capB] = 0.0;
    hs.B_hash[(long long)b * hs.capB] = kHashSeed;
    hs.B_len[(long long)b * hs.capB] = 0;
    hs.nB[b] = 1; hs.nTop[b] = 1; hs.B_top[b * kMaxBeam] = 0;
  }
  if (!hs.stateless) {
    const int nhc = hs.L * 2 * hs.Hd;
    for (int i = threadIdx.x; i < nhc; i += blockDim.x) hs.slot_hc[gs * nhc + i] = hs.init_hc[i];
    for (int i = threadIdx.x; i < hs.J; i += blockDim.x) hs.slot_Pp[gs * hs.J + i] = hs.init_Pp[i];
  }
  __syncthreads();
  if (hs.len[b] > 0) turn_over(hs, b);
}

__device__ __forceinline__ bool better(float v, int k, float v2, int k2) {
  return v > v2 || (v == v2 && k < k2);
}

__global__ void __launch_bounds__(kThreads) hyp_step_kernel(HypState hs) {
  __shared__ int s_scratch[kThreads / 32];
  __shared__ int s_nB, s_hasthr, s_nkeep, s_ntot;
  __shared__ int s_touched[kMaxBeam];
  __shared__ double s_Als[kMaxBeam];
  __shared__ int s_Aslot[kMaxBeam];
  __shared__ double s_thr;
  __shared__ float s_cv[kMaxBeam][kMaxBeam];
  __shared__ int s_ck[kMaxBeam][kMaxBeam];
  __shared__ int s_cnt[kMaxBeam];
  __shared__ double s_abs[kMaxBeam * kMaxBeam];
  __shared__ int s_sel[kMaxBeam];
  __shared__ int s_keep_h[kMaxBeam], s_keep_k[kMaxBeam], s_keep_slot[kMaxBeam];
  __shared__ double s_keep_ls[kMaxBeam];
  __shared__ double s_newld[kMaxBeam][kMaxSeg];

  const int b = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int H = hs.nA[b];
  if (H == 0) return;                       // idle (finished) utterance
  const int N = hs.N, S = hs.S, V = hs.V;
  const int r0 = hs.row_off[b];
  const int slen = hs.slen[b];
  const long long bB = (long long)b * hs.capB;
  const long long bS = (long long)b * hs.capSlot;

  if (tid < H) { s_Als[tid] = hs.A_ls[b * kMaxBeam + tid]; s_Aslot[tid] = hs.A_slot[b * kMaxBeam + tid]; }
  if (tid == 0) {
    s_nB = hs.nB[b];
    hs.calls[b] += 1;
    hs.joins[b] += slen;
  }
  __syncthreads();

  // ---- AddAndMerge of the blank expansions (tok, delta_phi, o) into list B -------------------
  for (int h = 0; h < H; ++h) {
    const int slot = s_Aslot[h];
    const unsigned long long hh = hs.slot_hash[bS + slot];
    const int ln = hs.slot_len[bS + slot];
    const int nB = s_nB;
    int start = 0, found = -1;
    while (true) {
      int local = 0x7fffffff;
      for (int e = start + tid; e < nB; e += kThreads) {
        if (hs.B_hash[bB + e] == hh && hs.B_len[bB + e] == ln) { local = e; break; }
      }
      const int cand = block_min_int(local, s_scratch);
      if (cand == 0x7fffffff) break;
      // verify token by token (a 64-bit hash match is not proof)
      const int oslot = hs.B_slot[bB + cand];
      int diff = 0;
      if (oslot != slot) {
        const int* ta = hs.slot_tok + (bS + slot) * hs.U_cap;
        const int* tb = hs.slot_tok + (bS + oslot) * hs.U_cap;
        for (int i = tid; i < ln; i += kThreads) diff |= (ta[i] != tb[i]);
      }
      if (!__syncthreads_or(diff)) { found = cand; break; }
      start = cand + 1;
    }
    if (tid == 0) {
      const double val = s_Als[h] + (hs.ldphi_d ? hs.ldphi_d[r0 + h] : (double)hs.ldphi[r0 + h]);
      if (found >= 0) {
        hs.B_ls[bB + found] = logaddexp_d(hs.B_ls[bB + found], val);
        s_touched[h] = found;
      } else {
        const int e = s_nB;                 // capB = N * I_max bounds this by construction
        hs.B_slot[bB + e] = slot; hs.B_ls[bB + e] = val; hs.B_hash[bB + e] = hh; hs.B_len[bB + e] = ln;
        s_touched[h] = e;
        s_nB = e + 1;
      }
    }
    __syncthreads();
  }

  // ---- ChooseNthScore: the best N of B are among the previous best N and the entries touched now
  if (warp == 0) {
    const int nT = hs.nTop[b];
    int idx = -1;
    if (lane < nT) {
      idx = hs.B_top[b * kMaxBeam + lane];
    } else if (lane - nT < H) {
      const int cand = s_touched[lane - nT];
      bool dup = false;
      for (int i = 0; i < nT; ++i) dup |= (hs.B_top[b * kMaxBeam + i] == cand);
      if (!dup) idx = cand;
    }
    const double score = idx >= 0 ? hs.B_ls[bB + idx] : -INFINITY;
    int rank = 0;
    for (int j = 0; j < 32; ++j) {
      const double sj = __shfl_sync(0xffffffffu, score, j);
      const int ij = __shfl_sync(0xffffffffu, idx, j);
      if (ij >= 0 && (sj > score || (sj == score && ij < idx))) ++rank;
    }
    const int count = __popc(__ballot_sync(0xffffffffu, idx >= 0));
    __syncwarp();
    if (idx >= 0 && rank < N) hs.B_top[b * kMaxBeam + rank] = idx;
    if (idx >= 0 && rank == N - 1) s_thr = score;
    if (lane == 0) {
      hs.nTop[b] = min(N, count);
      s_hasthr = (count >= N);
      hs.nB[b] = s_nB;
    }
  }
  __syncthreads();
  const bool hasthr = s_hasthr != 0;
  const double thr = hasthr ? s_thr : -INFINITY;

  // ---- ChooseNBestExpansions, stage 1: per hypothesis row, the N best non-blank tokens -------
  for (int h = warp; h < H; h += kThreads / 32) {
    const float* row = hs.ldnb + (long long)(r0 + h) * V;
    // anything at or below the threshold fails the filter later; a small slack keeps the exact
    // float64 comparison authoritative
    const float bound = hasthr ? (float)(thr - s_Als[h]) - 1e-3f : -INFINITY;
    float lv[kMaxBeam]; int lk[kMaxBeam];
#pragma unroll
    for (int j = 0; j < kMaxBeam; ++j) { lv[j] = -INFINITY; lk[j] = 0x7fffffff; }
    float admit = bound;
    for (int k = lane; k < V; k += 32) {
      const float v = row[k];               // the blank column holds -inf and never passes
      if (v > admit) {
        float cv = v; int ck = k;
#pragma unroll
        for (int j = 0; j < kMaxBeam; ++j) {
          if (better(cv, ck, lv[j], lk[j])) {
            const float tv = lv[j]; const int tk = lk[j];
            lv[j] = cv; lk[j] = ck; cv = tv; ck = tk;
          }
        }
        float last = -INFINITY;
#pragma unroll
        for (int j = 0; j < kMaxBeam; ++j) if (j == N - 1) last = lv[j];
        admit = fmaxf(bound, last);
      }
    }
    int cnt = 0;
    for (int j = 0; j < N; ++j) {
      float bv = lv[0]; int bk = lk[0]; int bl = lane;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int ok = __shfl_xor_sync(0xffffffffu, bk, o);
        const int ol = __shfl_xor_sync(0xffffffffu, bl, o);
        if (better(ov, ok, bv, bk)) { bv = ov; bk = ok; bl = ol; }
      }
      if (bv == -INFINITY) break;
      if (lane == 0) { s_cv[h][j] = bv; s_ck[h][j] = bk; }
      if (lane == bl) {
#pragma unroll
        for (int i = 0; i < kMaxBeam - 1; ++i) { lv[i] = lv[i + 1]; lk[i] = lk[i + 1]; }
        lv[kMaxBeam - 1] = -INFINITY; lk[kMaxBeam - 1] = 0x7fffffff;
      }
      ++cnt;
    }
    if (lane == 0) s_cnt[h] = cnt;
  }
  __syncthreads();

  // ---- stage 2: the N best (h, k) over all rows, in float64; order (score desc, h asc, k asc) -
  {
    const int h = tid / kMaxBeam, j = tid % kMaxBeam;
    const bool valid = h < H && j < s_cnt[h];
    s_abs[tid] = valid ? s_Als[h] + (double)s_cv[h][j] : -INFINITY;
    if (tid == 0) s_ntot = 0;
    __syncthreads();
    if (valid) {
      const double mine = s_abs[tid];
      int rank = 0;
      for (int o = 0; o < kMaxBeam * kMaxBeam; ++o) {
        const int oh = o / kMaxBeam, oj = o % kMaxBeam;
        if (oh < H && oj < s_cnt[oh]) {
          const double so = s_abs[o];
          if (so > mine || (so == mine && o < tid)) ++rank;   // o < tid  <=>  (h, k) order: rows are sorted by (v desc, k asc)
        }
      }
      if (rank < N) s_sel[rank] = tid;
      atomicAdd(&s_ntot, 1);
    }
    __syncthreads();
  }

  // ---- filter against the threshold, allocate slots ------------------------------------------
  if (tid == 0) {
    const int nC = min(N, s_ntot);
    int nk = 0;
    int cur = hs.cursor[b];
    const bool capped = hs.iters[b] + 1 >= hs.I_max;
    hs.iters[b] += 1;
    for (int i = 0; i < nC; ++i) {
      const int c = s_sel[i];
      const int h = c / kMaxBeam, j = c % kMaxBeam;
      const double sc = s_abs[c];
      if (hasthr && !(sc > thr)) continue;            // Length(B) < N or delta_nb > threshold
      if (capped) { hs.status[b] = TW_ERR_LIMIT; break; }
      if (hs.slot_len[bS + s_Aslot[h]] + 1 > hs.U_cap) { hs.status[b] = TW_ERR_LIMIT; continue; }
      // next free slot of the ring: skip slots still held by hypotheses carried into this segment
      bool busy;
      do {
        cur = (cur + 1 == hs.capSlot) ? 0 : cur + 1;
        busy = false;
        for (int q = 0; q < kMaxBeam; ++q) busy |= (hs.carry[b * kMaxBeam + q] == cur);
      } while (busy);
      s_keep_h[nk] = h; s_keep_k[nk] = s_ck[h][j]; s_keep_ls[nk] = sc; s_keep_slot[nk] = cur;
      ++nk;
    }
    hs.cursor[b] = cur;
    s_nkeep = nk;
  }
  __syncthreads();
  const int nk = s_nkeep;

  // ---- new list A: tokens, hash, frame distribution d_h(k) (Eq. 5) ----------------------------
  for (int i = 0; i < nk; ++i) {
    const int h = s_keep_h[i], k = s_keep_k[i];
    const long long gp = bS + s_Aslot[h], gn = bS + s_keep_slot[i];
    const int plen = hs.slot_len[gp];
    const int* src = hs.slot_tok + gp * hs.U_cap;
    int* dst = hs.slot_tok + gn * hs.U_cap;
    for (int q = tid; q < plen; q += kThreads) dst[q] = src[q];
    if (tid == 0) {
      dst[plen] = k;
      hs.slot_len[gn] = plen + 1;
      hs.slot_hash[gn] = hash_push(hs.slot_hash[gp], k);
      hs.new_slot[b * kMaxBeam + i] = (int)gn;
      hs.new_par[b * kMaxBeam + i] = (int)gp;
      hs.new_tok[b * kMaxBeam + i] = k;
    }
    if (tid < S) {
      double v = -INFINITY;
      if (tid < slen && hs.logp != nullptr) {
        const long long r = r0 + h;
        const double a = hs.la_d ? hs.la_d[r * S + tid] : (double)hs.la[r * S + tid];
        v = s_Als[h] + a + (double)hs.logp[(r * S + tid) * V + k];
      }
      s_newld[i][tid] = v;
    }
  }
  __syncthreads();
  if (tid < nk) {
    hs.A_slot[b * kMaxBeam + tid] = s_keep_slot[tid];
    hs.A_ls[b * kMaxBeam + tid] = s_keep_ls[tid];
  }
  for (int i = tid; i < nk * S; i += kThreads) {
    const int a = i / S, t = i - a * S;
    hs.A_ld[((long long)b * kMaxBeam + a) * S + t] = s_newld[a][t];
  }
  if (tid == 0) { hs.nA[b] = nk; hs.n_new[b] = nk; }
  __syncthreads();

  // ---- list A empty: this segment is done ------------------------------------------------------
  if (nk == 0 && hs.t0[b] + slen < hs.len[b]) turn_over(hs, b);
}

// One CTA: packs the live hypotheses of all utterances into joiner rows and the new hypotheses
// into the predictor's work list.
__global__ void __launch_bounds__(1024) compact_kernel(HypState hs, int B, int T) {
  __shared__ int s_a[1024], s_n[1024];
  __shared__ int s_base_a, s_base_n, s_frames;
  const int tid = threadIdx.x;
  if (tid == 0) { s_base_a = 0; s_base_n = 0; s_frames = 0; }
  __syncthreads();
  for (int b0 = 0; b0 < B; b0 += 1024) {
    const int b = b0 + tid;
    const int a = b < B ? hs.nA[b] : 0;
    const int nn = b < B ? hs.n_new[b] : 0;
    s_a[tid] = a; s_n[tid] = nn;
    __syncthreads();
    for (int o = 1; o < 1024; o <<= 1) {          // inclusive scan
      int va = 0, vn = 0;
      if (tid >= o) { va = s_a[tid - o]; vn = s_n[tid - o]; }
      __syncthreads();
      s_a[tid] += va; s_n[tid] += vn;
      __syncthreads();
    }
    const int off_a = s_base_a + s_a[tid] - a;
    const int off_n = s_base_n + s_n[tid] - nn;
    if (b < B) {
      hs.row_off[b] = off_a;
      const int t0 = hs.t0[b], sl = hs.slen[b];
      if (a > 0) atomicAdd(&s_frames, a * sl);
      for (int h = 0; h < a; ++h) {
        const int r = off_a + h;
        const int slot = hs.A_slot[b * kMaxBeam + h];
        const long long gs = (long long)b * hs.capSlot + slot;
        hs.row_b[r] = b;
        hs.row_e0[r] = b * T + t0;
        hs.row_slen[r] = sl;
        if (hs.stateless) {
          const int ln = hs.slot_len[gs];
          hs.row_p[r] = ln > 0 ? hs.slot_tok[gs * hs.U_cap + ln - 1] : hs.blank;
        } else {
          hs.row_p[r] = (int)gs;
        }
        const double ls = hs.A_ls[b * kMaxBeam + h];
        for (int t = 0; t < hs.S; ++t) {
          const double d = hs.A_ld[((long long)b * kMaxBeam + h) * hs.S + t];
          hs.row_ld[(long long)r * hs.S + t] = (d == -INFINITY) ? -INFINITY : (float)(d - ls);
        }
      }
      for (int j = 0; j < nn; ++j) {
        hs.pw_new[off_n + j] = hs.new_slot[b * kMaxBeam + j];
        hs.pw_par[off_n + j] = hs.new_par[b * kMaxBeam + j];
        hs.pw_tok[off_n + j] = hs.new_tok[b * kMaxBeam + j];
      }
      hs.n_new[b] = 0;
    }
    __syncthreads();
    if (tid == 1023) { s_base_a += s_a[1023]; s_base_n += s_n[1023]; }
    __syncthreads();
  }
  if (tid == 0) {
    const int R = s_base_a;
    hs.scalars[kScR] = R;
    hs.scalars[kScM] = R * hs.S;
    hs.scalars[kScNPred] = s_base_n;
    hs.scalars[kScActive] = R > 0;
    if (R > 0) { hs.scalars[kScSteps] += 1; hs.rows_total[0] += R; hs.rows_total[1] += s_frames; }
  }
}

// ChooseNBest(B) at the end of the utterance, best first.
__global__ void __launch_bounds__(kThreads) finish_kernel(HypState hs, int* out_tokens, int* out_lens,
                                                          double* out_scores, int* out_status) {
  const int b = blockIdx.x;
  const int nT = hs.nTop[b];
  for (int i = 0; i < hs.N; ++i) {
    int* dst = out_tokens + ((long long)b * hs.N + i) * hs.U_cap;
    int ln = -1;
    double sc = -INFINITY;
    const int* src = nullptr;
    if (i < nT) {
      const int e = hs.B_top[b * kMaxBeam + i];
      const long long gs = (long long)b * hs.capSlot + hs.B_slot[(long long)b * hs.capB + e];
      ln = hs.slot_len[gs];
      sc = hs.B_ls[(long long)b * hs.capB + e];
      src = hs.slot_tok + gs * hs.U_cap;
    }
    for (int q = threadIdx.x; q < hs.U_cap; q += blockDim.x) dst[q] = (q < ln) ? src[q] : -1;
    if (threadIdx.x == 0) { out_lens[b * hs.N + i] = ln; out_scores[b * hs.N + i] = sc; }
  }
  if (threadIdx.x == 0) out_status[b] = hs.status[b];
}

__device__ __forceinline__ float sigmoidf_acc(float x) { return 1.f / (1.f + expf(-x)); }

// c' = sigma(f) c + sigma(i) tanh(g);  h' = sigma(o) tanh(c')   (gate order i, f, g, o)
__global__ void lstm_pointwise_kernel(const float* gates, const int* pw_new, const int* pw_par,
                                      const int* n_dev, int n_max, const float* hc_in, float* hc_out,
                                      int L, int l, int Hd) {
  const int n = n_dev ? *n_dev : n_max;
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long long)n * Hd) return;
  const int r = (int)(i / Hd), j = (int)(i - (long long)r * Hd);
  const float* g = gates + (long long)r * 4 * Hd;
  const long long stride = (long long)L * 2 * Hd;
  const long long pin = (pw_par ? pw_par[r] : r) * stride + (long long)l * 2 * Hd;
  const long long pout = (pw_new ? pw_new[r] : r) * stride + (long long)l * 2 * Hd;
  const float c_prev = hc_in[pin + Hd + j];
  const float c = sigmoidf_acc(g[Hd + j]) * c_prev + sigmoidf_acc(g[j]) * tanhf(g[2 * Hd + j]);
  const float h = sigmoidf_acc(g[3 * Hd + j]) * tanhf(c);
  hc_out[pout + j] = h;
  hc_out[pout + Hd + j] = c;
}

}  // namespace

void launch_hyp_init(const HypState& hs, const int* lengths, int B, int T, cudaStream_t st) {
  if (B > 0) hyp_init_kernel<<<B, kThreads, 0, st>>>(hs, lengths, T);
}
void launch_hyp_step(const HypState& hs, int B, cudaStream_t st) {
  if (B > 0) hyp_step_kernel<<<B, kThreads, 0, st>>>(hs);
}
void launch_compact(const HypState& hs, int B, int T, cudaStream_t st) {
  compact_kernel<<<1, 1024, 0, st>>>(hs, B, T);
}
void launch_finish(const HypState& hs, int B, int* out_tokens, int* out_lens, double* out_scores,
                   int* out_status, cudaStream_t st) {
  if (B > 0) finish_kernel<<<B, kThreads, 0, st>>>(hs, out_tokens, out_lens, out_scores, out_status);
}
void launch_lstm_pointwise(const float* gates, const int* idx_out, const int* idx_in, const int* n_dev,
                           int n_max, const float* hc_in, float* hc_out, int L, int l, int Hd, cudaStream_t st) {
  if (n_max <= 0) return;
  const long long tot = (long long)n_max * Hd;
  lstm_pointwise_kernel<<<(unsigned)((tot + 255) / 256), 256, 0, st>>>(gates, idx_out, idx_in, n_dev, n_max, hc_in,
                                                                      hc_out, L, l, Hd);
}

}  // namespace tw
