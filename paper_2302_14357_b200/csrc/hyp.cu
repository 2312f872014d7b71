// Hypothesis management of Algorithm 1 on the device: lists A and B, AddAndMerge, the N-th score
// threshold, N-best expansions with the strict '>' filter, segment turn-over, N-best read-out.
// One CTA owns one utterance; utterances advance independently of each other (an utterance whose
// list A runs empty moves to its next segment at once, it does not wait for the batch).
//
// Scores are carried in float64: a hypothesis' log-probability reaches thousands of nats, where
// float32 spacing (1.2e-4 at 2048) is coarser than the accuracy the stage kernels deliver.  The
// stage kernels work on values relative to the row's score, which stay small.
#include <cuda_bf16.h>

#include "tw_internal.cuh"
#include "sm100.cuh"

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

// Starts the next segment of utterance b: A = ChooseNBest(B), B = [], t += S, d = (s, 0, ..., 0).
// Precondition: list A is empty and frames remain.  Called by the whole CTA.
__device__ void turn_over(const HypState& hs, int b) {
  __shared__ double s_ls[kMaxBeam];
  __syncthreads();
  const int n = hs.nTop[b];                  // read by every thread before thread 0 clears it below
  if (threadIdx.x < kMaxBeam) {              // one thread per carried hypothesis
    const int i = threadIdx.x;
    if (i < n) {
      const int e = hs.B_top[b * kMaxBeam + i];
      const int slot = hs.B_slot[(long long)b * hs.capB + e];
      const double ls = hs.B_ls[(long long)b * hs.capB + e];
      hs.A_slot[b * kMaxBeam + i] = slot;
      hs.A_ls[b * kMaxBeam + i] = ls;
      hs.A_done[b * kMaxBeam + i] = -INFINITY;
      hs.carry[b * kMaxBeam + i] = slot;
      s_ls[i] = ls;
    } else {
      hs.carry[b * kMaxBeam + i] = -1;
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const int t0 = hs.t0[b] + hs.slen[b];
    hs.t0[b] = t0;
    hs.slen[b] = min(hs.S, hs.len[b] - t0);
    hs.nA[b] = n;
    hs.nB[b] = 0;
    hs.nTop[b] = 0;
    hs.iters[b] = 0;
  }
  for (int i = threadIdx.x; i < n * hs.S; i += blockDim.x) {
    const int a = i / hs.S, t = i - a * hs.S;
    hs.A_ld[((long long)b * kMaxBeam + a) * hs.S + t] = (t == 0) ? s_ls[a] : -INFINITY;
  }
}

__global__ void __launch_bounds__(kThreads) hyp_init_kernel(HypState hs, const int* lengths, int T) {
  const int b = blockIdx.x;
  const long long gs = (long long)b * hs.capSlot;   // slot 0 holds the empty hypothesis
  if (threadIdx.x == 0) {
    int len = lengths[b], st = TW_OK;
    if (len < 0) { len = 0; st = TW_ERR_ARG; }
    if (len > T) { len = T; st = TW_ERR_ARG; }
    hs.len[b] = len; hs.status[b] = st; hs.avail[b] = len;
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

constexpr int kStepThreads = 512;   // 16 warps: one per hypothesis of list A
constexpr int kSelCap = 64;         // survivors of a row's bound that are ranked directly

__device__ __forceinline__ bool tok_better(float v1, int k1, float v2, int k2) { return v1 > v2 || (v1 == v2 && k1 < k2); }

// Order-preserving integer image of a score: a < b as doubles <=> order_key(a) < order_key(b) as unsigned
// integers (-0 counts as +0; scores are never NaN).  The ranking loops compare these instead of doubles.
__device__ __forceinline__ unsigned long long order_key(double x) {
  const unsigned long long u = (unsigned long long)__double_as_longlong(x + 0.0);
  return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}

__global__ void __launch_bounds__(2 * kStepThreads) hyp_step_kernel(HypState hs) {
  __shared__ int s_nB, s_hasthr, s_nkeep, s_wbase;
  __shared__ int s_found[kMaxBeam], s_touched[kMaxBeam], s_carry[kMaxBeam];
  __shared__ double s_Als[kMaxBeam], s_Adone[kMaxBeam];
  __shared__ int s_Aslot[kMaxBeam], s_Alen[kMaxBeam];
  __shared__ double s_thr;
  __shared__ int s_ck[kMaxBeam * kMaxBeam];
  __shared__ double s_abs[kMaxBeam * kMaxBeam];
  __shared__ unsigned long long s_key[kMaxBeam * kMaxBeam];
  __shared__ unsigned long long s_nkey[32];
  __shared__ int s_nidx[32];
  __shared__ float s_lm[kMaxBeam][32], s_sv[kMaxBeam][kSelCap];   // in-kernel selection: lane maxima, survivors of a row
  __shared__ int s_sk[kMaxBeam][kSelCap], s_cnt[kMaxBeam];
  __shared__ int s_cursor, s_iters, s_nT0, s_Btop[kMaxBeam];     // per-utterance state fetched up front
  __shared__ double s_Btopls[kMaxBeam], s_tval[kMaxBeam];         // scores of B's old best / of the entries touched now
  __shared__ int s_sel[kMaxBeam];
  __shared__ int s_keep_h[kMaxBeam], s_keep_k[kMaxBeam], s_keep_slot[kMaxBeam];
  __shared__ double s_keep_ls[kMaxBeam];

  const int b = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // The lists and counters read below were written by the previous pass's kernels, all of which had finished before
  // the joiner kernel that runs ahead of this one began (and that kernel writes none of them): they are fetched
  // before the wait for it, under its tail.  Every first-round load is issued before the early exit, so that none
  // of them waits for H.
  const int H = hs.nA[b];
  const int r0 = hs.row_off[b];
  const int slen = hs.slen[b];
  const int nB0 = hs.nB[b];
  double ld_Als = 0.0, ld_Adone = -INFINITY;
  int ld_Aslot = 0, ld_carry = -1;
  if (tid < kMaxBeam) {                     // all kMaxBeam entries of the lists; those past H are never used
    ld_Als = hs.A_ls[b * kMaxBeam + tid]; ld_Aslot = hs.A_slot[b * kMaxBeam + tid];
    if (hs.mono) ld_Adone = hs.A_done[b * kMaxBeam + tid];
    ld_carry = hs.carry[b * kMaxBeam + tid];
  }
  const long long bB = (long long)b * hs.capB;
  const long long bS = (long long)b * hs.capSlot;
  // the search of list B (warp h looks for hypothesis h's tokens): its own slot and the first 32 entries of the list are
  // asked for now as well; the slot's hash and length follow as soon as the slot is there, still before the barriers
  int my_slot = 0, pre_len = -1, pre_slot = 0;
  unsigned long long pre_hash = 0;
  if (warp < kMaxBeam) {
    my_slot = hs.A_slot[b * kMaxBeam + warp];
    if (lane < hs.capB) { pre_hash = hs.B_hash[bB + lane]; pre_len = hs.B_len[bB + lane]; pre_slot = hs.B_slot[bB + lane]; }
  }
  unsigned long long my_hash = 0;
  int my_len = 0;
  if (warp < H) { my_hash = hs.slot_hash[bS + my_slot]; my_len = hs.slot_len[bS + my_slot]; }
  pdl_wait();                               // from here on: what the joiner kernel wrote (delta_phi, delta_nb, occupancies)
  pdl_trigger();
  if (H == 0) return;                       // idle (finished) utterance
  const int N = hs.N, S = hs.S, V = hs.V;

  if (tid < kMaxBeam) { s_Als[tid] = ld_Als; s_Aslot[tid] = ld_Aslot; s_Adone[tid] = ld_Adone; s_carry[tid] = ld_carry; }
  if (tid == 0) { hs.calls[b] += 1; hs.joins[b] += slen; }
  // With in-kernel selection the CTA has 32 warps: warps 16..31 select (one row each) while warps 0..15 merge the
  // blank expansions into list B and find the threshold; the two halves meet at the barrier before the ranking.
  // Until then the merging half synchronises on a named barrier of its own.
  const bool two_halves = hs.dnb_sel != nullptr;
  auto sync_merge = [&]() {
    if (two_halves) asm volatile("bar.sync 1, 512;" ::: "memory");
    else __syncthreads();
  };
  if (two_halves && warp >= 16) {
    // ---- ChooseNBestExpansions, first stage, for the row of hypothesis warp - 16: its N best tokens by delta_nb,
    // order (value desc, token asc), straight into the candidate table of the second stage.
    const int h = warp - 16;
    if (lane < kMaxBeam) {
      s_abs[h * kMaxBeam + lane] = -INFINITY; s_ck[h * kMaxBeam + lane] = -1; s_key[h * kMaxBeam + lane] = order_key(-INFINITY);
    }
    __syncwarp();
    if (h < H) {
      const float* src = hs.dnb_sel + (long long)(r0 + h) * V;
      const double base = hs.A_ls[b * kMaxBeam + h];
      // a lower bound of the N-th best value: the N-th largest of the 32 lane maxima (distinct elements)
      const int nchunk = V >> 5;
      const float* cmax = (hs.dnb_max != nullptr && (V & 31) == 0 && nchunk <= 128) ? hs.dnb_max + (long long)(r0 + h) * nchunk : nullptr;
      float lmax = 0.f;
      float m4[4] = {0.f, 0.f, 0.f, 0.f};        // with chunk maxima: those of chunks lane, lane + 32, lane + 64, lane + 96
      if (cmax != nullptr) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int c = lane + 32 * u;
          if (c < nchunk) m4[u] = __ldg(cmax + c);
          lmax = fmaxf(lmax, m4[u]);
        }
      } else {
#pragma unroll 8
        for (int k = lane * 4; k < V; k += 128) {             // eight independent loads in flight per lane
          const float4 v = __ldg(reinterpret_cast<const float4*>(src + k));
          lmax = fmaxf(fmaxf(lmax, fmaxf(v.x, v.y)), fmaxf(v.z, v.w));
        }
      }
      s_lm[h][lane] = lmax;
      if (lane == 0) s_cnt[h] = 0;
      __syncwarp();
      int lrank = 0;
#pragma unroll
      for (int j = 0; j < 32; ++j) { const float o = s_lm[h][j]; lrank += (o > lmax || (o == lmax && j < lane)) ? 1 : 0; }
      const unsigned who = __ballot_sync(0xffffffffu, lrank == N - 1);        // exactly one lane: the ranks are 0..31
      const float bound = __shfl_sync(0xffffffffu, lmax, __ffs(who) - 1);
      auto push4 = [&](const float4& v4, int k) {
        const float vv[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          if (vv[c] >= bound && vv[c] > 0.f) {
            const int i = atomicAdd(&s_cnt[h], 1);
            if (i < kSelCap) { s_sv[h][i] = vv[c]; s_sk[h][i] = k + c; }
          }
        }
      };
      if (cmax != nullptr) {
        // Only the chunks whose maximum reaches the bound can hold a survivor: a few 128-byte pieces of the row.  The
        // warp takes them together, a lane per element and up to eight chunks per round, so that their loads (mostly
        // from DRAM: a step moves more than L2 holds) are in flight at the same time.
        unsigned qm[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) qm[u] = __ballot_sync(0xffffffffu, m4[u] >= bound && m4[u] > 0.f);
        int u = 0;
        unsigned m = qm[0];
        for (;;) {
          int ids[8];
          int n = 0;
#pragma unroll
          for (int x = 0; x < 8; ++x) {
            while (m == 0u && u < 3) { ++u; m = (u == 1) ? qm[1] : (u == 2 ? qm[2] : qm[3]); }
            ids[x] = -1;
            if (m != 0u) { ids[x] = (__ffs(m) - 1) + 32 * u; m &= m - 1; ++n; }
          }
          if (n == 0) break;
          float v[8];
#pragma unroll
          for (int x = 0; x < 8; ++x) v[x] = ids[x] >= 0 ? __ldg(src + ids[x] * 32 + lane) : 0.f;
#pragma unroll
          for (int x = 0; x < 8; ++x) {
            if (v[x] >= bound && v[x] > 0.f) {
              const int i = atomicAdd(&s_cnt[h], 1);
              if (i < kSelCap) { s_sv[h][i] = v[x]; s_sk[h][i] = ids[x] * 32 + lane; }
            }
          }
        }
      } else {
        // second sweep (the row is in L2): eight loads at a time, and only a group of four that holds a survivor
        // enters the branch with the shared-memory counter
        for (int k0 = lane * 4; k0 < V; k0 += 8 * 128) {
          float4 v8[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const int k = k0 + u * 128;
            v8[u] = k < V ? __ldg(reinterpret_cast<const float4*>(src + k)) : make_float4(0.f, 0.f, 0.f, 0.f);
          }
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const float g = fmaxf(fmaxf(v8[u].x, v8[u].y), fmaxf(v8[u].z, v8[u].w));
            if (g >= bound && g > 0.f) push4(v8[u], k0 + u * 128);
          }
        }
      }
      __syncwarp();
      const int ns = s_cnt[h];
      if (ns <= kSelCap) {
        for (int i = lane; i < ns; i += 32) {
          const float v = s_sv[h][i]; const int k = s_sk[h][i];
          int rank = 0;
          for (int j = 0; j < ns; ++j) rank += tok_better(s_sv[h][j], s_sk[h][j], v, k) ? 1 : 0;
          if (rank < N) {
            const double sc = base + (double)__logf(v);
            s_abs[h * kMaxBeam + rank] = sc; s_ck[h * kMaxBeam + rank] = k; s_key[h * kMaxBeam + rank] = order_key(sc);
          }
        }
      } else {
        // many ties at the bound: N rounds, each taking the best element after the previous pick in that order
        float pv = INFINITY; int pk = -1;
        for (int j = 0; j < N; ++j) {
          float bv = 0.f; int bk = 0x7fffffff;
          for (int k = lane * 4; k < V; k += 128) {
            const float4 v4 = __ldg(reinterpret_cast<const float4*>(src + k));
            const float vv[4] = {v4.x, v4.y, v4.z, v4.w};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              const bool after = vv[c] < pv || (vv[c] == pv && k + c > pk);
              if (vv[c] > 0.f && after && tok_better(vv[c], k + c, bv, bk)) { bv = vv[c]; bk = k + c; }
            }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int ok = __shfl_xor_sync(0xffffffffu, bk, o);
            if (tok_better(ov, ok, bv, bk)) { bv = ov; bk = ok; }
          }
          if (!(bv > 0.f)) break;
          if (lane == 0) {
            const double sc = base + (double)__logf(bv);
            s_abs[h * kMaxBeam + j] = sc; s_ck[h * kMaxBeam + j] = bk; s_key[h * kMaxBeam + j] = order_key(sc);
          }
          pv = bv; pk = bk;
        }
      }
    }
  }
  if (warp == 15) {
    // ring cursor, pass counter and the best-N set of list B as the previous pass left it: fetched now, by a
    // warp that has nothing to do in the search, so that the later phases find them in shared memory
    const int nT = hs.nTop[b];
    if (lane == 0) { s_cursor = hs.cursor[b]; s_iters = hs.iters[b]; s_nT0 = nT; }
    if (lane < kMaxBeam) {
      const int bt = hs.B_top[b * kMaxBeam + lane];
      s_Btop[lane] = bt;
      if (lane < nT) s_Btopls[lane] = hs.B_ls[bB + bt];       // before this pass's merges; touched entries are patched below
    }
  }
  if (warp < 16) sync_merge();

  // ---- AddAndMerge, search: warp h looks for the tokens of A_h among the entries already in B.
  // (Entries of A are distinct sequences, so two of them never merge with each other.)
  if (warp < H) {
    const int slot = my_slot;
    const unsigned long long hh = my_hash;
    const int ln = my_len;
    const int* ta = hs.slot_tok + (bS + slot) * hs.U_cap;
    int found = -1;
    for (int base = 0; base < nB0 && found < 0; base += 32) {
      const int e = base + lane;
      const bool match = e < nB0 && (base == 0 ? (pre_hash == hh && pre_len == ln)
                                               : (hs.B_hash[bB + e] == hh && hs.B_len[bB + e] == ln));
      unsigned mask = __ballot_sync(0xffffffffu, match);
      while (mask != 0 && found < 0) {
        const int c = base + __ffs(mask) - 1;
        mask &= mask - 1;
        const int oslot = base == 0 ? __shfl_sync(0xffffffffu, pre_slot, c) : hs.B_slot[bB + c];
        int diff = 0;                       // a 64-bit hash match is not proof: compare the tokens
        if (oslot != slot) {
          const int* tb = hs.slot_tok + (bS + oslot) * hs.U_cap;
          for (int i = lane; i < ln; i += 32) diff |= (ta[i] != tb[i]);
        }
        if (!__any_sync(0xffffffffu, diff)) found = c;
      }
    }
    if (lane == 0) { s_found[warp] = found; s_Alen[warp] = ln; }
  }
  if (warp < 16) sync_merge();
  // ---- AddAndMerge, apply: sum into the matching entry or append (appends keep the order of A)
  if (tid < H) {
    const int h = tid;
    const int slot = s_Aslot[h];
    double val = s_Als[h] + (hs.ldphi_d ? hs.ldphi_d[r0 + h] : (double)hs.ldphi[r0 + h]);
    val = logaddexp_d(val, s_Adone[h]);       // monotonic: plus what had already left the segment (else log 0)
    int e = s_found[h];
    if (e >= 0) {
      val = logaddexp_d(hs.B_ls[bB + e], val);
      hs.B_ls[bB + e] = val;
    } else {
      e = nB0;                              // capB = N * I_max bounds this by construction
      for (int q = 0; q < h; ++q) e += (s_found[q] < 0);
      hs.B_slot[bB + e] = slot; hs.B_ls[bB + e] = val;
      hs.B_hash[bB + e] = hs.slot_hash[bS + slot]; hs.B_len[bB + e] = hs.slot_len[bS + slot];
    }
    s_touched[h] = e;
    s_tval[h] = val;
  }
  if (tid == 0) {
    int nB = nB0;
    for (int q = 0; q < H; ++q) nB += (s_found[q] < 0);
    s_nB = nB;
    hs.nB[b] = nB;
  }
  if (warp < 16) sync_merge();

  // ---- ChooseNthScore: the best N of B are among the previous best N and the entries touched now
  if (warp == 0) {
    const int nT = s_nT0;
    int idx = -1;
    double score = -INFINITY;
    if (lane < nT) {
      idx = s_Btop[lane];
      score = s_Btopls[lane];
      for (int q = 0; q < H; ++q) if (s_touched[q] == idx) score = s_tval[q];   // merged into in this pass
    } else if (lane - nT < H) {
      const int cand = s_touched[lane - nT];
      bool dup = false;
      for (int i = 0; i < nT; ++i) dup |= (s_Btop[i] == cand);
      if (!dup) { idx = cand; score = s_tval[lane - nT]; }
    }
    const unsigned long long key = order_key(score);
    s_nkey[lane] = key; s_nidx[lane] = idx;
    __syncwarp();
    int rank = 0;
#pragma unroll
    for (int j = 0; j < 32; ++j) {          // all lanes read the same word: broadcasts, independent of each other
      const unsigned long long kj = s_nkey[j];
      const int ij = s_nidx[j];
      rank += (ij >= 0 && (kj > key || (kj == key && ij < idx))) ? 1 : 0;
    }
    const int count = __popc(__ballot_sync(0xffffffffu, idx >= 0));
    __syncwarp();
    if (idx >= 0 && rank < N) hs.B_top[b * kMaxBeam + rank] = idx;
    if (idx >= 0 && rank == N - 1) s_thr = score;
    if (lane == 0) { hs.nTop[b] = min(N, count); s_hasthr = (count >= N); }
  }
  // ---- ChooseNBestExpansions, second stage: the N best (h, k) over the rows' candidate lists, in
  // float64; order (score desc, h asc, k asc).  The lists are sorted by (score desc, k asc).
  if (hs.dnb_sel == nullptr && tid < kMaxBeam * kMaxBeam) {
    const int h = tid / kMaxBeam, j = tid % kMaxBeam;
    const bool valid = h < H && j < hs.cand_n[r0 + h];
    s_abs[tid] = valid ? s_Als[h] + (double)hs.cand_v[(long long)(r0 + h) * kMaxBeam + j] : -INFINITY;
    s_ck[tid] = valid ? hs.cand_k[(long long)(r0 + h) * kMaxBeam + j] : -1;
    s_key[tid] = order_key(s_abs[tid]);
  }
  if (tid < kMaxBeam) s_sel[tid] = -1;
  __syncthreads();
  if (tid < kMaxBeam * kMaxBeam && s_ck[tid] >= 0) {
    const unsigned long long mine = s_key[tid];
    const int h = tid / kMaxBeam, jj = tid % kMaxBeam;
    // Rank = how many candidates come before this one in the order (score desc, h asc, k asc).  Every row's list is
    // sorted that way and padded with the key of log 0, so the candidates of a row that come before this one are a
    // prefix of its list: its length is found by bisection (four probes and a last one for a full list) instead of
    // a look at all sixteen entries.  Rows before h count their ties with this score, rows after it do not, and in
    // its own row exactly the jj entries ahead of it count.
    int rank = jj;
    for (int hh = 0; hh < H; ++hh) {
      if (hh == h) continue;
      const unsigned long long* key = s_key + hh * kMaxBeam;
      const bool ties = hh < h;
      int cnt = 0;
#pragma unroll
      for (int st = kMaxBeam / 2; st > 0; st >>= 1) {
        const unsigned long long so = key[cnt + st - 1];
        if (so > mine || (ties && so == mine)) cnt += st;
      }
      if (cnt == kMaxBeam - 1) { const unsigned long long so = key[cnt]; cnt += (so > mine || (ties && so == mine)) ? 1 : 0; }
      rank += cnt;
    }
    if (rank < N) s_sel[rank] = tid;
  }
  __syncthreads();
  const bool hasthr = s_hasthr != 0;
  const double thr = hasthr ? s_thr : -INFINITY;

  // ---- filter against the threshold, allocate slots: lane i of warp 0 takes the i-th best expansion
  if (warp == 0) {
    const int c = lane < N ? s_sel[lane] : -1;
    const int h = c >= 0 ? c / kMaxBeam : 0;
    const double sc = c >= 0 ? s_abs[c] : -INFINITY;
    const bool pass = c >= 0 && (!hasthr || sc > thr);      // Length(B) < N or delta_nb > threshold
    const bool capped = s_iters + 1 >= hs.I_max;
    const bool fits = s_Alen[h] + 1 <= hs.U_cap;
    const bool keep = pass && !capped && fits;
    const unsigned passm = __ballot_sync(0xffffffffu, pass), keepm = __ballot_sync(0xffffffffu, keep);
    const int nk = __popc(keepm), m = __popc(keepm & ((1u << lane) - 1u));
    if (keep) {
      // the (m + 1)-th free slot of the ring after the cursor: slots still held by hypotheses carried into
      // this segment are skipped
      int cur = s_cursor, need = m + 1;
      while (need > 0) {
        cur = (cur + 1 == hs.capSlot) ? 0 : cur + 1;
        bool busy = false;
#pragma unroll
        for (int q = 0; q < kMaxBeam; ++q) busy |= (s_carry[q] == cur);
        if (!busy) --need;
      }
      s_keep_h[m] = h; s_keep_k[m] = s_ck[c]; s_keep_ls[m] = sc; s_keep_slot[m] = cur;
      if (m == nk - 1) hs.cursor[b] = cur;
    }
    if (lane == 0) {
      hs.iters[b] = s_iters + 1;
      if (passm != 0 && (capped || (passm & ~keepm) != 0)) hs.status[b] = TW_ERR_LIMIT;   // pass cap or token capacity
      s_nkeep = nk;
      hs.nA[b] = nk; hs.n_new[b] = nk;
      s_wbase = (hs.inline_gather && nk > 0) ? atomicAdd(&hs.scalars[kScNPred], nk) : 0;   // this utterance's work-list entries
    }
  }
  __syncthreads();
  const int nk = s_nkeep;

  // ---- new list A (one warp per kept expansion): tokens, hash, frame distribution d_h(k) (Eq. 5)
  if (warp < nk) {
    const int i = warp;
    const int h = s_keep_h[i], k = s_keep_k[i];
    const long long gp = bS + s_Aslot[h], gn = bS + s_keep_slot[i];
    const int plen = hs.slot_len[gp];
    const int* src = hs.slot_tok + gp * hs.U_cap;
    int* dst = hs.slot_tok + gn * hs.U_cap;
    for (int q = lane; q < plen; q += 32) dst[q] = src[q];
    if (lane == 0) {
      dst[plen] = k;
      hs.slot_len[gn] = plen + 1;
      hs.slot_hash[gn] = hash_push(hs.slot_hash[gp], k);
      hs.new_slot[b * kMaxBeam + i] = (int)gn;
      hs.new_par[b * kMaxBeam + i] = (int)gp;
      hs.new_tok[b * kMaxBeam + i] = k;
      hs.new_row[b * kMaxBeam + i] = r0 + h;
      hs.A_slot[b * kMaxBeam + i] = s_keep_slot[i];
      hs.A_ls[b * kMaxBeam + i] = s_keep_ls[i];
    }
    if (hs.inline_gather && lane == 0) {           // the predictor's work-list entry of this hypothesis
      if (hs.pf_table != nullptr) sm100::prefetch_l2_bulk(hs.pf_table + (long long)k * hs.pf_row_bytes, (uint32_t)hs.pf_row_bytes);
      if ((hs.Hd & 3) == 0) {
        const float* pc = hs.slot_hc + gp * ((long long)hs.L * 2 * hs.Hd) + hs.Hd;      // the parent's c, layer by layer
        for (int l = 0; l < hs.L; ++l) sm100::prefetch_l2_bulk(pc + (long long)l * 2 * hs.Hd, (uint32_t)hs.Hd * 4u);
      }
      const int wrow = s_wbase + i;
      if (wrow < hs.B * hs.N) { hs.pw_new[wrow] = (int)gn; hs.pw_par[wrow] = (int)gp; hs.pw_tok[wrow] = k; }
      else hs.status[b] = TW_ERR_LIMIT;            // cannot happen: the list holds at most N entries per utterance
    }
    const long long r = r0 + h;
    // d_h(k) at frame t of the segment: occupancy times J(t, k)
    auto d_at = [&](int t) -> double {
      if (t < 0 || t >= slen) return -INFINITY;
      const double a = hs.la_d ? hs.la_d[r * S + t] : (double)hs.la[r * S + t];
      double v = s_Als[h] + a;
      if (hs.logp != nullptr) {      // otherwise log J(t, k) is added by a follow-up kernel
        double lj = (double)hs.logp[(r * S + t) * V + k];
        if (hs.lse) lj -= (double)hs.lse[r * S + t];
        v += lj;
      }
      return v;
    };
    if (!hs.mono) {
      for (int t = lane; t < S; t += 32) hs.A_ld[((long long)b * kMaxBeam + i) * S + t] = d_at(t);
    } else {
      // emitted at frame t: the hypothesis continues at frame t + 1, or has left the segment
      for (int t = lane; t < S; t += 32) hs.A_ld[((long long)b * kMaxBeam + i) * S + t] = t < slen ? d_at(t - 1) : -INFINITY;
      if (lane == 0) hs.A_done[b * kMaxBeam + i] = d_at(slen - 1);
    }
  }
  // ---- the parents' h of every layer as bf16 in the recurrent halves of the gate GEMMs' operand rows (all threads:
  // 16-byte pieces, independent of each other)
  if (hs.inline_gather && nk > 0 && s_wbase + nk <= hs.B * hs.N) {
    const long long stride = (long long)hs.L * 2 * hs.Hd;
    const bool vec = (hs.Hd & 7) == 0 && (reinterpret_cast<uintptr_t>(hs.slot_hc) & 15) == 0;
    const int per = vec ? hs.Hd >> 3 : hs.Hd;                 // pieces per (hypothesis, layer)
    const int total = nk * hs.L * per;
    for (int c = threadIdx.x; c < total; c += blockDim.x) {
      const int i = c / (hs.L * per), rem = c - i * (hs.L * per), l = rem / per, x = rem - l * per;
      const long long gp = bS + s_Aslot[s_keep_h[i]];
      const float* hsrc = hs.slot_hc + gp * stride + (long long)l * 2 * hs.Hd;
      __nv_bfloat16* d = reinterpret_cast<__nv_bfloat16*>(hs.xg_dst[l]) + (long long)(s_wbase + i) * hs.xg_ld[l] + hs.xg_off[l];
      if (vec && (reinterpret_cast<uintptr_t>(d) & 15) == 0) {
        const float4 a = *reinterpret_cast<const float4*>(hsrc + x * 8), e = *reinterpret_cast<const float4*>(hsrc + x * 8 + 4);
        __nv_bfloat162 p0 = __floats2bfloat162_rn(a.x, a.y), p1 = __floats2bfloat162_rn(a.z, a.w);
        __nv_bfloat162 p2 = __floats2bfloat162_rn(e.x, e.y), p3 = __floats2bfloat162_rn(e.z, e.w);
        uint4 pk;
        pk.x = *reinterpret_cast<uint32_t*>(&p0); pk.y = *reinterpret_cast<uint32_t*>(&p1);
        pk.z = *reinterpret_cast<uint32_t*>(&p2); pk.w = *reinterpret_cast<uint32_t*>(&p3);
        *reinterpret_cast<uint4*>(d + x * 8) = pk;
      } else if (vec) {
        for (int u = 0; u < 8; ++u) d[x * 8 + u] = __float2bfloat16_rn(hsrc[x * 8 + u]);
      } else {
        d[x] = __float2bfloat16_rn(hsrc[x]);
      }
    }
  }
  // ---- list A empty: this segment is done ------------------------------------------------------
  if (nk == 0 && hs.t0[b] + slen < hs.len[b]) turn_over(hs, b);
}

// One CTA: packs the live hypotheses of all utterances into joiner rows and the new hypotheses
// into the predictor's work list.
__global__ void __launch_bounds__(1024) compact_kernel(HypState hs, int B, int T) {
  __shared__ int s_wa[32], s_wn[32];       // per-warp totals of the two scans
  __shared__ int s_cnt[1024], s_off[1024]; // batches of up to 1024 utterances: nA | n_new << 8, row_off | new_off << 16 kept on chip
  __shared__ int s_base_a, s_base_n, s_frames;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_wait();
  pdl_trigger();
  if (tid == 0) { s_base_a = 0; s_base_n = 0; s_frames = 0; }
  __syncthreads();
  // exclusive scans of the list sizes -> row_off, new_off (shuffle scan per warp, then over the warp totals)
  for (int b0 = 0; b0 < B; b0 += 1024) {
    const int b = b0 + tid;
    const int a = b < B ? hs.nA[b] : 0;
    const int nn = b < B ? hs.n_new[b] : 0;
    const int fr = (b < B && a > 0) ? a * hs.slen[b] : 0;
    int ia = a, in = nn;                   // inclusive scans inside the warp
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int va = __shfl_up_sync(0xffffffffu, ia, o), vn = __shfl_up_sync(0xffffffffu, in, o);
      if (lane >= o) { ia += va; in += vn; }
    }
    if (lane == 31) { s_wa[warp] = ia; s_wn[warp] = in; }
    if (fr > 0) atomicAdd(&s_frames, fr);
    __syncthreads();
    int pa = 0, pn = 0;                    // totals of the warps before this one
    for (int w = 0; w < warp; ++w) { pa += s_wa[w]; pn += s_wn[w]; }
    if (b < B) {
      hs.row_off[b] = s_base_a + pa + ia - a;
      hs.new_off[b] = s_base_n + pn + in - nn;
      if (B <= 1024) { s_cnt[tid] = a | (nn << 8); s_off[tid] = (pa + ia - a) | ((pn + in - nn) << 16); }
    }
    __syncthreads();
    if (tid == 1023) { s_base_a += pa + ia; s_base_n += pn + in; }
    __syncthreads();
  }
  // fill: one thread per (utterance, list position)
  for (int idx = tid; idx < B * kMaxBeam; idx += 1024) {
    const int b = idx / kMaxBeam, h = idx % kMaxBeam;
    const bool chip = B <= 1024;           // offsets fit 16 bits: at most 1024 * kMaxBeam rows
    const int nA_b = chip ? (s_cnt[b] & 255) : hs.nA[b], nnew_b = chip ? (s_cnt[b] >> 8) : hs.n_new[b];
    if (h < nA_b && !hs.defer_rows) {
      const int r = (chip ? (s_off[b] & 0xffff) : hs.row_off[b]) + h;
      const int slot = hs.A_slot[b * kMaxBeam + h];
      const long long gs = (long long)b * hs.capSlot + slot;
      hs.row_b[r] = b;
      hs.row_e0[r] = b * T + hs.t0[b];
      hs.row_slen[r] = hs.slen[b];
      if (hs.stateless) {
        const int ln = hs.slot_len[gs];
        hs.row_p[r] = ln > 0 ? hs.slot_tok[gs * hs.U_cap + ln - 1] : hs.empty_row;
      } else {
        hs.row_p[r] = (int)gs;
      }
      const double ls = hs.A_ls[b * kMaxBeam + h];
      for (int t = 0; t < hs.S; ++t) {
        const double d = hs.A_ld[((long long)b * kMaxBeam + h) * hs.S + t];
        hs.row_ld[(long long)r * hs.S + t] = (d == -INFINITY) ? -INFINITY : (float)(d - ls);
      }
    }
    if (h < nnew_b) {
      const int o = (chip ? (s_off[b] >> 16) : hs.new_off[b]) + h;
      hs.pw_new[o] = hs.new_slot[b * kMaxBeam + h];
      hs.pw_par[o] = hs.new_par[b * kMaxBeam + h];
      hs.pw_tok[o] = hs.new_tok[b * kMaxBeam + h];
    }
  }
  __syncthreads();
  if (!hs.defer_rows) for (int b = tid; b < B; b += 1024) hs.n_new[b] = 0;
  if (tid == 0) {
    const int R = s_base_a;
    hs.scalars[kScR] = R;
    hs.scalars[kScM] = R * hs.S;
    hs.scalars[kScNPred] = s_base_n;
    hs.scalars[kScActive] = R > 0;
    if (R > 0) { hs.scalars[kScSteps] += 1; hs.rows_total[0] += R; hs.rows_total[1] += s_frames; }
  }
}

__global__ void stream_rows_kernel(HypState hs, const int* chunk_lens, int B, int Tc, int max_T, int dump_row, int* oidx) {
  const int m = blockIdx.x * blockDim.x + threadIdx.x;
  if (m >= B * Tc) return;
  const int b = m / Tc, i = m - b * Tc;
  const int have = hs.avail[b];
  const bool ok = i < chunk_lens[b] && have + i < max_T;
  oidx[m] = ok ? b * max_T + have + i : dump_row;
}

__global__ void __launch_bounds__(kThreads) stream_advance_kernel(HypState hs, const int* chunk_lens, int max_T, int closing) {
  const int b = blockIdx.x;
  __shared__ int s_go;
  if (threadIdx.x == 0) {
    int add = chunk_lens ? max(chunk_lens[b], 0) : 0;
    int have = hs.avail[b];
    if (have + add > max_T) { add = max_T - have; hs.status[b] = TW_ERR_LIMIT; }
    have += add;
    hs.avail[b] = have;
    const int len = closing ? have : (have / hs.S) * hs.S;    // only whole segments while the stream is open
    hs.len[b] = len;
    s_go = (hs.nA[b] == 0 && hs.t0[b] + hs.slen[b] < len);
  }
  __syncthreads();
  if (s_go) turn_over(hs, b);
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
  if (B > 0) launch_pdl(hyp_step_kernel, dim3(B), dim3(hs.dnb_sel ? 2 * kStepThreads : kStepThreads), 0, st, hs);
}
void launch_compact(const HypState& hs, int B, int T, cudaStream_t st) {
  launch_pdl(compact_kernel, dim3(1), dim3(1024), 0, st, hs, B, T);
}
void launch_stream_rows(const HypState& hs, const int* chunk_lens, int B, int Tc, int max_T, int dump_row,
                        int* oidx, cudaStream_t st) {
  const int n = B * Tc;
  if (n > 0) stream_rows_kernel<<<(n + 255) / 256, 256, 0, st>>>(hs, chunk_lens, B, Tc, max_T, dump_row, oidx);
}
void launch_stream_advance(const HypState& hs, const int* chunk_lens, int B, int max_T, int closing,
                           cudaStream_t st) {
  if (B > 0) stream_advance_kernel<<<B, kThreads, 0, st>>>(hs, chunk_lens, max_T, closing);
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
