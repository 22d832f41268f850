// Vocab softmax statistics, accept/reject scan, residual / bonus sampling: ONE launch.
//
// The grid is made of thread-block clusters of `team` CTAs (1, 2, 4 or 8) of 1024 threads, one CTA per SM.
//   The first cluster of a sequence is its TAIL TEAM; the clusters behind it hold the statistics CTAs.
//   statistics CTAs: one coalesced pass over all (2*gamma+1) logit rows, a contiguous chunk of one row each ->
//     (max, sum exp) of the chunk in the workspace, then one atomic count per sequence.  Few, fat CTAs: with the
//     cluster launch at most 15 clusters of 8 such CTAs are resident at once, so the chunk size is chosen to fit
//     every CTA of a single-sequence call into one wave (100 CTAs at the 152k vocabulary with gamma = 12).
//   the team waits (bounded) until the count says every partial is written and then runs the whole
//     latency-bound tail without another launch and without another trip through global memory:
//       row merge   : every team CTA merges all rows' partials -> lse per row (redundantly: cheaper than a hand-over)
//       accept scan : p(x_t), q(x_t); first rejection n
//       residual    : the weights max(0, p_n - q_n) (or p_n: bonus token, plain sampling) over the team's share of
//                     the vocabulary: warp-contiguous ranges, all loads of a lane in flight at once, the lane sums of
//                     each 128-entry step kept in registers
//       exchange    : every CTA stores its total into every team member's shared memory, one cluster barrier
//       pick        : the CTA, warp, step, lane and element where the running sum crosses u * Z
// The wait cannot deadlock: it only needs the statistics CTAs to be dispatched, the team occupies at most 8 of the
// 148 SMs, and statistics CTAs never wait.  It is bounded anyway.
//
// Precision: row statistics in fp32 (ex2.approx), lse through an fp64 log.  The residual weights are evaluated in
// fp32 relative to the row maximum (exponent = (x - max) * c - log2(sum), the last term carried as two floats), so
// their relative error is a few 1e-7 and random; sums and the running prefix are fp64.  The drawn token equals the
// fp64 reference's except where u * Z falls within ~1e-6 * Z of a step of the cumulative sum.
#include "pvlm_common.cuh"

#include <cooperative_groups.h>

namespace pvlm {

namespace {

namespace cg = cooperative_groups;

constexpr int kAccThreads = 1024;
constexpr int kAccWarps = kAccThreads / 32;
constexpr int kStatGrain = 4096;     // a statistics chunk is a multiple of this (one float4 per thread)
constexpr int kStatBudget = 104;     // statistics CTAs of one call that fit one wave beside the team (13 clusters of 8)
constexpr int kTeamMax = 8;          // CTAs of the tail team (one portable cluster)
constexpr int kWarpSpan = 128;       // elements a warp covers per step of the residual pass (float4 per lane)
constexpr int kRegIt = 5;            // steps of a warp's range whose loads are in flight together and whose lane sums stay in registers
constexpr unsigned long long kTeamWaitLimitNs = 1000000000ull;   // a second: the statistics pass takes microseconds

struct AccArgs {
  const float *tl, *dl;
  long long trs, drs, tbs, dbs;
  const int* tok;
  const float* u;
  int batch, gamma, V, rows;
  int vec_ok;         // rows are 16-byte aligned: float4 loads allowed
  float inv_temp;
  int* n_accept;
  int* out_tokens;
  float *p_tok, *q_tok, *lse_p, *lse_q, *probs_p, *probs_q;
  float2* stats;      // [batch][rows][n_stat_chunks]  (max of raw logits, sum exp((x-max)/temp))
  double* lse;        // [batch][rows]   (written by team CTA 0; read by the full-probability kernel)
  int* sync;          // [batch] statistics CTAs finished (zeroed per call)
  int n_stat_chunks;  // statistics CTAs per row
  int stat_chunk;     // elements per statistics CTA (a multiple of kStatGrain)
  int team;           // CTAs of the tail team = cluster size: 1, 2, 4 or 8
  int nit;            // steps per warp range: the team's warps cover nit * kWarpSpan elements each
};

__device__ __forceinline__ const float* row_ptr(const AccArgs& a, int b, int row) {
  return row <= a.gamma ? a.tl + (long long)b * a.tbs + (long long)row * a.trs
                        : a.dl + (long long)b * a.dbs + (long long)(row - a.gamma - 1) * a.drs;
}

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}

// merge two (max, sum) pairs; c = log2(e) / temperature
__device__ __forceinline__ void merge_ml(float& m, float& l, float m2, float l2, float c) {
  const float mn = fmaxf(m, m2);
  if (mn == -INFINITY) { m = mn; l = 0.f; return; }
  l = l * ex2f((m - mn) * c) + l2 * ex2f((m2 - mn) * c);
  m = mn;
}

// The accept test of one drafted token (paper Sec. 2.2: accept with probability min{1, p/q}), division-free:
// one rounded fp32 multiply, strict compare.  u in [0,1): a ratio >= 1 always accepts, p = 0 never does.
__device__ __forceinline__ bool accept_test(float u, float p, float q) { return __fmul_rn(u, q) < p; }

__device__ __forceinline__ double warp_sum_d(double v) {     // butterfly: every lane ends with the same bits
#pragma unroll
  for (int sh = 16; sh >= 1; sh >>= 1) v += __shfl_xor_sync(0xffffffffu, v, sh);
  return v;
}
__device__ __forceinline__ int warp_max_i(int v) {
#pragma unroll
  for (int sh = 16; sh >= 1; sh >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, sh));
  return v;
}

// Per-row constants of the residual pass: exponent of entry x is (x - m) * c - (d_hi + d_lo) in log2 units.
struct RowExp {
  const float* x;
  float m, d_hi, d_lo;
};

// Four consecutive logits starting at i (-inf beyond V).
__device__ __forceinline__ float4 load4(const AccArgs& a, const float* row, long long i) {
  if (a.vec_ok && i + 3 < a.V) return __ldg(reinterpret_cast<const float4*>(row + i));
  float4 t;
  t.x = (i + 0 < a.V) ? __ldg(row + i + 0) : -INFINITY;
  t.y = (i + 1 < a.V) ? __ldg(row + i + 1) : -INFINITY;
  t.z = (i + 2 < a.V) ? __ldg(row + i + 2) : -INFINITY;
  t.w = (i + 3 < a.V) ? __ldg(row + i + 3) : -INFINITY;
  return t;
}

// Weights of four consecutive vocabulary entries from their logits: mode 0 = max(0, p - q), 1 = p; 0 for -inf logits.
__device__ __forceinline__ void weights_of(const float4 xp4, const float4 xq4, const RowExp& rp, const RowExp& rq, int mode,
                                           float c, float (&w)[4]) {
  const float xp[4] = {xp4.x, xp4.y, xp4.z, xp4.w}, xq[4] = {xq4.x, xq4.y, xq4.z, xq4.w};
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float yp = fmaf(xp[e] - rp.m, c, -rp.d_hi) - rp.d_lo;
    const float p = ex2f(yp);
    if (mode == 0) {
      const float yq = fmaf(xq[e] - rq.m, c, -rq.d_hi) - rq.d_lo;
      const float q = ex2f(yq);
      w[e] = fmaxf(0.f, p - q);
    } else {
      w[e] = p;
    }
  }
}

__device__ __forceinline__ void weights4(const AccArgs& a, const RowExp& rp, const RowExp& rq, int mode, long long i, float c,
                                         float (&w)[4]) {
  const float4 xp4 = load4(a, rp.x, i);
  const float4 xq4 = mode == 0 ? load4(a, rq.x, i) : make_float4(0.f, 0.f, 0.f, 0.f);
  weights_of(xp4, xq4, rp, rq, mode, c, w);
}

// ---------------------------------------------------------------------------------------------------------
// The tail team.  Called by all threads of the team's CTAs (blockIdx.x = rank in the cluster).
// ---------------------------------------------------------------------------------------------------------
__device__ void team_body(const AccArgs& a, const int b) {
  cg::cluster_group cluster = cg::this_cluster();
  const int rank = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = a.gamma;
  const float c = a.inv_temp * kLog2e;
  __shared__ double s_lse[2 * 64 + 1];       // natural-log lse per row
  __shared__ double s_l2[2 * 64 + 1];        // log2 of the row's sum of exponentials relative to its maximum
  __shared__ float s_m[2 * 64 + 1];          // row maximum (raw logits)
  __shared__ unsigned s_rej[2];
  __shared__ int s_ok;
  __shared__ double s_wtot[kAccWarps];
  __shared__ int s_wlast[kAccWarps];
  // one slot per team member and attempt, written by that member into EVERY member's copy (distributed shared memory)
  __shared__ double s_team_tot[2][kTeamMax];
  __shared__ int s_team_last[2][kTeamMax], s_team_ok[2][kTeamMax];

  // ---- before the wait: what the scan needs of the call's own inputs ----
  int x = -1;
  float xp = 0.f, xq = 0.f, ut = 0.f;
  if (tid < g) {
    x = a.tok[(long long)b * g + tid];
    ut = a.u[(long long)b * (g + 1) + tid];
    if (x >= 0 && x < a.V) {
      xp = row_ptr(a, b, tid)[x];
      xq = row_ptr(a, b, g + 1 + tid)[x];
    }
  }
  const float u_draw = a.u[(long long)b * (g + 1) + g];
  // ---- wait until every statistics CTA of this sequence has published its partial ----
  if (tid == 0) {
    const int total = a.rows * a.n_stat_chunks;
    const int* cnt = a.sync + b;
    unsigned long long t0;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    int ok = 0;
    for (;;) {
      int v;
      asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(cnt) : "memory");
      if (v >= total) { ok = 1; break; }
      __nanosleep(20);
      unsigned long long t1;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
      if (t1 - t0 > kTeamWaitLimitNs) break;
    }
    s_ok = ok;
  }
  __syncthreads();
  const bool ok = s_ok != 0;
  int n = 0;
  if (ok) {
    // ---- row merge: a warp per row, lanes over the row's chunk partials, fixed merge order ----
    for (int row = warp; row < a.rows; row += kAccWarps) {
      float m = -INFINITY, l = 0.f;
      const float2* st = a.stats + ((long long)b * a.rows + row) * a.n_stat_chunks;
      for (int ch = lane; ch < a.n_stat_chunks; ch += 32) {
        const float2 v = __ldcg(st + ch);                 // other CTAs wrote it: read through L2
        merge_ml(m, l, v.x, v.y, c);
      }
#pragma unroll
      for (int sh = 16; sh >= 1; sh >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, sh), l2 = __shfl_xor_sync(0xffffffffu, l, sh);
        merge_ml(m, l, m2, l2, c);
      }
      if (lane == 0) {
        const double ln_l = log((double)l);
        s_m[row] = m;
        s_l2[row] = ln_l * 1.4426950408889634;
        s_lse[row] = (double)m * (double)a.inv_temp + ln_l;
      }
    }
    __syncthreads();
    // ---- accept scan ----
    bool rej = false;
    if (tid < g) {
      float p = 0.f, q = 1.f;
      if (x >= 0 && x < a.V) {
        p = (float)exp((double)xp * (double)a.inv_temp - s_lse[tid]);
        q = (float)exp((double)xq * (double)a.inv_temp - s_lse[g + 1 + tid]);
      }
      if (rank == 0) {
        if (a.p_tok) a.p_tok[(long long)b * g + tid] = p;
        if (a.q_tok) a.q_tok[(long long)b * g + tid] = q;
      }
      rej = !accept_test(ut, p, q);
    }
    if (warp < 2) {
      const unsigned bal = __ballot_sync(0xffffffffu, rej);
      if (lane == 0) s_rej[warp] = bal;
    }
    __syncthreads();
    n = s_rej[0] ? __ffs(s_rej[0]) - 1 : (s_rej[1] ? 32 + __ffs(s_rej[1]) - 1 : g);
    if (rank == 0) {
      if (tid == 0) a.n_accept[b] = n;
      int* out = a.out_tokens + (long long)b * (g + 1);
      if (tid <= g && tid != n) out[tid] = (tid < n) ? a.tok[(long long)b * g + tid] : -1;      // out[n] is the drawn token's
      if (tid < a.rows) {
        const double lse = s_lse[tid];
        a.lse[(long long)b * a.rows + tid] = lse;
        if (tid <= g) { if (a.lse_p) a.lse_p[(long long)b * (g + 1) + tid] = (float)lse; }
        else if (a.lse_q) a.lse_q[(long long)b * g + tid - g - 1] = (float)lse;
      }
    }
  }

  // ---- residual pass, exchange, pick; run a second time with weights p_n if the residual has no weight at all ----
  const long long w_start = ((long long)rank * kAccWarps + warp) * a.nit * kWarpSpan + lane * 4;
  int mode = (n < g) ? 0 : 1;
  for (int attempt = 0; attempt < 2; ++attempt) {
    RowExp rp = {}, rq = {};
    double s_it[kRegIt];
    double lane_tot = 0.0;
    int lane_last = -1;
#pragma unroll
    for (int j = 0; j < kRegIt; ++j) s_it[j] = 0.0;
    if (ok) {
      rp.x = row_ptr(a, b, n);
      rp.m = s_m[n];
      rp.d_hi = (float)s_l2[n];
      rp.d_lo = (float)(s_l2[n] - (double)rp.d_hi);
      if (mode == 0) {
        const int rq_row = g + 1 + n;
        rq.x = row_ptr(a, b, rq_row);
        rq.m = s_m[rq_row];
        rq.d_hi = (float)s_l2[rq_row];
        rq.d_lo = (float)(s_l2[rq_row] - (double)rq.d_hi);
      }
      {
        // the first kRegIt steps: every load is issued before the first exponential
        const float4 none = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        float4 xp4[kRegIt], xq4[kRegIt];
#pragma unroll
        for (int j = 0; j < kRegIt; ++j) {
          const long long i = w_start + (long long)j * kWarpSpan;
          const bool live = j < a.nit && i < a.V;
          xp4[j] = live ? load4(a, rp.x, i) : none;
          xq4[j] = (live && mode == 0) ? load4(a, rq.x, i) : none;
        }
#pragma unroll
        for (int j = 0; j < kRegIt; ++j) {
          const long long i = w_start + (long long)j * kWarpSpan;
          float w[4];
          weights_of(xp4[j], xq4[j], rp, rq, mode, c, w);
          s_it[j] = (double)((w[0] + w[1]) + (w[2] + w[3]));     // four fp32 terms, then fp64 (conversions are scarce)
#pragma unroll
          for (int e = 0; e < 4; ++e) if (w[e] > 0.f) lane_last = (int)i + e;
          lane_tot += s_it[j];
        }
      }
      for (int it = kRegIt; it < a.nit; ++it) {           // very large vocabularies only
        const long long i = w_start + (long long)it * kWarpSpan;
        if (i < a.V) {
          float w[4];
          weights4(a, rp, rq, mode, i, c, w);
          lane_tot += (double)((w[0] + w[1]) + (w[2] + w[3]));
#pragma unroll
          for (int e = 0; e < 4; ++e) if (w[e] > 0.f) lane_last = (int)i + e;
        }
      }
    }
    const double wtot = warp_sum_d(lane_tot);
    const int wlast = warp_max_i(lane_last);
    if (attempt) __syncthreads();                         // the slots below may still be read from the first attempt
    if (lane == 0) { s_wtot[warp] = wtot; s_wlast[warp] = wlast; }
    __syncthreads();
    // inclusive scan of the warp totals, computed alike by every warp (lane l stands for warp l)
    double wincl = s_wtot[lane];
#pragma unroll
    for (int sh = 1; sh < 32; sh <<= 1) {
      const double t = __shfl_up_sync(0xffffffffu, wincl, sh);
      if (lane >= sh) wincl += t;
    }
    const double cta_tot = __shfl_sync(0xffffffffu, wincl, 31);
    if (warp == 0) {
      const int cta_last = warp_max_i(s_wlast[lane]);
      if (lane < a.team) {                                // lane r stores this CTA's slot into member r's shared memory
        *cluster.map_shared_rank(&s_team_tot[attempt][rank], lane) = cta_tot;
        *cluster.map_shared_rank(&s_team_last[attempt][rank], lane) = cta_last;
        *cluster.map_shared_rank(&s_team_ok[attempt][rank], lane) = ok ? 1 : 0;
      }
    }
    cluster.sync();                                       // every member's slots are complete; nobody writes them again
    double z = 0.0, before = 0.0;
    int all_ok = 1, z_last = -1;
#pragma unroll
    for (int r = 0; r < kTeamMax; ++r) {
      if (r < a.team) {
        if (r == rank) before = z;
        z += s_team_tot[attempt][r];
        z_last = max(z_last, s_team_last[attempt][r]);
        all_ok &= s_team_ok[attempt][r];
      }
    }
    if (!all_ok) {                                        // an expired wait somewhere in the team: no token
      if (rank == 0 && tid == 0 && ok) a.out_tokens[(long long)b * (g + 1) + n] = -1;
      return;
    }
    if (mode == 0 && !(z > 0.0)) { mode = 1; continue; }   // no residual weight at all (p == q numerically): draw from p_n
    const double target = (double)u_draw * z;
    int* out = a.out_tokens + (long long)b * (g + 1) + n;
    // the CTA whose share holds the crossing: the first whose inclusive prefix exceeds the target
    // (the last CTA also takes a target that rounding pushed past the total)
    const bool here = target >= before && (target < before + cta_tot || rank == a.team - 1);
    if (!here) return;
    // warp: the first whose inclusive prefix exceeds the target
    const unsigned wcross = __ballot_sync(0xffffffffu, before + wincl > target);
    if (!wcross) {                                        // rounding left no crossing: the last token with weight
      if (warp == 0) {
        const int cta_last = warp_max_i(s_wlast[lane]);
        if (lane == 0) *out = cta_last >= 0 ? cta_last : z_last;
      }
      return;
    }
    const int wsel = __ffs(wcross) - 1;
    if (warp != wsel) return;
    double run = before + __shfl_sync(0xffffffffu, wincl - s_wtot[lane], wsel);
    // step: totals of the registered steps (butterfly sums: identical in every lane)
    double t_it[kRegIt];
#pragma unroll
    for (int j = 0; j < kRegIt; ++j) t_it[j] = warp_sum_d(s_it[j]);
    int it_sel = -1;
    double sel = 0.0;
#pragma unroll
    for (int j = 0; j < kRegIt; ++j) {
      if (j < a.nit && it_sel < 0) {
        if (run + t_it[j] > target) { it_sel = j; sel = s_it[j]; }
        else run += t_it[j];
      }
    }
    for (int it = kRegIt; it < a.nit && it_sel < 0; ++it) {     // beyond the registered steps: recompute
      const long long i = w_start + (long long)it * kWarpSpan;
      double sm = 0.0;
      if (i < a.V) {
        float w[4];
        weights4(a, rp, rq, mode, i, c, w);
        sm = (double)((w[0] + w[1]) + (w[2] + w[3]));
      }
      const double t = warp_sum_d(sm);
      if (run + t > target) { it_sel = it; sel = sm; }
      else run += t;
    }
    const int fallback = s_wlast[wsel] >= 0 ? s_wlast[wsel] : z_last;
    if (it_sel < 0) {
      if (lane == 0) *out = fallback;
      return;
    }
    // lane: inclusive scan of the lanes' sums of that step
    double incl = sel;
#pragma unroll
    for (int sh = 1; sh < 32; sh <<= 1) {
      const double t = __shfl_up_sync(0xffffffffu, incl, sh);
      if (lane >= sh) incl += t;
    }
    const unsigned cross = __ballot_sync(0xffffffffu, run + incl > target);
    const unsigned has_w = __ballot_sync(0xffffffffu, sel > 0.0);
    const int lsel = cross ? __ffs(cross) - 1 : (has_w ? 31 - __clz(has_w) : -1);
    if (lsel < 0) {
      if (lane == 0) *out = fallback;
      return;
    }
    if (lane != lsel) return;
    // element
    const long long i = w_start + (long long)it_sel * kWarpSpan;
    float w[4];
    weights4(a, rp, rq, mode, i, c, w);
    const double acc0 = run + (incl - sel);
    float part = 0.f;
    int pick = -1, lastw = -1;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      part += w[e];
      const double acc = acc0 + (double)part;
      if (w[e] > 0.f) lastw = (int)i + e;
      if (pick < 0 && w[e] > 0.f && acc > target) pick = (int)i + e;
    }
    *out = pick >= 0 ? pick : lastw;
    return;
  }
}

// One statistics CTA: (max, sum exp) of one chunk of one logit row, kept online per thread so that the chunk size is a
// run-time choice; ten 16-byte loads per thread are in flight at a time (a whole chunk at the 152k vocabulary).
// (Bringing the chunk into shared memory with bulk copies instead was measured and is no faster: the pass is then
// bound by the exponentials that follow the last byte, 16 per clock and SM.)
__device__ void stats_body(const AccArgs& a, const int b, const int row, const int chunk) {
  const float* x = row_ptr(a, b, row);
  const float c = a.inv_temp * kLog2e;
  const long long begin = (long long)chunk * a.stat_chunk;
  const long long end = begin + a.stat_chunk < a.V ? begin + a.stat_chunk : a.V;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float m = -INFINITY, l = 0.f;
  constexpr int kInFlight = 10;
  const float4 none = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
  for (long long i0 = begin + tid * 4; i0 < end; i0 += (long long)kInFlight * kAccThreads * 4) {
    float4 v[kInFlight];
#pragma unroll
    for (int k = 0; k < kInFlight; ++k) {
      const long long i = i0 + (long long)k * kAccThreads * 4;
      v[k] = none;
      if (i < end) {
        if (a.vec_ok && i + 3 < end) {
          v[k] = __ldg(reinterpret_cast<const float4*>(x + i));
        } else {
          v[k].x = __ldg(x + i);
          if (i + 1 < end) v[k].y = __ldg(x + i + 1);
          if (i + 2 < end) v[k].z = __ldg(x + i + 2);
          if (i + 3 < end) v[k].w = __ldg(x + i + 3);
        }
      }
    }
    // one reference for the batch: its maximum (40 exponentials for 40 logits, one more if the reference moved)
    float mx = m;
#pragma unroll
    for (int k = 0; k < kInFlight; ++k) mx = fmaxf(mx, fmaxf(fmaxf(v[k].x, v[k].y), fmaxf(v[k].z, v[k].w)));
    if (mx != -INFINITY) {
      float add[2] = {0.f, 0.f};
#pragma unroll
      for (int k = 0; k < kInFlight; ++k)
        add[k & 1] += (ex2f((v[k].x - mx) * c) + ex2f((v[k].y - mx) * c)) + (ex2f((v[k].z - mx) * c) + ex2f((v[k].w - mx) * c));
      if (mx > m) l *= ex2f((m - mx) * c);                // m = -inf: l is 0 and the factor ex2(-inf) = 0
      l += add[0] + add[1];
      m = mx;
    }
  }
#pragma unroll
  for (int sh = 16; sh >= 1; sh >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, sh), l2 = __shfl_xor_sync(0xffffffffu, l, sh);
    merge_ml(m, l, m2, l2, c);
  }
  __shared__ float sm[kAccWarps], sl[kAccWarps];
  if (lane == 0) { sm[warp] = m; sl[warp] = l; }
  __syncthreads();
  if (warp == 0) {
    m = sm[lane];
    l = sl[lane];
#pragma unroll
    for (int sh = 16; sh >= 1; sh >>= 1) {
      const float m2 = __shfl_xor_sync(0xffffffffu, m, sh), l2 = __shfl_xor_sync(0xffffffffu, l, sh);
      merge_ml(m, l, m2, l2, c);
    }
    if (lane == 0) {
      a.stats[((long long)b * a.rows + row) * a.n_stat_chunks + chunk] = make_float2(m, l);
      __threadfence();                                   // the partial is visible before it is counted
      atomicAdd(a.sync + b, 1);
    }
  }
}

// Grid: x = rank in the cluster, y = cluster of the sequence (0 = the tail team, then the statistics CTAs in row-major
// (row, chunk) order, `team` per cluster), z = sequence.
__global__ void __launch_bounds__(kAccThreads, 1) spec_accept_kernel(const AccArgs a) {
  const int b = blockIdx.z;
  if (blockIdx.y == 0) {
    team_body(a, b);
    return;
  }
  const int s = (blockIdx.y - 1) * a.team + blockIdx.x;
  if (s >= a.rows * a.n_stat_chunks) return;             // padding of the last cluster
  stats_body(a, b, s / a.n_stat_chunks, s % a.n_stat_chunks);
}

__global__ void __launch_bounds__(256) write_probs_kernel(const AccArgs a) {
  const int row = blockIdx.y, b = blockIdx.z;
  const int i = blockIdx.x * 256 + threadIdx.x;
  if (i >= a.V) return;
  const bool is_t = row <= a.gamma;
  float* dst = is_t ? a.probs_p : a.probs_q;
  if (!dst) return;
  const long long off = is_t ? (long long)b * a.tbs + (long long)row * a.trs
                             : (long long)b * a.dbs + (long long)(row - a.gamma - 1) * a.drs;
  const double lse = a.lse[(long long)b * a.rows + row];
  dst[off + i] = (float)exp((double)row_ptr(a, b, row)[i] * (double)a.inv_temp - lse);
}

// First rejection from given probabilities: the decision of the accept scan on its own (one thread per sequence).
__global__ void accept_from_probs_kernel(const float* __restrict__ p_tok, const float* __restrict__ q_tok,
                                         const float* __restrict__ u, long long u_stride, int gamma, int batch,
                                         int* __restrict__ n_accept) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= batch) return;
  int n = gamma;
  for (int t = 0; t < gamma; ++t)
    if (!accept_test(u[(long long)b * u_stride + t], p_tok[(long long)b * gamma + t], q_tok[(long long)b * gamma + t])) { n = t; break; }
  n_accept[b] = n;
}

}  // namespace

bool make_accept_plan(const pvlm_accept_params& p, AcceptPlan& plan) {
  if (p.gamma < 0 || p.gamma > 64 || p.V < 1 || p.batch < 1) return false;
  plan.rows = 2 * p.gamma + 1;
  // statistics chunks: as many per row as fit the one-wave budget, never smaller than one 16-byte load per thread
  long long per_row = kStatBudget / ((long long)plan.rows * p.batch);
  if (per_row < 1) per_row = 1;
  const long long grains = ceil_div(p.V, kStatGrain);
  if (per_row > grains) per_row = grains;
  plan.stat_chunk = (int)(ceil_div(grains, per_row)) * kStatGrain;
  plan.n_stat_chunks = ceil_div(p.V, plan.stat_chunk);
  // team size: enough warps that a warp's range fits the registered steps, at most one portable cluster
  const long long per_cta = (long long)kAccWarps * kWarpSpan * kRegIt;
  plan.team = 1;
  while (plan.team < kTeamMax && (long long)plan.team * per_cta < p.V) plan.team *= 2;
  plan.nit = ceil_div(p.V, (long long)plan.team * kAccWarps * kWarpSpan);
  size_t off = 0;
  plan.off_stats = off; off += align_up((size_t)p.batch * plan.rows * plan.n_stat_chunks * 8, 256);
  plan.off_lse = off;   off += align_up((size_t)p.batch * plan.rows * 8, 256);
  plan.off_sync = off;  off += align_up((size_t)p.batch * 4, 256);          // one counter per sequence
  plan.total = off;
  return true;
}

pvlm_status launch_spec_accept(const pvlm_accept_params& p, const AcceptPlan& plan, cudaStream_t s) {
  AccArgs a;
  a.tl = p.target_logits; a.dl = p.draft_logits;
  a.trs = p.target_row_stride; a.drs = p.draft_row_stride;
  a.tbs = p.target_batch_stride; a.dbs = p.draft_batch_stride;
  a.tok = p.draft_tokens; a.u = p.uniforms;
  a.batch = p.batch; a.gamma = p.gamma; a.V = p.V; a.rows = plan.rows;
  a.vec_ok = ((reinterpret_cast<uintptr_t>(p.target_logits) | reinterpret_cast<uintptr_t>(p.draft_logits)) % 16 == 0) &&
             ((p.target_row_stride | p.draft_row_stride | p.target_batch_stride | p.draft_batch_stride) % 4 == 0);
  a.inv_temp = (p.temperature == 0.f || p.temperature == 1.f) ? 1.f : 1.f / p.temperature;
  a.n_accept = p.n_accept; a.out_tokens = p.out_tokens;
  a.p_tok = p.p_tok; a.q_tok = p.q_tok; a.lse_p = p.lse_p; a.lse_q = p.lse_q;
  a.probs_p = p.probs_p; a.probs_q = p.probs_q;
  char* ws = (char*)p.workspace;
  a.stats = (float2*)(ws + plan.off_stats);
  a.lse = (double*)(ws + plan.off_lse);
  a.sync = (int*)(ws + plan.off_sync);
  a.n_stat_chunks = plan.n_stat_chunks;
  a.stat_chunk = plan.stat_chunk;
  a.team = plan.team;
  a.nit = plan.nit;
  cudaError_t e = cudaMemsetAsync(a.sync, 0, (size_t)p.batch * 4, s);
  if (e != cudaSuccess) { set_cuda_error((int)e); return PVLM_ERR_CUDA; }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(plan.team, 1 + ceil_div((long long)plan.rows * plan.n_stat_chunks, plan.team), p.batch);
  cfg.blockDim = dim3(kAccThreads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = plan.team;
  attr.val.clusterDim.y = 1;
  attr.val.clusterDim.z = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  e = cudaLaunchKernelEx(&cfg, spec_accept_kernel, a);
  if (e != cudaSuccess) { set_cuda_error((int)e); return PVLM_ERR_CUDA; }
  if (p.probs_p || p.probs_q)
    write_probs_kernel<<<dim3(ceil_div(p.V, 256), plan.rows, p.batch), 256, 0, s>>>(a);
  return check_launch();
}

pvlm_status launch_accept_from_probs(const float* p_tok, const float* q_tok, const float* uniforms, long long u_stride,
                                     int gamma, int batch, int* n_accept, cudaStream_t s) {
  accept_from_probs_kernel<<<ceil_div(batch, 128), 128, 0, s>>>(p_tok, q_tok, uniforms, u_stride, gamma, batch, n_accept);
  return check_launch();
}

}  // namespace pvlm
