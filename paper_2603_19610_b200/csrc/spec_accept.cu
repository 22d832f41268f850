// Vocab softmax statistics, accept/reject scan, residual / bonus sampling.
//
//   row_stats   : one coalesced pass over all (2*gamma+1) logit rows -> per-chunk (max, sum exp)
//   accept_scan : merge chunks -> lse per row; p(x_t), q(x_t); first rejection n
//   resid_sums  : row pair n only: per-chunk sums of max(0, p-q) and of p (fp64)
//   resid_pick  : inverse CDF over the chunk sums, then inside the crossing chunk
// Two launches: the CTA of row_stats / resid_sums that finishes last for a sequence (a ticket counter in the
// workspace) goes straight on to that sequence's accept_scan / resid_pick, so the two small single-CTA
// steps cost no launch of their own.
#include "pvlm_common.cuh"

namespace pvlm {

namespace {

constexpr int kStatThreads = 256;
constexpr int kStatChunk = 4096;     // elements per CTA (16 per thread)
constexpr int kSampThreads = 256;
constexpr int kSampChunk = 1024;     // elements per CTA (4 consecutive per thread)

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
  double* lse;        // [batch][rows]
  double* csum;       // [batch][n_samp_chunks][2]
  int* clast;         // [batch][n_samp_chunks][2]
  int* tickets;       // [batch][2] CTAs finished per sequence in the two launches (zeroed per call, reset by the last CTA)
  int n_stat_chunks, n_samp_chunks;
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

__device__ void accept_scan_body(const AccArgs& a, int b);
__device__ void resid_pick_body(const AccArgs& a, int b);

__global__ void __launch_bounds__(kStatThreads) row_stats_kernel(const AccArgs a) {
  pdl_launch_dependents();
  const int chunk = blockIdx.x, row = blockIdx.y, b = blockIdx.z;
  const float* x = row_ptr(a, b, row);
  const float c = a.inv_temp * kLog2e;
  const int base = chunk * kStatChunk;
  float v[16];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int i = base + k * (kStatThreads * 4) + threadIdx.x * 4;
    if (a.vec_ok && i + 3 < a.V) {
      const float4 t = __ldg(reinterpret_cast<const float4*>(x + i));
      v[4 * k] = t.x; v[4 * k + 1] = t.y; v[4 * k + 2] = t.z; v[4 * k + 3] = t.w;
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) v[4 * k + e] = (i + e < a.V) ? __ldg(x + i + e) : -INFINITY;
    }
  }
  float m = -INFINITY;
#pragma unroll
  for (int e = 0; e < 16; ++e) m = fmaxf(m, v[e]);
  float l = 0.f;
  if (m != -INFINITY) {
#pragma unroll
    for (int e = 0; e < 16; ++e) l += ex2f((v[e] - m) * c);
  }
#pragma unroll
  for (int sh = 16; sh >= 1; sh >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, sh), l2 = __shfl_xor_sync(0xffffffffu, l, sh);
    merge_ml(m, l, m2, l2, c);
  }
  __shared__ float sm[kStatThreads / 32], sl[kStatThreads / 32];
  if ((threadIdx.x & 31) == 0) { sm[threadIdx.x >> 5] = m; sl[threadIdx.x >> 5] = l; }
  __syncthreads();
  __shared__ int s_is_last;
  if (threadIdx.x == 0) {
    for (int w = 1; w < kStatThreads / 32; ++w) merge_ml(m, l, sm[w], sl[w], c);
    a.stats[((long long)b * a.rows + row) * a.n_stat_chunks + chunk] = make_float2(m, l);
    __threadfence();                                   // the partial is visible before the ticket is taken
    const int ticket = atomicAdd(&a.tickets[2 * b], 1);
    s_is_last = ticket == a.rows * a.n_stat_chunks - 1;
    if (s_is_last) a.tickets[2 * b] = 0;
  }
  __syncthreads();
  if (s_is_last) {                                     // every partial of this sequence has been written
    __threadfence();
    accept_scan_body(a, b);
  }
}

__device__ void accept_scan_body(const AccArgs& a, const int b) {
  const float c = a.inv_temp * kLog2e;
  __shared__ int s_reject[64];
  // one warp per logit row: lanes take chunk partials round-robin, then a fixed-order butterfly merge
  for (int row = threadIdx.x >> 5; row < a.rows; row += blockDim.x >> 5) {
    const float2* st = a.stats + ((long long)b * a.rows + row) * a.n_stat_chunks;
    const int lane = threadIdx.x & 31;
    float m = -INFINITY, l = 0.f;
    for (int ch = lane; ch < a.n_stat_chunks; ch += 32) {
      const float2 v = __ldcg(st + ch);                // written by other CTAs: read through L2
      merge_ml(m, l, v.x, v.y, c);
    }
#pragma unroll
    for (int sh = 16; sh >= 1; sh >>= 1) {
      const float m2 = __shfl_xor_sync(0xffffffffu, m, sh), l2 = __shfl_xor_sync(0xffffffffu, l, sh);
      merge_ml(m, l, m2, l2, c);
    }
    if (lane == 0) {
      const double lse = (double)m * (double)a.inv_temp + log((double)l);
      a.lse[(long long)b * a.rows + row] = lse;
      if (row <= a.gamma) { if (a.lse_p) a.lse_p[(long long)b * (a.gamma + 1) + row] = (float)lse; }
      else if (a.lse_q) a.lse_q[(long long)b * a.gamma + row - a.gamma - 1] = (float)lse;
    }
  }
  __syncthreads();
  for (int t = threadIdx.x; t < a.gamma; t += blockDim.x) {
    const int x = a.tok[(long long)b * a.gamma + t];
    float p = 0.f, q = 1.f;
    if (x >= 0 && x < a.V) {
      const double lp = a.lse[(long long)b * a.rows + t], lq = a.lse[(long long)b * a.rows + a.gamma + 1 + t];
      p = (float)exp((double)row_ptr(a, b, t)[x] * (double)a.inv_temp - lp);
      q = (float)exp((double)row_ptr(a, b, a.gamma + 1 + t)[x] * (double)a.inv_temp - lq);
    }
    if (a.p_tok) a.p_tok[(long long)b * a.gamma + t] = p;
    if (a.q_tok) a.q_tok[(long long)b * a.gamma + t] = q;
    const float uq = __fmul_rn(a.u[(long long)b * (a.gamma + 1) + t], q);
    s_reject[t] = !(uq < p);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int n = a.gamma;
    for (int t = 0; t < a.gamma; ++t)
      if (s_reject[t]) { n = t; break; }
    a.n_accept[b] = n;
    int* out = a.out_tokens + (long long)b * (a.gamma + 1);
    for (int t = 0; t <= a.gamma; ++t) out[t] = (t < n) ? a.tok[(long long)b * a.gamma + t] : -1;
  }
}

// weights of 4 consecutive vocabulary entries starting at i for the stopping position n
__device__ __forceinline__ void resid_weights(const AccArgs& a, int b, int n, int i, double (&wr)[4], double (&wp)[4]) {
  const float* xp = row_ptr(a, b, n);
  const double lp = a.lse[(long long)b * a.rows + n];
  const bool has_q = n < a.gamma;
  const float* xq = has_q ? row_ptr(a, b, a.gamma + 1 + n) : nullptr;
  const double lq = has_q ? a.lse[(long long)b * a.rows + a.gamma + 1 + n] : 0.0;
  const double it = (double)a.inv_temp;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    if (i + e < a.V) {
      const double p = exp((double)__ldg(xp + i + e) * it - lp);
      wp[e] = p;
      wr[e] = has_q ? fmax(0.0, p - exp((double)__ldg(xq + i + e) * it - lq)) : 0.0;
    } else {
      wp[e] = 0.0;
      wr[e] = 0.0;
    }
  }
}

__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int sh = 16; sh >= 1; sh >>= 1) v += __shfl_xor_sync(0xffffffffu, v, sh);
  return v;
}

__global__ void __launch_bounds__(kSampThreads) resid_sums_kernel(const AccArgs a) {
  pdl_wait();                  // the accept scan of the kernel before decides which row pair this one reads
  const int chunk = blockIdx.x, b = blockIdx.y;
  const int n = a.n_accept[b];
  const int i = chunk * kSampChunk + threadIdx.x * 4;
  double wr[4], wp[4];
  resid_weights(a, b, n, i, wr, wp);
  double sr = (wr[0] + wr[1]) + (wr[2] + wr[3]), sp = (wp[0] + wp[1]) + (wp[2] + wp[3]);
  int lr = -1, lp = -1;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    if (wr[e] > 0.0) lr = i + e;
    if (wp[e] > 0.0) lp = i + e;
  }
  sr = warp_sum_d(sr);
  sp = warp_sum_d(sp);
#pragma unroll
  for (int sh = 16; sh >= 1; sh >>= 1) {
    lr = max(lr, __shfl_xor_sync(0xffffffffu, lr, sh));
    lp = max(lp, __shfl_xor_sync(0xffffffffu, lp, sh));
  }
  __shared__ double ssr[kSampThreads / 32], ssp[kSampThreads / 32];
  __shared__ int slr[kSampThreads / 32], slp[kSampThreads / 32];
  const int w = threadIdx.x >> 5;
  if ((threadIdx.x & 31) == 0) { ssr[w] = sr; ssp[w] = sp; slr[w] = lr; slp[w] = lp; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int k = 1; k < kSampThreads / 32; ++k) { sr += ssr[k]; sp += ssp[k]; lr = max(lr, slr[k]); lp = max(lp, slp[k]); }
    const long long o = ((long long)b * a.n_samp_chunks + chunk) * 2;
    a.csum[o] = sr; a.csum[o + 1] = sp;
    a.clast[o] = lr; a.clast[o + 1] = lp;
  }
  __shared__ int s_is_last;
  if (threadIdx.x == 0) {
    __threadfence();
    const int ticket = atomicAdd(&a.tickets[2 * b + 1], 1);
    s_is_last = ticket == a.n_samp_chunks - 1;
    if (s_is_last) a.tickets[2 * b + 1] = 0;
  }
  __syncthreads();
  if (s_is_last) {
    __threadfence();
    resid_pick_body(a, b);
  }
}

__device__ void resid_pick_body(const AccArgs& a, const int b) {
  const int n = a.n_accept[b];
  __shared__ int s_chunk, s_fallback, s_pick;
  __shared__ double s_base, s_target;
  __shared__ double wsum[kSampThreads / 32];
  const double* cs = a.csum + (long long)b * a.n_samp_chunks * 2;
  const int* cl = a.clast + (long long)b * a.n_samp_chunks * 2;
  // block-wide fp64 reductions / scan over the chunk sums (chunks in index order, 256 per round)
  const int lane_ = threadIdx.x & 31, warp_ = threadIdx.x >> 5;
  __shared__ double red[kSampThreads / 32];
  __shared__ int s_last;
  auto block_sum = [&](double v) -> double {
    v = warp_sum_d(v);
    __syncthreads();
    if (lane_ == 0) red[warp_] = v;
    __syncthreads();
    double t = 0.0;
    for (int k = 0; k < kSampThreads / 32; ++k) t += red[k];
    return t;
  };
  double zr_part = 0.0, zp_part = 0.0;
  int last_r = -1, last_p = -1;
  for (int ch = threadIdx.x; ch < a.n_samp_chunks; ch += kSampThreads) {
    zr_part += __ldcg(cs + 2 * ch);                    // written by other CTAs: read through L2
    zp_part += __ldcg(cs + 2 * ch + 1);
    last_r = max(last_r, __ldcg(cl + 2 * ch));
    last_p = max(last_p, __ldcg(cl + 2 * ch + 1));
  }
  const double zr = block_sum(zr_part);
  const int mode = (zr > 0.0) ? 0 : 1;             // no residual weight at all => draw from p
  const double z = mode == 0 ? zr : block_sum(zp_part);
  const double target = (double)a.u[(long long)b * (a.gamma + 1) + a.gamma] * z;
  if (threadIdx.x == 0) { s_chunk = 0x7fffffff; s_last = -1; s_pick = 0x7fffffff; }
  __syncthreads();
  atomicMax(&s_last, mode == 0 ? last_r : last_p);
  double run_base = 0.0;
  for (int c0 = 0; c0 < a.n_samp_chunks; c0 += kSampThreads) {
    const int ch = c0 + threadIdx.x;
    const double v = ch < a.n_samp_chunks ? __ldcg(cs + 2 * ch + mode) : 0.0;
    double incl = v;
#pragma unroll
    for (int sh = 1; sh < 32; sh <<= 1) {
      const double t = __shfl_up_sync(0xffffffffu, incl, sh);
      if (lane_ >= sh) incl += t;
    }
    __syncthreads();
    if (lane_ == 31) red[warp_] = incl;
    __syncthreads();
    double off = run_base;
    for (int k = 0; k < warp_; ++k) off += red[k];
    incl += off;
    if (ch < a.n_samp_chunks && incl > target && incl - v <= target) {   // first crossing: unique
      if (atomicMin(&s_chunk, ch) > ch) s_base = incl - v;
    }
    double tot = run_base;
    for (int k = 0; k < kSampThreads / 32; ++k) tot += red[k];
    run_base = tot;
    __syncthreads();
    if (s_chunk != 0x7fffffff) break;
  }
  if (threadIdx.x == 0) {
    s_target = target;
    s_fallback = s_last;
    if (s_chunk == 0x7fffffff) s_chunk = -1;
  }
  __syncthreads();
  const int chunk = s_chunk;
  int* out = a.out_tokens + (long long)b * (a.gamma + 1) + n;
  if (chunk < 0) {                                 // rounding left no crossing: last token with weight
    if (threadIdx.x == 0) *out = s_fallback;
    return;
  }
  const int i = chunk * kSampChunk + threadIdx.x * 4;
  double wr[4], wp[4];
  resid_weights(a, b, n, i, wr, wp);
  double w4[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) w4[e] = mode == 0 ? wr[e] : wp[e];
  const double tsum = (w4[0] + w4[1]) + (w4[2] + w4[3]);
  // exclusive scan of per-thread sums across the block
  double incl = tsum;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
  for (int sh = 1; sh < 32; sh <<= 1) {
    const double t = __shfl_up_sync(0xffffffffu, incl, sh);
    if (lane >= sh) incl += t;
  }
  if (lane == 31) wsum[w] = incl;
  __syncthreads();
  double excl = s_base + (incl - tsum);
  for (int k = 0; k < w; ++k) excl += wsum[k];
  double run = excl;
  int mine = 0x7fffffff;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    run += w4[e];
    if (mine == 0x7fffffff && w4[e] > 0.0 && run > s_target) mine = i + e;
  }
  if (mine != 0x7fffffff) atomicMin(&s_pick, mine);
  __syncthreads();
  if (threadIdx.x == 0) *out = (s_pick != 0x7fffffff) ? s_pick : __ldcg(cl + 2 * chunk + mode);
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

}  // namespace

bool make_accept_plan(const pvlm_accept_params& p, AcceptPlan& plan) {
  if (p.gamma < 0 || p.gamma > 64 || p.V < 1 || p.batch < 1) return false;
  plan.rows = 2 * p.gamma + 1;
  plan.stat_chunk = kStatChunk;
  plan.n_stat_chunks = ceil_div(p.V, kStatChunk);
  plan.samp_chunk = kSampChunk;
  plan.n_samp_chunks = ceil_div(p.V, kSampChunk);
  size_t off = 0;
  plan.off_stats = off; off += align_up((size_t)p.batch * plan.rows * plan.n_stat_chunks * 8, 256);
  plan.off_lse = off;   off += align_up((size_t)p.batch * plan.rows * 8, 256);
  plan.off_csum = off;  off += align_up((size_t)p.batch * plan.n_samp_chunks * 2 * 8, 256);
  plan.off_clast = off; off += align_up((size_t)p.batch * plan.n_samp_chunks * 2 * 4, 256);
  plan.off_n = off;     off += align_up((size_t)p.batch * 2 * 4, 256);       // ticket counters
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
  a.csum = (double*)(ws + plan.off_csum);
  a.clast = (int*)(ws + plan.off_clast);
  a.tickets = (int*)(ws + plan.off_n);
  a.n_stat_chunks = plan.n_stat_chunks; a.n_samp_chunks = plan.n_samp_chunks;
  const cudaError_t e = cudaMemsetAsync(a.tickets, 0, (size_t)p.batch * 2 * 4, s);
  if (e != cudaSuccess) { set_cuda_error((int)e); return PVLM_ERR_CUDA; }
  row_stats_kernel<<<dim3(plan.n_stat_chunks, plan.rows, p.batch), kStatThreads, 0, s>>>(a);      // + accept scan
  {
    const cudaError_t e = launch_dependent(resid_sums_kernel, dim3(plan.n_samp_chunks, p.batch), dim3(kSampThreads), 0, s, a);   // + pick
    if (e != cudaSuccess) set_cuda_error((int)e);
  }
  if (p.probs_p || p.probs_q)
    write_probs_kernel<<<dim3(ceil_div(p.V, 256), plan.rows, p.batch), 256, 0, s>>>(a);
  return check_launch();
}

}  // namespace pvlm
