// Parallel decoding round loop (Algorithm 1: Pre-verify / Post-verify) on two CUDA streams.
// The host side is the mode machine; every token is drawn, tested and replaced by the accept kernels.
// The two models' caches are followed token by token: the verification call of a round sees the committed tokens
// and the window under test, every draft step sees what the draft has written so far, and a rejection rolls the
// draft's cache back to the committed prefix (appendix "Parallel Pipeline Details").
#include "pvlm_common.cuh"

#include <vector>
#include <cstring>

namespace pvlm {

namespace {

constexpr int kMaxGamma = 64;

// Device scratch of one call, after the two accept workspaces.
struct DecodeScratch {
  float* u_round;      // [gamma + 1]  accept uniforms of the round, then its resampling uniform
  int* verify_tok;     // [gamma]      tokens under test
  int* fresh[2];       // [gamma] x 2  tokens drafted in this / the previous round
  int* n_accept;       // [1]
  int* out_tokens;     // [gamma + 1]
  int* samp_n;         // [gamma]      n_accept of the sampling call (always 0)
};

struct DecodeLayout {
  size_t accept_ws, sample_ws, off_sample, off_small, total;
};

// Fills the fields of an accept call that are the same for every round: strides, sizes, temperature.
void accept_block(const pvlm_decode_params& p, int gamma, int batch, pvlm_accept_params& c) {
  c = pvlm_accept_params{};
  c.target_row_stride = c.draft_row_stride = p.row_stride;
  c.target_batch_stride = c.draft_batch_stride = p.row_stride;
  c.batch = batch;
  c.gamma = gamma;
  c.V = p.V;
  c.temperature = p.temperature;
}

bool make_layout(const pvlm_decode_params& p, DecodeLayout& l) {
  pvlm_accept_params c;
  AcceptPlan plan;
  // A round verifies between 1 and gamma tokens, and a SHORTER window can need more scratch (fewer logit rows are cut
  // into more statistics chunks each): size for the largest of them.
  l.accept_ws = 0;
  for (int nv = 1; nv <= p.gamma; ++nv) {
    accept_block(p, nv, 1, c);
    if (!make_accept_plan(c, plan)) return false;
    if (align_up(plan.total, 256) > l.accept_ws) l.accept_ws = align_up(plan.total, 256);
  }
  accept_block(p, 0, p.gamma, c);
  if (!make_accept_plan(c, plan)) return false;
  l.sample_ws = align_up(plan.total, 256);
  l.off_sample = l.accept_ws;
  l.off_small = l.off_sample + l.sample_ws;
  l.total = l.off_small + align_up((size_t)(6 * (kMaxGamma + 1)) * 4, 256);
  return true;
}

// Builds the verification call's small inputs on the device: the tokens under test (the pending drafts, or
// the first fresh draft in a Pre-verify round) and [accept uniforms of this round | resampling uniform].
__global__ void decode_prepare_kernel(const int* __restrict__ src_tok, int nv, const float* __restrict__ u_accept_row,
                                      const float* __restrict__ u_resample, int* __restrict__ verify_tok,
                                      float* __restrict__ u_round) {
  const int t = threadIdx.x;
  if (t < nv) {
    verify_tok[t] = src_tok[t];
    u_round[t] = u_accept_row[t];
  }
  if (t == nv) u_round[nv] = *u_resample;
}

}  // namespace

}  // namespace pvlm

using namespace pvlm;

extern "C" {

size_t pvlm_parallel_decode_workspace_bytes(const pvlm_decode_params* p) {
  DecodeLayout l;
  if (!p || p->gamma < 1 || p->gamma > kMaxGamma || p->V < 1 || p->row_stride < p->V) return 0;
  return make_layout(*p, l) ? l.total : 0;
}

pvlm_status pvlm_parallel_decode(const pvlm_decode_params* p, void* target_stream, void* draft_stream) {
  if (!p) return PVLM_ERR_INVALID_ARG;
  if (p->gamma < 1 || p->gamma > kMaxGamma || p->V < 1 || p->K < 1 || p->row_stride < p->V || p->max_rounds < 1)
    return PVLM_ERR_INVALID_ARG;
  if (!p->target_logits || !p->draft_logits || !p->u_draft || !p->u_accept || !p->u_resample || !p->tokens)
    return PVLM_ERR_INVALID_ARG;
  if (p->temperature < 0.f) return PVLM_ERR_INVALID_ARG;
  if ((long long)p->P < (long long)p->K + 2 * p->gamma + 1) return PVLM_ERR_TOO_LARGE;
  if (!p->serial && (!draft_stream || draft_stream == target_stream)) return PVLM_ERR_INVALID_ARG;
  DecodeLayout lay;
  if (!make_layout(*p, lay)) return PVLM_ERR_UNSUPPORTED;
  if (!p->workspace || reinterpret_cast<uintptr_t>(p->workspace) % 256 || p->workspace_bytes < lay.total) return PVLM_ERR_WORKSPACE;

  cudaStream_t ts = (cudaStream_t)target_stream;
  cudaStream_t ds = p->serial ? ts : (cudaStream_t)draft_stream;
  const int g = p->gamma;
  char* ws = (char*)p->workspace;
  DecodeScratch sc;
  {
    int* small = (int*)(ws + lay.off_small);
    const int w = kMaxGamma + 1;
    sc.u_round = (float*)small;
    sc.verify_tok = small + w;
    sc.fresh[0] = small + 2 * w;
    sc.fresh[1] = small + 3 * w;
    sc.out_tokens = small + 4 * w;
    sc.samp_n = small + 5 * w;
    sc.n_accept = small + 5 * w + kMaxGamma;      // last word of the sampling block's row
  }

  cudaEvent_t ev_drafted = nullptr, ev_draft_done = nullptr, ev_round_start = nullptr, ev_t0 = nullptr, ev_t1 = nullptr;
  cudaError_t e = cudaEventCreateWithFlags(&ev_drafted, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ev_draft_done, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ev_round_start, cudaEventDisableTiming);
  if (e == cudaSuccess && p->round_ms) e = cudaEventCreate(&ev_t0);
  if (e == cudaSuccess && p->round_ms) e = cudaEventCreate(&ev_t1);
  pvlm_status st = PVLM_OK;
  auto fail = [&](pvlm_status s) { if (st == PVLM_OK) st = s; };
  if (e != cudaSuccess) { set_cuda_error((int)e); fail(PVLM_ERR_CUDA); }

  // host copies of one round's results, in pinned memory (one small buffer per host thread, kept):
  // [n_accept | out_tokens (g+1) | fresh (g) | status words: target, draft step 0..g-1]
  static thread_local int* h_pinned = nullptr;
  constexpr int kResWords = 1 + (kMaxGamma + 1) + kMaxGamma + 1 + kMaxGamma;
  if (!h_pinned && cudaHostAlloc((void**)&h_pinned, kResWords * sizeof(int), cudaHostAllocDefault) != cudaSuccess) {
    (void)cudaGetLastError();
    h_pinned = nullptr;
  }
  std::vector<int> h_fallback(h_pinned ? 0 : kResWords), h_pending(g, 0);
  int* h_res = h_pinned ? h_pinned : h_fallback.data();
  int* h_status = h_res + 2 + 2 * g;                       // [0] target, [1 + t] draft step t
  memset(h_res, 0, kResWords * sizeof(int));
  int mode = 0 /* Pre */, n_pending = 0, committed = 0, round = 0, cur = 0;
  // Where a call's status word lives (a bounded wait inside the attention kernels that expired sets it).
  auto status_word = [](const pvlm_attn_params& ap) -> const int* {
    AttnPlan plan;
    if (!make_attn_plan(ap, plan) || !plan.use_tc) return nullptr;
    return reinterpret_cast<const int*>(static_cast<const char*>(ap.workspace) + plan.off_tc + plan.tc.off_status);
  };

  while (st == PVLM_OK && committed < p->K) {
    if (round >= p->max_rounds) { fail(PVLM_ERR_TOO_LARGE); break; }
    const bool post = mode == 1 && n_pending > 0;
    const int nv = post ? n_pending : 1;
    const int L = committed;
    const int base = L + (post ? n_pending : 0);               // first position the draft writes in this round
    int* fresh = sc.fresh[cur];
    int* pending = sc.fresh[cur ^ 1] + (g - n_pending);         // the pending drafts are the tail of last round's

    if (p->round_ms) e = cudaEventRecord(ev_t0, ts);
    if (!p->serial) {                                           // the draft stream starts where the target stream stands
      if (e == cudaSuccess) e = cudaEventRecord(ev_round_start, ts);
      if (e == cudaSuccess) e = cudaStreamWaitEvent(ds, ev_round_start, 0);
    }
    if (e != cudaSuccess) { set_cuda_error((int)e); fail(PVLM_ERR_CUDA); break; }

    // ---- draft side: gamma draws from the draft rows base .. base+gamma-1, then the draft forwards' traffic ----
    {
      pvlm_accept_params c;
      accept_block(*p, 0, g, c);
      c.target_logits = p->draft_logits + (long long)base * p->row_stride;
      c.uniforms = p->u_draft + (long long)round * g;
      c.n_accept = sc.samp_n;
      c.out_tokens = fresh;
      c.workspace = ws + lay.off_sample;
      c.workspace_bytes = lay.sample_ws;
      const pvlm_status s2 = pvlm_spec_accept(&c, ds);
      if (s2 != PVLM_OK) { fail(s2); break; }
      if (!p->serial) e = cudaEventRecord(ev_drafted, ds);
      // the draft's forwards: step t reads the cache as it stands after the tokens written so far
      // (compacted context, committed tokens, pending drafts, this round's first t drafts) and adds one row
      for (int i = 0; i < g && p->draft_attn && st == PVLM_OK; ++i) {
        pvlm_attn_params da = *p->draft_attn;
        da.n_ctx = p->draft_attn->n_ctx + base + i;
        const pvlm_status s3 = pvlm_verify_attn(&da, ds);
        if (s3 != PVLM_OK) { fail(s3); break; }
        if (const int* w = status_word(da)) e = cudaMemcpyAsync(h_status + 1 + i, w, 4, cudaMemcpyDeviceToHost, ds);
        if (e != cudaSuccess) break;
      }
      if (!p->serial && e == cudaSuccess) e = cudaEventRecord(ev_draft_done, ds);
      if (e != cudaSuccess) { set_cuda_error((int)e); fail(PVLM_ERR_CUDA); }
      if (st != PVLM_OK) break;
    }

    // ---- target side: the target forward's traffic, then accept / reject / resample over the tokens under test ----
    // the target's forward: the committed tokens are context, the window holds the last committed token and the
    // nv tokens under test
    if (p->target_attn) {
      pvlm_attn_params ta = *p->target_attn;
      ta.n_ctx = p->target_attn->n_ctx + L;
      ta.R = nv + 1;
      const pvlm_status s3 = pvlm_verify_attn(&ta, ts);
      if (s3 != PVLM_OK) { fail(s3); break; }
      if (const int* w = status_word(ta)) e = cudaMemcpyAsync(h_status, w, 4, cudaMemcpyDeviceToHost, ts);
      if (e != cudaSuccess) { set_cuda_error((int)e); fail(PVLM_ERR_CUDA); break; }
    }
    if (!post && !p->serial) e = cudaStreamWaitEvent(ts, ev_drafted, 0);     // Pre-verify tests this round's first draft
    if (e != cudaSuccess) { set_cuda_error((int)e); fail(PVLM_ERR_CUDA); break; }
    decode_prepare_kernel<<<1, 128, 0, ts>>>(post ? pending : fresh, nv, p->u_accept + (long long)round * g,
                                             p->u_resample + round, sc.verify_tok, sc.u_round);
    if (check_launch() != PVLM_OK) { fail(PVLM_ERR_CUDA); break; }
    {
      pvlm_accept_params c;
      accept_block(*p, nv, 1, c);
      c.target_logits = p->target_logits + (long long)L * p->row_stride;
      c.draft_logits = p->draft_logits + (long long)L * p->row_stride;
      c.draft_tokens = sc.verify_tok;
      c.uniforms = sc.u_round;
      c.n_accept = sc.n_accept;
      c.out_tokens = sc.out_tokens;
      c.workspace = ws;
      c.workspace_bytes = lay.accept_ws;
      const pvlm_status s2 = pvlm_spec_accept(&c, ts);
      if (s2 != PVLM_OK) { fail(s2); break; }
    }
    // ---- join, read the round's outcome ----
    if (!p->serial) e = cudaStreamWaitEvent(ts, ev_draft_done, 0);
    if (e == cudaSuccess && p->round_ms) e = cudaEventRecord(ev_t1, ts);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h_res, sc.n_accept, 4, cudaMemcpyDeviceToHost, ts);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h_res + 1, sc.out_tokens, (size_t)(nv + 1) * 4, cudaMemcpyDeviceToHost, ts);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h_res + 2 + g, fresh, (size_t)g * 4, cudaMemcpyDeviceToHost, ts);
    if (e == cudaSuccess) e = cudaStreamSynchronize(ts);
    if (e != cudaSuccess) { set_cuda_error((int)e); fail(PVLM_ERR_CUDA); break; }
    if (p->round_ms) {
      float ms = 0.f;
      cudaEventElapsedTime(&ms, ev_t0, ev_t1);
      p->round_ms[round] = ms;
    }

    // a bounded wait that expired inside one of this round's attention calls: its outputs are undefined
    {
      int any = h_status[0];
      for (int i = 0; i < g; ++i) any |= h_status[1 + i];
      if (any) { fail(PVLM_ERR_TIMEOUT); break; }
    }
    // ---- the mode machine ----
    const int n = h_res[0];
    const int* h_fresh = h_res + 2 + g;
    if (n < 0 || n > nv) { fail(PVLM_ERR_CUDA); break; }
    int emitted, dropped, next_mode, next_pending;
    auto commit = [&](int tok) { if (committed < p->K) p->tokens[committed] = tok; ++committed; };
    for (int i = 0; i < n; ++i) commit(post ? h_pending[g - n_pending + i] : h_fresh[0]);
    if (n < nv) {                                   // rejection: the replacement token, everything else is dropped
      commit(h_res[1 + n]);
      emitted = n + 1;
      dropped = (post ? nv - n : 0) + g;
      next_mode = 0;
      next_pending = 0;
    } else if (post) {
      emitted = nv; dropped = 0; next_mode = 1; next_pending = g;
    } else {
      emitted = 1; dropped = 0; next_pending = g - 1; next_mode = next_pending > 0 ? 1 : 0;
    }
    if (p->round_log) {
      int* r = p->round_log + (long long)round * PVLM_DECODE_LOG_COLS;
      r[0] = post ? 1 : 0; r[1] = nv; r[2] = n; r[3] = emitted; r[4] = dropped; r[5] = L;
      r[6] = L;                              // generated tokens in the verification call's context
      r[7] = base;                           // generated tokens in the draft's cache before its first step of the round
      r[8] = L + emitted + next_pending;     // ... and after the round: a rejection truncates it to the committed prefix
    }
    for (int i = 0; i < g; ++i) h_pending[i] = h_fresh[i];      // tail [g - next_pending, g) is what stays pending
    mode = next_mode;
    n_pending = next_pending;
    cur ^= 1;
    ++round;
  }
  if (st != PVLM_OK) {                               // leave both streams idle whatever happened
    cudaStreamSynchronize(ts);
    if (!p->serial) cudaStreamSynchronize(ds);
  }
  if (p->n_rounds) *p->n_rounds = round;
  if (ev_drafted) cudaEventDestroy(ev_drafted);
  if (ev_draft_done) cudaEventDestroy(ev_draft_done);
  if (ev_round_start) cudaEventDestroy(ev_round_start);
  if (ev_t0) cudaEventDestroy(ev_t0);
  if (ev_t1) cudaEventDestroy(ev_t1);
  return st;
}

}  // extern "C"
