// C-ABI entry points: host-side argument validation, workspace queries, dispatch.
#include "pvlm_common.cuh"
#include <cstdlib>

#include <atomic>
#include <cmath>
#include <cstring>

namespace pvlm {

static thread_local int g_last_cuda_error = 0;

void set_cuda_error(int e) { g_last_cuda_error = e; }

static thread_local cudaEvent_t g_after_main_event = nullptr;

bool pdl_enabled() {
  static const bool on = [] { const char* e = getenv("PVLM_PDL"); return !(e && e[0] == '0'); }();
  return on;
}

// Process-wide switches.  Their defaults come from the environment, read once when the first one is looked at;
// after that only pvlm_set_option changes them, so no call reads the environment on its launch path.
static std::atomic<int>* option_slots() {
  static std::atomic<int> slots[PVLM_OPT_COUNT];
  static const bool init = [] {
    const char* e = getenv("PVLM_ATTN_IMPL");
    slots[PVLM_OPT_ATTN_MMA_SYNC].store(e && strcmp(e, "mma") == 0);
    e = getenv("PVLM_SELECT_IMPL");
    slots[PVLM_OPT_SELECT_ONE_CTA].store(e && strcmp(e, "cta") == 0);
    e = getenv("PVLM_TC_CTAS");
    slots[PVLM_OPT_ATTN_MAX_CTAS].store(e ? atoi(e) : 0);
    return true;
  }();
  (void)init;
  return slots;
}

int option_value(int option) { return option_slots()[option].load(std::memory_order_relaxed); }

void set_after_main_event(cudaEvent_t ev) { g_after_main_event = ev; }
cudaEvent_t take_after_main_event() {
  cudaEvent_t ev = g_after_main_event;
  g_after_main_event = nullptr;
  return ev;
}

pvlm_status check_launch() {
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    g_last_cuda_error = (int)e;
    return PVLM_ERR_CUDA;
  }
  return PVLM_OK;
}

static inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

static pvlm_status check_ws(const void* ws, size_t have, size_t need) {
  if (need == 0) return PVLM_OK;
  if (!ws || !aligned(ws, 256) || have < need) return PVLM_ERR_WORKSPACE;
  return PVLM_OK;
}

}  // namespace pvlm

using namespace pvlm;

extern "C" {

const char* pvlm_status_string(pvlm_status s) {
  switch (s) {
    case PVLM_OK: return "PVLM_OK";
    case PVLM_ERR_INVALID_ARG: return "PVLM_ERR_INVALID_ARG";
    case PVLM_ERR_UNSUPPORTED: return "PVLM_ERR_UNSUPPORTED";
    case PVLM_ERR_WORKSPACE: return "PVLM_ERR_WORKSPACE";
    case PVLM_ERR_CUDA: return "PVLM_ERR_CUDA";
    case PVLM_ERR_TOO_LARGE: return "PVLM_ERR_TOO_LARGE";
    case PVLM_ERR_TIMEOUT: return "PVLM_ERR_TIMEOUT";
    default: return "PVLM_ERR_UNKNOWN";
  }
}

int pvlm_last_cuda_error(void) { return g_last_cuda_error; }

int pvlm_version(void) { return 1001; }

int pvlm_set_option(int option, int value) {
  if (option < 0 || option >= PVLM_OPT_COUNT) return -1;
  if (value < 0) return -1;
  return option_slots()[option].exchange(value);
}

size_t pvlm_verify_attn_workspace_bytes(const pvlm_attn_params* p) {
  AttnPlan plan;
  if (!p || !make_attn_plan(*p, plan)) return 0;
  return plan.total;
}

// Every host-side check of an attention call; fills the plan.  Nothing is launched.
static pvlm_status validate_attn(const pvlm_attn_params* p, AttnPlan& plan) {
  if (!p) return PVLM_ERR_INVALID_ARG;
  if (p->n_layers < 1 || p->R < 1 || p->Hq < 1 || p->Hkv < 1 || p->D < 1 || p->n_ctx < 0) return PVLM_ERR_INVALID_ARG;
  if (!p->q || !p->k || !p->v || !p->o) return PVLM_ERR_INVALID_ARG;
  if (!make_attn_plan(*p, plan)) return PVLM_ERR_UNSUPPORTED;
  if (!aligned(p->q, 16) || !aligned(p->k, 16) || !aligned(p->v, 16) || !aligned(p->o, 16)) return PVLM_ERR_INVALID_ARG;
  if (p->kv_head_stride < p->D || p->kv_head_stride % 8) return PVLM_ERR_INVALID_ARG;
  if (p->kv_token_stride < p->D || p->kv_token_stride % 8) return PVLM_ERR_INVALID_ARG;   // token-major or head-major caches
  if (p->n_layers > 1) {
    if (p->kv_layer_stride < (long long)plan.T * p->D || p->kv_layer_stride % 8) return PVLM_ERR_INVALID_ARG;
    if (p->q_layer_stride < (long long)p->R * p->Hq * p->D || p->q_layer_stride % 8) return PVLM_ERR_INVALID_ARG;
  }
  if (p->mass) {
    const int n_mass = p->mass_layers ? p->n_mass_layers : p->n_layers;
    if (p->mass_layers) {
      if (p->n_mass_layers < 1) return PVLM_ERR_INVALID_ARG;
      if (p->n_mass_layers > 8) return PVLM_ERR_UNSUPPORTED;
      for (int i = 0; i < p->n_mass_layers; ++i)
        if (p->mass_layers[i] < 0 || p->mass_layers[i] >= p->n_layers) return PVLM_ERR_INVALID_ARG;
    }
    if (n_mass > 1 && p->mass_layer_stride < plan.T) return PVLM_ERR_INVALID_ARG;
  }
  if (p->n_layers > 65535 || p->Hkv > 65535) return PVLM_ERR_UNSUPPORTED;
  if (p->max_ctas < 0) return PVLM_ERR_INVALID_ARG;
  return check_ws(p->workspace, p->workspace_bytes, plan.total);
}

pvlm_status pvlm_verify_attn(const pvlm_attn_params* p, void* stream) {
  AttnPlan plan;
  const pvlm_status v = validate_attn(p, plan);
  if (v != PVLM_OK) return v;
  return launch_verify_attn(*p, plan, (cudaStream_t)stream);
}

pvlm_status pvlm_verify_attn_check(const pvlm_attn_params* p, void* stream) {
  if (!p) return PVLM_ERR_INVALID_ARG;
  AttnPlan plan;
  if (!make_attn_plan(*p, plan)) return PVLM_ERR_UNSUPPORTED;
  const pvlm_status w = check_ws(p->workspace, p->workspace_bytes, plan.total);
  if (w != PVLM_OK) return w;
  int word = 0;
  cudaError_t e = cudaSuccess;
  if (plan.use_tc)
    e = cudaMemcpyAsync(&word, (const char*)p->workspace + plan.off_tc + plan.tc.off_status, 4, cudaMemcpyDeviceToHost,
                        (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
  if (e != cudaSuccess) { set_cuda_error((int)e); return PVLM_ERR_CUDA; }
  return word ? PVLM_ERR_TIMEOUT : PVLM_OK;
}

size_t pvlm_uvprune_workspace_bytes(const pvlm_prune_params* p) {
  if (!p || p->m < 0) return 0;
  return uvprune_workspace(*p);
}

static pvlm_status validate_prune(const pvlm_prune_params* p) {
  if (!p) return PVLM_ERR_INVALID_ARG;
  if (p->m < 0 || p->k < 0 || p->k > p->m || p->vis_start < 0) return PVLM_ERR_INVALID_ARG;
  if (p->m > (1 << 24)) return PVLM_ERR_UNSUPPORTED;
  if (p->m > 0 && !p->mass_cur) return PVLM_ERR_INVALID_ARG;
  if (p->k > 0 && !p->kept_idx) return PVLM_ERR_INVALID_ARG;
  const bool gather = p->src_k || p->src_v || p->dst_k || p->dst_v;
  if (gather) {
    if (!p->src_k || !p->src_v) return PVLM_ERR_INVALID_ARG;
    if (p->n_layers < 1 || p->row_bytes <= 0 || p->src_len < p->vis_start + p->m) return PVLM_ERR_INVALID_ARG;
    const long long dst_len = (long long)p->src_len - p->m + p->k;
    if (dst_len > 0 && (!p->dst_k || !p->dst_v)) return PVLM_ERR_INVALID_ARG;     // an empty compacted cache needs no storage
    if (p->row_bytes % 16) return PVLM_ERR_UNSUPPORTED;
    if (!aligned(p->src_k, 16) || !aligned(p->src_v, 16) || !aligned(p->dst_k, 16) || !aligned(p->dst_v, 16))
      return PVLM_ERR_INVALID_ARG;
    if (p->n_layers > 1) {
      if (p->src_layer_stride_bytes < (long long)p->src_len * p->row_bytes || p->src_layer_stride_bytes % 16) return PVLM_ERR_INVALID_ARG;
      if (p->dst_layer_stride_bytes < dst_len * p->row_bytes || p->dst_layer_stride_bytes % 16) return PVLM_ERR_INVALID_ARG;
    }
  }
  return check_ws(p->workspace, p->workspace_bytes, uvprune_workspace(*p));
}

pvlm_status pvlm_uvprune_select_gather(const pvlm_prune_params* p, void* stream) {
  const pvlm_status w = validate_prune(p);
  if (w != PVLM_OK) return w;
  return launch_uvprune(*p, (cudaStream_t)stream);
}

static bool similarity_supported(const pvlm_similarity_params* p) {
  return p->d >= 8 && p->d <= 16384 && p->d % 8 == 0;
}

size_t pvlm_uvprune_similarity_workspace_bytes(const pvlm_similarity_params* p) {
  if (!p || p->m < 0 || p->n < 0 || p->n_layers < 0 || p->n_layers > 65535 || !similarity_supported(p)) return 0;
  return similarity_workspace(*p);
}

pvlm_status pvlm_uvprune_similarity(const pvlm_similarity_params* p, void* stream) {
  if (!p) return PVLM_ERR_INVALID_ARG;
  if (p->m < 0 || p->n < 0 || p->vis_start < 0 || p->text_start < 0 || p->d < 1) return PVLM_ERR_INVALID_ARG;
  if (!similarity_supported(p)) return PVLM_ERR_UNSUPPORTED;
  if (!p->hidden || (p->m > 0 && !p->sim)) return PVLM_ERR_INVALID_ARG;
  if (!aligned(p->hidden, 16) || p->hidden_row_stride < p->d || p->hidden_row_stride % 8) return PVLM_ERR_INVALID_ARG;
  if (p->n_layers < 0) return PVLM_ERR_INVALID_ARG;
  if (p->n_layers > 65535) return PVLM_ERR_UNSUPPORTED;
  if (p->n_layers > 1 && (p->hidden_layer_stride < 0 || p->hidden_layer_stride % 8 || p->sim_layer_stride < p->m)) return PVLM_ERR_INVALID_ARG;
  const pvlm_status w = check_ws(p->workspace, p->workspace_bytes, similarity_workspace(*p));
  if (w != PVLM_OK) return w;
  return launch_similarity(*p, (cudaStream_t)stream);
}

size_t pvlm_spec_accept_workspace_bytes(const pvlm_accept_params* p) {
  AcceptPlan plan;
  if (!p || !make_accept_plan(*p, plan)) return 0;
  return plan.total;
}

// Every host-side check of an accept call; fills the plan.  Nothing is launched.
static pvlm_status validate_accept(const pvlm_accept_params* p, AcceptPlan& plan) {
  if (!p) return PVLM_ERR_INVALID_ARG;
  if (p->gamma < 0 || p->V < 1 || p->batch < 1) return PVLM_ERR_INVALID_ARG;
  if (!p->target_logits || !p->uniforms || !p->n_accept || !p->out_tokens) return PVLM_ERR_INVALID_ARG;
  if (p->gamma > 0 && (!p->draft_logits || !p->draft_tokens)) return PVLM_ERR_INVALID_ARG;
  if (!make_accept_plan(*p, plan)) return PVLM_ERR_UNSUPPORTED;
  if (p->batch > 65535) return PVLM_ERR_UNSUPPORTED;
  if (!aligned(p->target_logits, 4) || !aligned(p->draft_logits, 4)) return PVLM_ERR_INVALID_ARG;
  if (p->target_row_stride < p->V || (p->gamma > 0 && p->draft_row_stride < p->V)) return PVLM_ERR_INVALID_ARG;
  if (p->batch > 1) {
    // batch stride 0 = every sequence reads the same logits
    if (p->target_batch_stride != 0 && (p->target_batch_stride < (long long)(p->gamma + 1) * p->target_row_stride)) return PVLM_ERR_INVALID_ARG;
    if (p->draft_batch_stride != 0 && (p->draft_batch_stride < (long long)p->gamma * p->draft_row_stride)) return PVLM_ERR_INVALID_ARG;
  }
  if (p->temperature < 0.f) return PVLM_ERR_INVALID_ARG;
  return check_ws(p->workspace, p->workspace_bytes, plan.total);
}

pvlm_status pvlm_spec_accept(const pvlm_accept_params* p, void* stream) {
  AcceptPlan plan;
  const pvlm_status v = validate_accept(p, plan);
  if (v != PVLM_OK) return v;
  return launch_spec_accept(*p, plan, (cudaStream_t)stream);
}

pvlm_status pvlm_select_from_scores(const float* score, int m, int k, int* kept_idx, void* workspace,
                                    size_t workspace_bytes, void* stream) {
  pvlm_prune_params p = {};
  p.mass_cur = score;
  p.m = m;
  p.k = k;
  p.kept_idx = kept_idx;
  p.workspace = workspace;
  p.workspace_bytes = workspace_bytes;
  return pvlm_uvprune_select_gather(&p, stream);
}

pvlm_status pvlm_accept_from_probs(const float* p_tok, const float* q_tok, const float* uniforms, int uniform_stride,
                                   int gamma, int batch, int* n_accept, void* stream) {
  if (gamma < 0 || batch < 1 || uniform_stride < gamma || !n_accept) return PVLM_ERR_INVALID_ARG;
  if (gamma > 0 && (!p_tok || !q_tok || !uniforms)) return PVLM_ERR_INVALID_ARG;
  return launch_accept_from_probs(p_tok, q_tok, uniforms, uniform_stride, gamma, batch, n_accept, (cudaStream_t)stream);
}

pvlm_status pvlm_verify_step(const pvlm_step_params* p, void* stream) {
  if (!p) return PVLM_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  const bool overlap = p->copy_stream && p->event_a && p->event_b;
  if (!overlap && (p->copy_stream || p->event_a || p->event_b)) return PVLM_ERR_INVALID_ARG;
  cudaStream_t cs = overlap ? (cudaStream_t)p->copy_stream : s;      // stream of the overlappable copies
  cudaEvent_t ea = (cudaEvent_t)p->event_a, eb = (cudaEvent_t)p->event_b;
  const pvlm_attn_params& a = p->attn;
  const pvlm_accept_params& c = p->accept;
  cudaError_t e = cudaSuccess;
  auto ok = [&]() { return e == cudaSuccess; };
  // ---- every argument check of the stages and the copies, before anything is queued on either stream ----
  if (p->run_attn) {
    AttnPlan plan;
    const pvlm_status va = validate_attn(&a, plan);
    if (va != PVLM_OK) return va;
  }
  if (p->run_attn && (p->h_k_window || p->h_v_window)) {
    const bool token_major = a.kv_head_stride == a.D && a.kv_token_stride == (long long)a.Hkv * a.D;
    const bool head_major = a.kv_token_stride == a.D && a.kv_head_stride >= (long long)(a.n_ctx + a.R) * a.D &&
                            (a.n_layers == 1 || a.kv_layer_stride == (long long)a.Hkv * a.kv_head_stride);
    if (!token_major && !head_major) return PVLM_ERR_UNSUPPORTED;
  }
  if (p->run_accept) {
    AcceptPlan plan;
    const pvlm_status vc = validate_accept(&c, plan);
    if (vc != PVLM_OK) return vc;
    if (p->h_target_logits || p->h_draft_logits) {
      if (c.target_row_stride != c.V || c.draft_row_stride != c.V) return PVLM_ERR_UNSUPPORTED;
      if (c.batch > 1 && (c.target_batch_stride != (long long)(c.gamma + 1) * c.V ||
                          c.draft_batch_stride != (long long)c.gamma * c.V)) return PVLM_ERR_UNSUPPORTED;
    }
  }
  if (p->run_prune) {
    const pvlm_status vp = validate_prune(&p->prune);
    if (vp != PVLM_OK) return vp;
  }
  // ---- host -> device: this step's inputs ----
  // The side stream is forked from `stream` (an event recorded there, a wait on the side) only at the first point where
  // something is queued on it, and joined back at the end if it was forked: a call with nothing for it costs no
  // stream operation, and a stream capture of the call always closes.
  bool forked = false;
  const bool side_uploads = p->run_accept && (p->h_target_logits || p->h_draft_logits || p->h_draft_tokens || p->h_uniforms);
  if (overlap && side_uploads) {       // the copies start after whatever is already queued on `stream`
    e = cudaEventRecord(ea, s);
    if (ok()) e = cudaStreamWaitEvent(cs, ea, 0);
    forked = true;
  }
  if (p->run_attn) {
    const size_t q_layer = (size_t)a.R * a.Hq * a.D * 2;
    if (p->h_q && ok())
      e = cudaMemcpy2DAsync(const_cast<void*>(a.q), (size_t)a.q_layer_stride * 2, p->h_q, q_layer, q_layer, a.n_layers,
                            cudaMemcpyHostToDevice, s);
    if (p->h_k_window || p->h_v_window) {
      const bool token_major = a.kv_head_stride == a.D && a.kv_token_stride == (long long)a.Hkv * a.D;
      const bool head_major = a.kv_token_stride == a.D && a.kv_head_stride >= (long long)(a.n_ctx + a.R) * a.D &&
                              (a.n_layers == 1 || a.kv_layer_stride == (long long)a.Hkv * a.kv_head_stride);
      size_t width, pitch, row0 = (size_t)a.n_ctx * a.kv_token_stride * 2;
      int height;
      if (token_major) {                   // host [n_layers][R][Hkv][D]: one piece of R rows per layer
        width = (size_t)a.R * a.Hkv * a.D * 2;
        pitch = a.n_layers > 1 ? (size_t)a.kv_layer_stride * 2 : width;
        height = a.n_layers;
      } else {                             // head-major (checked above); host [n_layers][Hkv][R][D]: one piece of R rows per (layer, KV head)
        width = (size_t)a.R * a.D * 2;
        pitch = (size_t)a.kv_head_stride * 2;
        height = a.n_layers * a.Hkv;
      }
      if (p->h_k_window && ok())
        e = cudaMemcpy2DAsync((char*)const_cast<void*>(a.k) + row0, pitch, p->h_k_window, width, width, height,
                              cudaMemcpyHostToDevice, s);
      if (p->h_v_window && ok())
        e = cudaMemcpy2DAsync((char*)const_cast<void*>(a.v) + row0, pitch, p->h_v_window, width, width, height,
                              cudaMemcpyHostToDevice, s);
    }
  }
  if (overlap && side_uploads && p->run_attn && (p->h_q || p->h_k_window || p->h_v_window) && ok()) {
    // the attention's own inputs go first over the link: the accept inputs, needed much later, queue behind them
    e = cudaEventRecord(eb, s);
    if (ok()) e = cudaStreamWaitEvent(cs, eb, 0);
  }
  if (p->run_accept) {
    const size_t B = (size_t)c.batch;
    if (p->h_target_logits && ok())
      e = cudaMemcpyAsync(const_cast<float*>(c.target_logits), p->h_target_logits, B * (c.gamma + 1) * c.V * 4, cudaMemcpyHostToDevice, cs);
    if (p->h_draft_logits && ok())
      e = cudaMemcpyAsync(const_cast<float*>(c.draft_logits), p->h_draft_logits, B * c.gamma * c.V * 4, cudaMemcpyHostToDevice, cs);
    if (p->h_draft_tokens && ok())
      e = cudaMemcpyAsync(const_cast<int*>(c.draft_tokens), p->h_draft_tokens, B * c.gamma * 4, cudaMemcpyHostToDevice, cs);
    if (p->h_uniforms && ok())
      e = cudaMemcpyAsync(const_cast<float*>(c.uniforms), p->h_uniforms, B * (c.gamma + 1) * 4, cudaMemcpyHostToDevice, cs);
  }
  if (!ok()) { set_cuda_error((int)e); return PVLM_ERR_CUDA; }
  // ---- the three stages ----
  // With a second stream, what does not depend on the attention's results runs there: the accept stage and the
  // part of the gather that does not depend on the selection (the rows before and after the visual span).  Both
  // are queued behind an event that the attention records right after its main kernel, so they start when
  // that kernel ends and fill the gap in which the main stream runs the small combine / mass / select kernels
  // and HBM would otherwise idle (queued earlier they would only take SMs from the main kernel's start).
  pvlm_status st;
  const bool accept_on_side = overlap && p->run_accept;
  const bool split_gather = overlap && p->run_prune && p->prune.src_k;
  if (p->run_attn) {
    if (accept_on_side || split_gather) set_after_main_event(eb);
    st = pvlm_verify_attn(&p->attn, stream);
    const bool recorded = take_after_main_event() == nullptr;     // consumed by the launch => eb is recorded
    if (st != PVLM_OK) return st;
    if ((accept_on_side || split_gather) && !recorded) e = cudaEventRecord(eb, s);
  } else if (accept_on_side || split_gather) {
    e = cudaEventRecord(eb, s);
  }
  if ((accept_on_side || split_gather) && ok()) {
    e = cudaStreamWaitEvent(cs, eb, 0);
    forked = true;
  }
  if (!ok()) { set_cuda_error((int)e); return PVLM_ERR_CUDA; }
  if (split_gather && (st = launch_uvprune_parts(p->prune, false, 1, cs)) != PVLM_OK) return st;
  if (accept_on_side) {
    if ((st = pvlm_spec_accept(&p->accept, cs)) != PVLM_OK) return st;
    if (p->h_n_accept && ok())
      e = cudaMemcpyAsync(p->h_n_accept, c.n_accept, (size_t)c.batch * 4, cudaMemcpyDeviceToHost, cs);
    if (p->h_out_tokens && ok())
      e = cudaMemcpyAsync(p->h_out_tokens, c.out_tokens, (size_t)c.batch * (c.gamma + 1) * 4, cudaMemcpyDeviceToHost, cs);
  }
  if (!ok()) { set_cuda_error((int)e); return PVLM_ERR_CUDA; }
  if (p->run_attn && p->h_o) {                                   // o is final: its download may overlap the rest
    const size_t q_layer = (size_t)a.R * a.Hq * a.D * 2;
    if (overlap) {
      e = cudaEventRecord(eb, s);
      if (ok()) e = cudaStreamWaitEvent(cs, eb, 0);
      forked = true;
    }
    if (ok()) e = cudaMemcpy2DAsync(p->h_o, q_layer, a.o, (size_t)a.q_layer_stride * 2, q_layer, a.n_layers, cudaMemcpyDeviceToHost, cs);
    if (!ok()) { set_cuda_error((int)e); return PVLM_ERR_CUDA; }
  }
  if (p->h_attn_status) {          // did a bounded wait inside the attention kernels (this step's, or the last call's) expire?
    AttnPlan plan;
    *p->h_attn_status = 0;
    if (a.workspace && make_attn_plan(a, plan) && plan.use_tc && a.workspace_bytes >= plan.total && ok())
      e = cudaMemcpyAsync(p->h_attn_status, (const char*)a.workspace + plan.off_tc + plan.tc.off_status, 4, cudaMemcpyDeviceToHost, s);
  }
  if (p->run_prune) {
    st = split_gather ? launch_uvprune_parts(p->prune, true, 2, s) : pvlm_uvprune_select_gather(&p->prune, stream);
    if (st != PVLM_OK) return st;
  }
  if (p->run_accept && !accept_on_side && (st = pvlm_spec_accept(&p->accept, stream)) != PVLM_OK) return st;
  // ---- device -> host: the rest of this step's results ----
  if (p->run_prune && p->h_kept_idx && p->prune.k > 0 && ok())
    e = cudaMemcpyAsync(p->h_kept_idx, p->prune.kept_idx, (size_t)p->prune.k * 4, cudaMemcpyDeviceToHost, s);
  if (p->run_accept && !accept_on_side && p->h_n_accept && ok())
    e = cudaMemcpyAsync(p->h_n_accept, c.n_accept, (size_t)c.batch * 4, cudaMemcpyDeviceToHost, s);
  if (p->run_accept && !accept_on_side && p->h_out_tokens && ok())
    e = cudaMemcpyAsync(p->h_out_tokens, c.out_tokens, (size_t)c.batch * (c.gamma + 1) * 4, cudaMemcpyDeviceToHost, s);
  // A forked side stream is joined back here, so that synchronising `stream` alone covers everything and a stream
  // capture of the call closes.
  if (overlap && forked && ok()) e = cudaEventRecord(ea, cs);
  if (overlap && forked && ok()) e = cudaStreamWaitEvent(s, ea, 0);
  if (!ok()) { set_cuda_error((int)e); return PVLM_ERR_CUDA; }
  return PVLM_OK;
}

int pvlm_window_size(double t_target, double t_draft, int mode) {
  if (!(t_target > 0.0) || !(t_draft > 0.0)) return 0;
  const double c = t_target / t_draft;
  double g;
  if (mode == PVLM_ROUND_NEAREST) g = floor(c + 0.5);
  else if (mode == PVLM_ROUND_DOWN) g = floor(c + 1e-9);
  else if (mode == PVLM_ROUND_UP) g = ceil(c - 1e-9);
  else return 0;
  if (g < 1.0) g = 1.0;
  if (g > 1e9) g = 1e9;
  return (int)g;
}

}  // extern "C"
