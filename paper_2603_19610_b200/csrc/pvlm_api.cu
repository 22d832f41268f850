// C-ABI entry points: host-side argument validation, workspace queries, dispatch.
#include "pvlm_common.cuh"

namespace pvlm {

static thread_local int g_last_cuda_error = 0;

void set_cuda_error(int e) { g_last_cuda_error = e; }

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
    default: return "PVLM_ERR_UNKNOWN";
  }
}

int pvlm_last_cuda_error(void) { return g_last_cuda_error; }

int pvlm_version(void) { return 1000; }

size_t pvlm_verify_attn_workspace_bytes(const pvlm_attn_params* p) {
  AttnPlan plan;
  if (!p || !make_attn_plan(*p, plan)) return 0;
  return plan.total;
}

pvlm_status pvlm_verify_attn(const pvlm_attn_params* p, void* stream) {
  if (!p) return PVLM_ERR_INVALID_ARG;
  if (p->n_layers < 1 || p->R < 1 || p->Hq < 1 || p->Hkv < 1 || p->D < 1 || p->n_ctx < 0) return PVLM_ERR_INVALID_ARG;
  if (!p->q || !p->k || !p->v || !p->o) return PVLM_ERR_INVALID_ARG;
  AttnPlan plan;
  if (!make_attn_plan(*p, plan)) return PVLM_ERR_UNSUPPORTED;
  if (!aligned(p->q, 16) || !aligned(p->k, 16) || !aligned(p->v, 16) || !aligned(p->o, 16)) return PVLM_ERR_INVALID_ARG;
  if (p->kv_head_stride < p->D || p->kv_head_stride % 8) return PVLM_ERR_INVALID_ARG;
  if (p->kv_token_stride < (long long)p->Hkv * p->kv_head_stride || p->kv_token_stride % 8) return PVLM_ERR_INVALID_ARG;
  if (p->n_layers > 1) {
    if (p->kv_layer_stride < (long long)plan.T * p->kv_token_stride || p->kv_layer_stride % 8) return PVLM_ERR_INVALID_ARG;
    if (p->q_layer_stride < (long long)p->R * p->Hq * p->D || p->q_layer_stride % 8) return PVLM_ERR_INVALID_ARG;
    if (p->mass && p->mass_layer_stride < plan.T) return PVLM_ERR_INVALID_ARG;
  }
  if (p->n_layers > 65535 || p->Hkv > 65535) return PVLM_ERR_UNSUPPORTED;
  const pvlm_status w = check_ws(p->workspace, p->workspace_bytes, plan.total);
  if (w != PVLM_OK) return w;
  return launch_verify_attn(*p, plan, (cudaStream_t)stream);
}

size_t pvlm_uvprune_workspace_bytes(const pvlm_prune_params* p) {
  if (!p || p->m < 0) return 0;
  return uvprune_workspace(*p);
}

pvlm_status pvlm_uvprune_select_gather(const pvlm_prune_params* p, void* stream) {
  if (!p) return PVLM_ERR_INVALID_ARG;
  if (p->m < 0 || p->k < 0 || p->k > p->m || p->vis_start < 0) return PVLM_ERR_INVALID_ARG;
  if (p->m > (1 << 24)) return PVLM_ERR_UNSUPPORTED;
  if (p->m > 0 && !p->mass_cur) return PVLM_ERR_INVALID_ARG;
  if (p->k > 0 && !p->kept_idx) return PVLM_ERR_INVALID_ARG;
  const bool gather = p->src_k || p->src_v || p->dst_k || p->dst_v;
  if (gather) {
    if (!p->src_k || !p->src_v || !p->dst_k || !p->dst_v) return PVLM_ERR_INVALID_ARG;
    if (p->n_layers < 1 || p->row_bytes <= 0 || p->src_len < p->vis_start + p->m) return PVLM_ERR_INVALID_ARG;
    if (p->row_bytes % 16) return PVLM_ERR_UNSUPPORTED;
    if (!aligned(p->src_k, 16) || !aligned(p->src_v, 16) || !aligned(p->dst_k, 16) || !aligned(p->dst_v, 16))
      return PVLM_ERR_INVALID_ARG;
    const long long dst_len = (long long)p->src_len - p->m + p->k;
    if (p->n_layers > 1) {
      if (p->src_layer_stride_bytes < (long long)p->src_len * p->row_bytes || p->src_layer_stride_bytes % 16) return PVLM_ERR_INVALID_ARG;
      if (p->dst_layer_stride_bytes < dst_len * p->row_bytes || p->dst_layer_stride_bytes % 16) return PVLM_ERR_INVALID_ARG;
    }
  }
  const pvlm_status w = check_ws(p->workspace, p->workspace_bytes, uvprune_workspace(*p));
  if (w != PVLM_OK) return w;
  return launch_uvprune(*p, (cudaStream_t)stream);
}

size_t pvlm_spec_accept_workspace_bytes(const pvlm_accept_params* p) {
  AcceptPlan plan;
  if (!p || !make_accept_plan(*p, plan)) return 0;
  return plan.total;
}

pvlm_status pvlm_spec_accept(const pvlm_accept_params* p, void* stream) {
  if (!p) return PVLM_ERR_INVALID_ARG;
  if (p->gamma < 1 || p->V < 1 || p->batch < 1) return PVLM_ERR_INVALID_ARG;
  if (!p->target_logits || !p->draft_logits || !p->draft_tokens || !p->uniforms || !p->n_accept || !p->out_tokens)
    return PVLM_ERR_INVALID_ARG;
  AcceptPlan plan;
  if (!make_accept_plan(*p, plan)) return PVLM_ERR_UNSUPPORTED;
  if (p->batch > 65535) return PVLM_ERR_UNSUPPORTED;
  if (!aligned(p->target_logits, 4) || !aligned(p->draft_logits, 4)) return PVLM_ERR_INVALID_ARG;
  if (p->target_row_stride < p->V || p->draft_row_stride < p->V) return PVLM_ERR_INVALID_ARG;
  if (p->batch > 1) {
    // batch stride 0 = every sequence reads the same logits
    if (p->target_batch_stride != 0 && (p->target_batch_stride < (long long)(p->gamma + 1) * p->target_row_stride)) return PVLM_ERR_INVALID_ARG;
    if (p->draft_batch_stride != 0 && (p->draft_batch_stride < (long long)p->gamma * p->draft_row_stride)) return PVLM_ERR_INVALID_ARG;
  }
  if (p->temperature < 0.f) return PVLM_ERR_INVALID_ARG;
  const pvlm_status w = check_ws(p->workspace, p->workspace_bytes, plan.total);
  if (w != PVLM_OK) return w;
  return launch_spec_accept(*p, plan, (cudaStream_t)stream);
}

}  // extern "C"
