// Shared host/device helpers of the pvlm library (internal).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include "pvlm.h"

namespace pvlm {

constexpr int kNumSMs = 148;          // B200: 2 dies x 74 SMs
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline int ceil_div(long long a, long long b) { return (int)((a + b - 1) / b); }

// ---- programmatic dependent launch ------------------------------------------------------------------
// A kernel lets the next one in the stream start its CTAs early (pdl_launch_dependents, at its top), and that one
// blocks in pdl_wait until every kernel before it has completed and their writes are visible.  Rule for kernels
// launched with launch_dependent(): everything read that an earlier kernel of the same call wrote, and every
// write to memory an earlier kernel may still read, comes after pdl_wait; only work on the call's own inputs
// (index arithmetic, barrier set-up, loads of caller-provided tensors) may precede it.  Both instructions are
// no-ops when the launch carries no dependency.  PVLM_PDL=0 in the environment launches everything plainly.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif
bool pdl_enabled();
// Current value of a process-wide switch (pvlm_set_option; the default comes from the environment, read once).
int option_value(int option);

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  if (pdl_enabled()) {
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
  }
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Records a failed launch for pvlm_last_cuda_error(); returns PVLM_ERR_CUDA or PVLM_OK.
pvlm_status check_launch();
void set_cuda_error(int e);

// A cudaEvent_t that the next attention launch of this host thread records right after its main kernel
// (before the combine / mass kernels).  take_* returns the pending event (nullptr once a launch has used it)
// and clears it.
void set_after_main_event(cudaEvent_t ev);
cudaEvent_t take_after_main_event();

// ---- verify attention -----------------------------------------------------
constexpr int kAttnBN = 64;           // keys per tile

struct AttnTcPlan {           // tensor-core (tcgen05) path, D = 128
  int nrp;                    // query rows per KV head padded to a multiple of 16
  int T, tiles_per_item, n_cta, seg_max;
  long long total_tiles;
  size_t off_part_o, off_part_ml, off_status, total;   // relative to the path's workspace region
};
bool make_attn_tc_plan(const pvlm_attn_params& p, AttnTcPlan& plan);
pvlm_status launch_verify_attn_tc(const pvlm_attn_params& p, const AttnTcPlan& plan, char* ws, float* lse2, cudaStream_t s);
// mass pass on the tensor-core path: needs lse2 of every row (log2 domain) and a [n_mass][Hkv][T_pad] scratch
pvlm_status launch_attn_mass_tc(const pvlm_attn_params& p, const float* lse2, float* part_mass, int* status, cudaStream_t s);

struct AttnPlan {
  bool use_tc;     // main pass on tcgen05; the mma.sync kernel still runs the mass pass
  AttnTcPlan tc;
  size_t off_tc;
  int rows;        // G * R valid rows per KV head
  int n_warps;     // 16-row MMA tiles (one warp each)
  int rows_pad;    // n_warps * 16
  int T;           // keys per layer
  int tiles;       // ceil(T / kAttnBN)
  int splits;      // key-range splits per (layer, KV head)
  int tiles_per_split;
  size_t off_part_o, off_part_ml, off_lse2, off_part_mass, total;   // workspace layout (bytes)
};
bool make_attn_plan(const pvlm_attn_params& p, AttnPlan& plan);

pvlm_status launch_verify_attn(const pvlm_attn_params& p, const AttnPlan& plan, cudaStream_t s);

// ---- uvprune ----------------------------------------------------------------
pvlm_status launch_uvprune(const pvlm_prune_params& p, cudaStream_t s);
pvlm_status launch_uvprune_parts(const pvlm_prune_params& p, bool select, int part, cudaStream_t s);
size_t uvprune_workspace(const pvlm_prune_params& p);

// ---- similarity (hidden-state criterion) --------------------------------------------
size_t similarity_workspace(const pvlm_similarity_params& p);
pvlm_status launch_similarity(const pvlm_similarity_params& p, cudaStream_t s);

// ---- accept -----------------------------------------------------------------
struct AcceptPlan {
  int rows;             // 2 * gamma + 1 logit rows per sequence
  int n_stat_chunks;    // statistics CTAs per row
  int stat_chunk;       // elements per statistics CTA
  int team;             // CTAs of the tail team per sequence (cluster size)
  int nit;              // residual-pass iterations per warp of the team
  size_t off_stats, off_lse, off_sync, total;
};
bool make_accept_plan(const pvlm_accept_params& p, AcceptPlan& plan);
pvlm_status launch_spec_accept(const pvlm_accept_params& p, const AcceptPlan& plan, cudaStream_t s);
pvlm_status launch_accept_from_probs(const float* p_tok, const float* q_tok, const float* uniforms, long long u_stride,
                                     int gamma, int batch, int* n_accept, cudaStream_t s);

}  // namespace pvlm
