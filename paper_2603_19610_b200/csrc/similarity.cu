// Vision-text similarity signal of UV-Prune on the target's token representations:
//   sim_i = sum_j cos(V_i, X_j) = (V_i / |V_i|) . u,   u = sum_j X_j / |X_j|
// so one layer costs one pass over the text rows (u) and one pass over the visual rows.
// A call may carry several layers (the variation score needs two): every kernel then covers all of them in one
// launch, so the launch, drain and fill of the latency-bound text kernels are paid once.
// All sums run in a fixed order (no float atomics): results are run-to-run deterministic.
#include "pvlm_common.cuh"

namespace pvlm {

namespace {


struct SimArgs {
  const __nv_bfloat16* h;
  long long row_stride;
  int vis_start, m, text_start, n, d;
  int n_layers, parts;           // layers of the call; text CTAs per layer
  long long layer_stride;        // elements between the layers' hidden states
  long long sim_stride;          // elements between the layers' outputs
  float* sim;
  float* u_part;     // [layer][text CTAs][d]
  float* u;          // [layer][d]
};

__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 t = __bfloat1622float2(p[i]);
    f[2 * i] = t.x;
    f[2 * i + 1] = t.y;
  }
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int sh = 16; sh >= 1; sh >>= 1) v += __shfl_xor_sync(0xffffffffu, v, sh);
  return v;
}

constexpr int kSimRowsPerCta = 8;      // text rows per CTA of the text pass (one per warp)

// Text pass, one read of the text rows from HBM: a CTA takes 8 consecutive rows; each warp computes 1 / |X_j| of
// one of them (0 for a zero row), then every thread sums its 8-channel groups over the 8 rows in row order
// (the rows come back from L1 / L2) and writes one partial of u.  Fixed order everywhere: deterministic.
__global__ void __launch_bounds__(256) sim_text_kernel(const SimArgs a) {
  __shared__ float s_inv[kSimRowsPerCta];
  pdl_launch_dependents();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int r0 = blockIdx.x * kSimRowsPerCta;
  const __nv_bfloat16* h = a.h + (long long)blockIdx.y * a.layer_stride;       // this CTA's layer
  for (int k = warp; k < kSimRowsPerCta; k += 8) {
    const int row = r0 + k;
    float acc = 0.f;
    if (row < a.n) {
      const uint4* src = reinterpret_cast<const uint4*>(h + (long long)(a.text_start + row) * a.row_stride);
      const int n4 = a.d / 8;
      int c = lane;
      for (; c + 7 * 32 < n4; c += 8 * 32) {              // eight 16-byte loads in flight per lane
        uint4 v[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = __ldg(src + c + i * 32);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          float f[8];
          unpack8(v[i], f);
#pragma unroll
          for (int e = 0; e < 8; ++e) acc = fmaf(f[e], f[e], acc);
        }
      }
      if (c < n4) {                                         // the remainder as one batch too (zeros add nothing)
        uint4 v[7];
#pragma unroll
        for (int i = 0; i < 7; ++i) v[i] = c + i * 32 < n4 ? __ldg(src + c + i * 32) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int i = 0; i < 7; ++i) {
          float f[8];
          unpack8(v[i], f);
#pragma unroll
          for (int e = 0; e < 8; ++e) acc = fmaf(f[e], f[e], acc);
        }
      }
    }
    acc = warp_sum(acc);
    if (lane == 0) s_inv[k] = acc > 0.f ? rsqrtf(acc) : 0.f;
  }
  __syncthreads();
  const int rows = min(kSimRowsPerCta, a.n - r0);
  for (int c = threadIdx.x; c < a.d / 8; c += 256) {
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    uint4 v[kSimRowsPerCta];
#pragma unroll
    for (int k = 0; k < kSimRowsPerCta; ++k)                 // all eight loads in flight, then a fixed-order sum
      v[k] = k < rows ? __ldg(reinterpret_cast<const uint4*>(h + (long long)(a.text_start + r0 + k) * a.row_stride) + c)
                      : make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int k = 0; k < kSimRowsPerCta; ++k) {
      const float w = k < rows ? s_inv[k] : 0.f;
      float f[8];
      unpack8(v[k], f);
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[e] = fmaf(f[e], w, acc[e]);
    }
    float* dst = a.u_part + ((long long)blockIdx.y * a.parts + blockIdx.x) * a.d + c * 8;
    *reinterpret_cast<float4*>(dst) = make_float4(acc[0], acc[1], acc[2], acc[3]);
    *reinterpret_cast<float4*>(dst + 4) = make_float4(acc[4], acc[5], acc[6], acc[7]);
  }
}

// u = sum of the partials: a CTA owns 32 channels (a lane each); its 8 warps take the partials round-robin with eight
// loads in flight each, and their sums are merged in warp order.  The order is fixed: deterministic.
__global__ void __launch_bounds__(256) sim_text_reduce_kernel(const SimArgs a, int n_part) {
  __shared__ float s_sum[8][32];
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int c = blockIdx.x * 32 + lane;
  const float* part = a.u_part + (long long)blockIdx.y * a.parts * a.d;      // this CTA's layer
  float sacc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  if (c < a.d) {
    int k = warp;
    for (; k + 56 < n_part; k += 64) {                     // eight loads in flight per lane
      float v[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = part[(long long)(k + 8 * i) * a.d + c];
#pragma unroll
      for (int i = 0; i < 8; ++i) sacc[i] += v[i];
    }
    for (; k < n_part; k += 8) sacc[0] += part[(long long)k * a.d + c];
  }
  s_sum[warp][lane] = ((sacc[0] + sacc[1]) + (sacc[2] + sacc[3])) + ((sacc[4] + sacc[5]) + (sacc[6] + sacc[7]));
  __syncthreads();
  if (warp == 0 && c < a.d) {
    float t = s_sum[0][lane];
#pragma unroll
    for (int w = 1; w < 8; ++w) t += s_sum[w][lane];
    a.u[(long long)blockIdx.y * a.d + c] = t;
  }
}

// sim_i = (V_i . u) / |V_i|: u staged in shared memory, one warp per visual row, 16-byte loads.  The grid is sized
// to what is resident at once, and every warp fetches the first batch of its first row BEFORE it waits for u: the
// hidden states are inputs of the call, so the memory system fills while the latency-bound text kernels still run.
constexpr int kSimBatch = 10;          // 16-byte loads in flight per lane (5 and 4 with more CTAs per SM measured slower)
__global__ void __launch_bounds__(256) sim_visual_kernel(const SimArgs a) {
  extern __shared__ float s_u[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const __nv_bfloat16* h = a.h + (long long)blockIdx.y * a.layer_stride;       // this CTA's layer
  float* sim = a.sim + (long long)blockIdx.y * a.sim_stride;
  const int n4 = a.d / 8;
  int row = blockIdx.x * 8 + warp;
  uint4 v[kSimBatch];
  const bool early = row < a.m && lane + (kSimBatch - 1) * 32 < n4;
  if (early) {
    const uint4* src = reinterpret_cast<const uint4*>(h + (long long)(a.vis_start + row) * a.row_stride);
#pragma unroll
    for (int i = 0; i < kSimBatch; ++i) v[i] = __ldg(src + lane + i * 32);
  }
  pdl_wait();
  for (int c = threadIdx.x; c < a.d; c += 256) s_u[c] = __ldcg(a.u + (long long)blockIdx.y * a.d + c);
  __syncthreads();
  bool have = early;
  for (; row < a.m; row += gridDim.x * 8) {
    const uint4* src = reinterpret_cast<const uint4*>(h + (long long)(a.vis_start + row) * a.row_stride);
    float dot = 0.f, nrm = 0.f;
    auto take = [&](const uint4& x, int c) {
      float f[8];
      unpack8(x, f);
      const float4 u0 = *reinterpret_cast<const float4*>(s_u + c * 8), u1 = *reinterpret_cast<const float4*>(s_u + c * 8 + 4);
      dot = fmaf(f[0], u0.x, dot); dot = fmaf(f[1], u0.y, dot); dot = fmaf(f[2], u0.z, dot); dot = fmaf(f[3], u0.w, dot);
      dot = fmaf(f[4], u1.x, dot); dot = fmaf(f[5], u1.y, dot); dot = fmaf(f[6], u1.z, dot); dot = fmaf(f[7], u1.w, dot);
#pragma unroll
      for (int e = 0; e < 8; ++e) nrm = fmaf(f[e], f[e], nrm);
    };
    int c = lane;
    for (; c + (kSimBatch - 1) * 32 < n4; c += kSimBatch * 32) {
      if (!have) {
#pragma unroll
        for (int i = 0; i < kSimBatch; ++i) v[i] = __ldg(src + c + i * 32);
      }
      have = false;
#pragma unroll
      for (int i = 0; i < kSimBatch; ++i) take(v[i], c + i * 32);
    }
    for (; c < n4; c += 32) take(__ldg(src + c), c);
    dot = warp_sum(dot);
    nrm = warp_sum(nrm);
    if (lane == 0) sim[row] = nrm > 0.f ? dot * rsqrtf(nrm) : 0.f;
  }
}

}  // namespace

static int sim_text_parts(int n) { return n > 0 ? ceil_div(n, kSimRowsPerCta) : 1; }
static int sim_layers(const pvlm_similarity_params& p) { return p.n_layers > 1 ? p.n_layers : 1; }

size_t similarity_workspace(const pvlm_similarity_params& p) {
  const size_t L = (size_t)sim_layers(p);
  return align_up(L * sim_text_parts(p.n) * p.d * 4, 256) + align_up(L * p.d * 4, 256);
}

pvlm_status launch_similarity(const pvlm_similarity_params& p, cudaStream_t s) {
  SimArgs a;
  const int L = sim_layers(p);
  a.h = (const __nv_bfloat16*)p.hidden;
  a.row_stride = p.hidden_row_stride;
  a.vis_start = p.vis_start; a.m = p.m; a.text_start = p.text_start; a.n = p.n; a.d = p.d;
  a.n_layers = L;
  a.layer_stride = L > 1 ? p.hidden_layer_stride : 0;
  a.sim_stride = L > 1 ? p.sim_layer_stride : 0;
  a.sim = p.sim;
  char* ws = (char*)p.workspace;
  const int parts = sim_text_parts(p.n);
  a.parts = parts;
  a.u_part = (float*)ws;
  a.u = (float*)(ws + align_up((size_t)L * parts * p.d * 4, 256));
  // the second and third kernel are launched as programmatic dependents of the one before (see pdl_wait)
  cudaError_t e = cudaSuccess;
  if (p.n > 0) sim_text_kernel<<<dim3(parts, L), 256, 0, s>>>(a);
  e = launch_dependent(sim_text_reduce_kernel, dim3(ceil_div(p.d, 32), L), dim3(256), 0, s, a, p.n > 0 ? parts : 0);
  if (e == cudaSuccess && p.m > 0) {
    const int smem = p.d * 4;
    e = cudaFuncSetAttribute(sim_visual_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    int per_sm = 0;
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, sim_visual_kernel, 256, smem);
    int blocks = ceil_div(p.m, 8);
    const int cap = kNumSMs * (per_sm > 0 ? per_sm : 1) / L;           // every CTA of every layer resident at once
    if (blocks > cap) blocks = cap > 1 ? cap : 1;
    if (e == cudaSuccess) e = launch_dependent(sim_visual_kernel, dim3(blocks, L), dim3(256), smem, s, a);
  }
  if (e != cudaSuccess) { set_cuda_error((int)e); return PVLM_ERR_CUDA; }
  return check_launch();
}

}  // namespace pvlm
