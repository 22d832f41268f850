// Vision-text similarity signal of UV-Prune on the target's token representations:
//   sim_i = sum_j cos(V_i, X_j) = (V_i / |V_i|) . u,   u = sum_j X_j / |X_j|
// so one layer costs one pass over the text rows (u) and one pass over the visual rows.
// All sums run in a fixed order (no float atomics): results are run-to-run deterministic.
#include "pvlm_common.cuh"

namespace pvlm {

namespace {

constexpr int kSimRowChunks = 64;      // text rows are summed in this many independent slices

struct SimArgs {
  const __nv_bfloat16* h;
  long long row_stride;
  int vis_start, m, text_start, n, d;
  float* sim;
  float* inv_norm;   // [n]
  float* u_part;     // [kSimRowChunks][d]
  float* u;          // [d]
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

// 1 / |X_j| per text row (0 for a zero row): one warp per row.
__global__ void __launch_bounds__(256) sim_text_norm_kernel(const SimArgs a) {
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (row >= a.n) return;
  const uint4* src = reinterpret_cast<const uint4*>(a.h + (long long)(a.text_start + row) * a.row_stride);
  float acc = 0.f;
  for (int c = lane; c < a.d / 8; c += 32) {
    float f[8];
    unpack8(__ldg(src + c), f);
#pragma unroll
    for (int e = 0; e < 8; ++e) acc = fmaf(f[e], f[e], acc);
  }
  acc = warp_sum(acc);
  if (lane == 0) a.inv_norm[row] = acc > 0.f ? rsqrtf(acc) : 0.f;
}

// Partial column sums of the normalised text rows: grid (ceil(d/8/256), kSimRowChunks).
__global__ void __launch_bounds__(256) sim_text_sum_kernel(const SimArgs a) {
  const int c = blockIdx.x * 256 + threadIdx.x;       // 8-channel group
  if (c >= a.d / 8) return;
  const int rows_per = (a.n + kSimRowChunks - 1) / kSimRowChunks;
  const int r0 = blockIdx.y * rows_per, r1 = min(a.n, r0 + rows_per);
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll 8
  for (int r = r0; r < r1; ++r) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(a.h + (long long)(a.text_start + r) * a.row_stride) + c);
    const float w = a.inv_norm[r];
    float f[8];
    unpack8(v, f);
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = fmaf(f[e], w, acc[e]);
  }
  float* dst = a.u_part + (long long)blockIdx.y * a.d + c * 8;
#pragma unroll
  for (int e = 0; e < 8; ++e) dst[e] = acc[e];
}

__global__ void __launch_bounds__(256) sim_text_reduce_kernel(const SimArgs a) {
  const int c = blockIdx.x * 256 + threadIdx.x;
  if (c >= a.d) return;
  float acc = 0.f;
  for (int k = 0; k < kSimRowChunks; ++k) acc += a.u_part[(long long)k * a.d + c];
  a.u[c] = acc;
}

// sim_i = (V_i . u) / |V_i|: u staged in shared memory, one warp per visual row, 16-byte loads.
__global__ void __launch_bounds__(256) sim_visual_kernel(const SimArgs a) {
  extern __shared__ float s_u[];
  for (int c = threadIdx.x; c < a.d; c += 256) s_u[c] = a.u[c];
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int row = blockIdx.x * 8 + warp; row < a.m; row += gridDim.x * 8) {
    const uint4* src = reinterpret_cast<const uint4*>(a.h + (long long)(a.vis_start + row) * a.row_stride);
    float dot = 0.f, nrm = 0.f;
#pragma unroll 4
    for (int c = lane; c < a.d / 8; c += 32) {
      float f[8];
      unpack8(__ldg(src + c), f);
      const float4 u0 = *reinterpret_cast<const float4*>(s_u + c * 8), u1 = *reinterpret_cast<const float4*>(s_u + c * 8 + 4);
      dot = fmaf(f[0], u0.x, dot); dot = fmaf(f[1], u0.y, dot); dot = fmaf(f[2], u0.z, dot); dot = fmaf(f[3], u0.w, dot);
      dot = fmaf(f[4], u1.x, dot); dot = fmaf(f[5], u1.y, dot); dot = fmaf(f[6], u1.z, dot); dot = fmaf(f[7], u1.w, dot);
#pragma unroll
      for (int e = 0; e < 8; ++e) nrm = fmaf(f[e], f[e], nrm);
    }
    dot = warp_sum(dot);
    nrm = warp_sum(nrm);
    if (lane == 0) a.sim[row] = nrm > 0.f ? dot * rsqrtf(nrm) : 0.f;
  }
}

}  // namespace

size_t similarity_workspace(const pvlm_similarity_params& p) {
  return align_up((size_t)(p.n > 0 ? p.n : 1) * 4, 256) + align_up((size_t)kSimRowChunks * p.d * 4, 256) +
         align_up((size_t)p.d * 4, 256);
}

pvlm_status launch_similarity(const pvlm_similarity_params& p, cudaStream_t s) {
  SimArgs a;
  a.h = (const __nv_bfloat16*)p.hidden;
  a.row_stride = p.hidden_row_stride;
  a.vis_start = p.vis_start; a.m = p.m; a.text_start = p.text_start; a.n = p.n; a.d = p.d;
  a.sim = p.sim;
  char* ws = (char*)p.workspace;
  a.inv_norm = (float*)ws;
  a.u_part = (float*)(ws + align_up((size_t)(p.n > 0 ? p.n : 1) * 4, 256));
  a.u = (float*)((char*)a.u_part + align_up((size_t)kSimRowChunks * p.d * 4, 256));
  if (p.n > 0) sim_text_norm_kernel<<<ceil_div(p.n, 8), 256, 0, s>>>(a);
  sim_text_sum_kernel<<<dim3(ceil_div(p.d / 8, 256), kSimRowChunks), 256, 0, s>>>(a);
  sim_text_reduce_kernel<<<ceil_div(p.d, 256), 256, 0, s>>>(a);
  if (p.m > 0) {
    int blocks = ceil_div(p.m, 8);
    if (blocks > kNumSMs * 16) blocks = kNumSMs * 16;
    const int smem = p.d * 4;
    cudaFuncSetAttribute(sim_visual_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    sim_visual_kernel<<<blocks, 256, smem, s>>>(a);
  }
  return check_launch();
}

}  // namespace pvlm
