// Token-wise acceptance rate of a given text: one streaming pass over the 2N logit rows.
//   rate_row_kernel  : one CTA per logit row, online (max, sum exp) per thread, fixed-order merge
//   rate_test_kernel : lse in fp64, p(x), q(x), the fp32 accept test, count
#include "pvlm_common.cuh"

namespace pvlm {

namespace {

constexpr int kRowThreads = 512;

struct RateArgs {
  const float *tl, *dl;
  long long trs, drs;
  const int* tok;
  const float* u;
  int N, V, vec_ok, n0;
  float inv_temp;
  int* accepted;
  float *p_tok, *q_tok;
  int* n_accepted;
  float2* stats;        // [2][N] (max of raw logits, sum exp((x - max) / temp))
};

__device__ __forceinline__ float ex2r(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void merge2(float& m, float& l, float m2, float l2, float c) {
  const float mn = fmaxf(m, m2);
  if (mn == -INFINITY) { m = mn; l = 0.f; return; }
  l = l * ex2r((m - mn) * c) + l2 * ex2r((m2 - mn) * c);
  m = mn;
}

__global__ void __launch_bounds__(kRowThreads) rate_row_kernel(const RateArgs a) {
  const int n = a.n0 + blockIdx.x, model = blockIdx.y;
  const float* x = model == 0 ? a.tl + (long long)n * a.trs : a.dl + (long long)n * a.drs;
  const float c = a.inv_temp * kLog2e;
  float m = -INFINITY, l = 0.f;
  auto take4 = [&](float v0, float v1, float v2, float v3) {
    const float m4 = fmaxf(fmaxf(v0, v1), fmaxf(v2, v3));
    if (m4 > m) {                      // rare once the running maximum has settled
      l *= ex2r((m - m4) * c);         // m = -inf: l is 0 and ex2(-inf) = 0
      m = m4;
    }
    if (m != -INFINITY) l += (ex2r((v0 - m) * c) + ex2r((v1 - m) * c)) + (ex2r((v2 - m) * c) + ex2r((v3 - m) * c));
  };
  if (a.vec_ok) {
    const float4* x4 = reinterpret_cast<const float4*>(x);
    const int n4 = a.V >> 2;
    int i = threadIdx.x;
    for (; i + 3 * kRowThreads < n4; i += 4 * kRowThreads) {          // four independent 16-byte loads in flight
      const float4 t0 = __ldg(x4 + i), t1 = __ldg(x4 + i + kRowThreads), t2 = __ldg(x4 + i + 2 * kRowThreads),
                   t3 = __ldg(x4 + i + 3 * kRowThreads);
      take4(t0.x, t0.y, t0.z, t0.w);
      take4(t1.x, t1.y, t1.z, t1.w);
      take4(t2.x, t2.y, t2.z, t2.w);
      take4(t3.x, t3.y, t3.z, t3.w);
    }
    for (; i < n4; i += kRowThreads) {
      const float4 t = __ldg(x4 + i);
      take4(t.x, t.y, t.z, t.w);
    }
    for (int j = (n4 << 2) + threadIdx.x; j < a.V; j += kRowThreads) take4(__ldg(x + j), -INFINITY, -INFINITY, -INFINITY);
  } else {
    for (int j = threadIdx.x; j < a.V; j += kRowThreads) take4(__ldg(x + j), -INFINITY, -INFINITY, -INFINITY);
  }
#pragma unroll
  for (int sh = 16; sh >= 1; sh >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, sh), l2 = __shfl_xor_sync(0xffffffffu, l, sh);
    merge2(m, l, m2, l2, c);
  }
  __shared__ float sm[kRowThreads / 32], sl[kRowThreads / 32];
  if ((threadIdx.x & 31) == 0) { sm[threadIdx.x >> 5] = m; sl[threadIdx.x >> 5] = l; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < kRowThreads / 32; ++w) merge2(m, l, sm[w], sl[w], c);
    a.stats[(long long)model * a.N + n] = make_float2(m, l);
  }
}

__global__ void __launch_bounds__(256) rate_test_kernel(const RateArgs a) {
  const int n = blockIdx.x * 256 + threadIdx.x;
  int ok = 0;
  if (n < a.N) {
    const int x = a.tok[n];
    float p = 0.f, q = 1.f;
    if (x >= 0 && x < a.V) {
      const float2 sp = a.stats[n], sq = a.stats[(long long)a.N + n];
      const double lp = (double)sp.x * (double)a.inv_temp + log((double)sp.y);
      const double lq = (double)sq.x * (double)a.inv_temp + log((double)sq.y);
      p = (float)exp((double)a.tl[(long long)n * a.trs + x] * (double)a.inv_temp - lp);
      q = (float)exp((double)a.dl[(long long)n * a.drs + x] * (double)a.inv_temp - lq);
    }
    ok = __fmul_rn(a.u[n], q) < p;
    a.accepted[n] = ok;
    if (a.p_tok) a.p_tok[n] = p;
    if (a.q_tok) a.q_tok[n] = q;
  }
  const int cnt = __syncthreads_count(ok);
  if (threadIdx.x == 0 && cnt) atomicAdd(a.n_accepted, cnt);       // integer: the total does not depend on the order
}

}  // namespace

}  // namespace pvlm

using namespace pvlm;

extern "C" {

size_t pvlm_acceptance_rate_workspace_bytes(const pvlm_rate_params* p) {
  if (!p || p->N < 0 || p->N >= (1 << 30)) return 0;
  return align_up((size_t)2 * (p->N > 0 ? p->N : 1) * sizeof(float2), 256);
}

pvlm_status pvlm_acceptance_rate(const pvlm_rate_params* p, void* stream) {
  if (!p) return PVLM_ERR_INVALID_ARG;
  if (p->N < 0 || p->N >= (1 << 30) || p->V < 1 || p->temperature < 0.f || !p->n_accepted) return PVLM_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  cudaError_t e = cudaMemsetAsync(p->n_accepted, 0, sizeof(int), s);
  if (e != cudaSuccess) { set_cuda_error((int)e); return PVLM_ERR_CUDA; }
  if (p->N == 0) return PVLM_OK;
  if (!p->target_logits || !p->draft_logits || !p->tokens || !p->uniforms || !p->accepted) return PVLM_ERR_INVALID_ARG;
  if (p->target_row_stride < p->V || p->draft_row_stride < p->V) return PVLM_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(p->target_logits) % 4 || reinterpret_cast<uintptr_t>(p->draft_logits) % 4) return PVLM_ERR_INVALID_ARG;
  const size_t need = pvlm_acceptance_rate_workspace_bytes(p);
  if (!p->workspace || reinterpret_cast<uintptr_t>(p->workspace) % 256 || p->workspace_bytes < need) return PVLM_ERR_WORKSPACE;
  RateArgs a;
  a.tl = p->target_logits; a.dl = p->draft_logits;
  a.trs = p->target_row_stride; a.drs = p->draft_row_stride;
  a.tok = p->tokens; a.u = p->uniforms;
  a.N = p->N; a.V = p->V;
  a.vec_ok = reinterpret_cast<uintptr_t>(a.tl) % 16 == 0 && reinterpret_cast<uintptr_t>(a.dl) % 16 == 0 && a.trs % 4 == 0 && a.drs % 4 == 0;
  a.inv_temp = (p->temperature == 0.f || p->temperature == 1.f) ? 1.f : 1.f / p->temperature;
  a.accepted = p->accepted; a.p_tok = p->p_tok; a.q_tok = p->q_tok; a.n_accepted = p->n_accepted;
  a.stats = (float2*)p->workspace;
  for (int n0 = 0; n0 < p->N; n0 += 32768) {            // launches of bounded size
    a.n0 = n0;
    const int cnt = p->N - n0 < 32768 ? p->N - n0 : 32768;
    rate_row_kernel<<<dim3(cnt, 2), kRowThreads, 0, s>>>(a);
  }
  rate_test_kernel<<<ceil_div(p->N, 256), 256, 0, s>>>(a);
  return check_launch();
}

}  // extern "C"
