// Window-verify GQA attention + attention mass: split-K flash-decoding.
//
// One CTA owns a contiguous key range of one (layer, KV head); each warp owns
// 16 of the G*R query rows (row = r*G + g), so every K/V byte staged in shared
// memory is used by all query rows of the group.  Scores and PV products run
// on the tensor cores (bf16 in, fp32 accumulate); softmax statistics stay fp32.
// Key ranges are merged by a log-sum-exp combine.  The mass pass re-reads K
// with the final lse, because per-key mass sums probabilities of rows with
// different normalisers and cannot be rescaled after the fact.
#include "pvlm_common.cuh"

#include <cstdlib>
#include <cstring>

namespace pvlm {

namespace {

struct AttnArgs {
  const __nv_bfloat16 *q, *k, *v;
  __nv_bfloat16* o;
  float* lse;        // user lse (natural log), nullable
  float* mass;       // user mass, nullable
  float *part_o, *part_ml, *lse2, *part_mass;
  int R, Hq, Hkv, G, n_ctx, T, T_pad, rows, rows_pad, splits, tiles_per_split, tiles;
  long long q_ls, kv_ls, kv_ts, kv_hs, mass_ls;
  float scale_log2;
  int n_mass;            // mass rows to produce
  int mass_layer[8];     // layer of mass row i (when listed; identity otherwise)
  int mass_listed;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

constexpr int kStages = 3;

// MODE 0: online-softmax attention over the CTA's key range (partials or final O).
// MODE 1: mass pass: P = exp2(s - lse2) summed over the group's rows per key.
// MAXW = most warps a CTA may have: up to 6 warps the register budget is held to 168 so that
// two CTAs (3 warps per scheduler) stay resident per SM.
template <int D, int MODE, int MAXW>
__global__ void __launch_bounds__(MAXW * 32, MAXW <= 6 ? 2 : 1) attn_kernel(const AttnArgs a) {
  constexpr int BN = kAttnBN;
  constexpr int CHUNKS = D / 8;
  constexpr int ROW_BYTES = D * 2;
  constexpr int TILE_BYTES = BN * ROW_BYTES;
  constexpr int STAGE_BYTES = (MODE == 0 ? 2 : 1) * TILE_BYTES;
  extern __shared__ __align__(128) unsigned char smem[];
  const uint32_t smem_base = smem_u32(smem);
  float* colsum = reinterpret_cast<float*>(smem + kStages * STAGE_BYTES);   // MODE 1 only: [8][BN]

  const int split = blockIdx.x, kvh = blockIdx.y;
  const int zrow = blockIdx.z;            // MODE 0: the layer; MODE 1: the mass row
  const int layer = (MODE == 1 && a.mass_listed) ? a.mass_layer[zrow] : zrow;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile_begin = split * a.tiles_per_split;
  const int n_tiles = min(a.tiles, tile_begin + a.tiles_per_split) - tile_begin;

  // ---- this thread's two query rows and their Q fragments ----
  const int row_lo = warp * 16 + (lane >> 2), row_hi = row_lo + 8;
  const bool ok_lo = row_lo < a.rows, ok_hi = row_hi < a.rows;
  const int r_lo = ok_lo ? row_lo / a.G : 0, g_lo = ok_lo ? row_lo % a.G : 0;
  const int r_hi = ok_hi ? row_hi / a.G : 0, g_hi = ok_hi ? row_hi % a.G : 0;
  const int kmax_lo = a.n_ctx + r_lo, kmax_hi = a.n_ctx + r_hi;      // last visible key of each row
  const __nv_bfloat16* qb = a.q + (long long)layer * a.q_ls;
  const __nv_bfloat16* q_lo = qb + ((long long)r_lo * a.Hq + kvh * a.G + g_lo) * D;
  const __nv_bfloat16* q_hi = qb + ((long long)r_hi * a.Hq + kvh * a.G + g_hi) * D;
  uint32_t qf[D / 16][4];
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks) {
    const int col = ks * 16 + 2 * (lane & 3);
    qf[ks][0] = ok_lo ? *reinterpret_cast<const uint32_t*>(q_lo + col) : 0u;
    qf[ks][1] = ok_hi ? *reinterpret_cast<const uint32_t*>(q_hi + col) : 0u;
    qf[ks][2] = ok_lo ? *reinterpret_cast<const uint32_t*>(q_lo + col + 8) : 0u;
    qf[ks][3] = ok_hi ? *reinterpret_cast<const uint32_t*>(q_hi + col + 8) : 0u;
  }

  const __nv_bfloat16* kbase = a.k + (long long)layer * a.kv_ls + (long long)kvh * a.kv_hs;
  const __nv_bfloat16* vbase = a.v + (long long)layer * a.kv_ls + (long long)kvh * a.kv_hs;
  auto load_tile = [&](int stage, int tile) {
    const int j0 = tile * BN;
    const uint32_t sb = smem_base + stage * STAGE_BYTES;
    for (int c = threadIdx.x; c < BN * CHUNKS; c += blockDim.x) {
      const int row = c / CHUNKS, ch = c % CHUNKS;
      const int j = j0 + row;
      const bool ok = j < a.T;
      const long long off = (long long)(ok ? j : 0) * a.kv_ts + ch * 8;
      const uint32_t dst = sb + row * ROW_BYTES + ((ch ^ (row & 7)) << 4);
      cp_async_16(dst, kbase + off, ok ? 16 : 0);
      if (MODE == 0) cp_async_16(dst + TILE_BYTES, vbase + off, ok ? 16 : 0);
    }
  };

  float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;
  float oacc[MODE == 0 ? D / 8 : 1][4];
#pragma unroll
  for (int i = 0; i < (MODE == 0 ? D / 8 : 1); ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
  float lse2_lo = INFINITY, lse2_hi = INFINITY;
  if (MODE == 1) {
    const float* l2 = a.lse2 + (long long)layer * a.Hq * a.R;
    if (ok_lo) lse2_lo = l2[(kvh * a.G + g_lo) * a.R + r_lo];
    if (ok_hi) lse2_hi = l2[(kvh * a.G + g_hi) * a.R + r_hi];
  }

#pragma unroll
  for (int s = 0; s < kStages - 1; ++s) {
    if (s < n_tiles) load_tile(s, tile_begin + s);
    cp_async_commit();
  }

  for (int it = 0; it < n_tiles; ++it) {
    cp_async_wait<kStages - 2>();
    __syncthreads();
    {
      const int nt = it + kStages - 1;
      if (nt < n_tiles) load_tile(nt % kStages, tile_begin + nt);
      cp_async_commit();
    }
    const uint32_t ks_base = smem_base + (it % kStages) * STAGE_BYTES;

    // ---- S = Q K^T for 16 rows x BN keys ----
    float sacc[BN / 8][4];
#pragma unroll
    for (int i = 0; i < BN / 8; ++i) sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f;
    const int mi = lane >> 3, rr = lane & 7;
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
      for (int np = 0; np < BN / 16; ++np) {
        const int token = np * 16 + (mi >> 1) * 8 + rr;
        const int chunk = ks * 2 + (mi & 1);
        uint32_t b[4];
        ldmatrix_x4(b, ks_base + token * ROW_BYTES + ((chunk ^ rr) << 4));
        mma_bf16_16816(sacc[2 * np], qf[ks], b[0], b[1]);
        mma_bf16_16816(sacc[2 * np + 1], qf[ks], b[2], b[3]);
      }
    }

    // ---- scale to log2 domain, mask keys a row must not see ----
    const int j0 = (tile_begin + it) * BN;
    const bool need_mask = (j0 + BN - 1 > a.n_ctx);
#pragma unroll
    for (int nt = 0; nt < BN / 8; ++nt) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float s = sacc[nt][e] * a.scale_log2;
        if (need_mask) {
          const int col = j0 + nt * 8 + 2 * (lane & 3) + (e & 1);
          if (col > (e < 2 ? kmax_lo : kmax_hi)) s = -INFINITY;
        }
        sacc[nt][e] = s;
      }
    }

    if (MODE == 0) {
      float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < BN / 8; ++nt) {
        mx_lo = fmaxf(mx_lo, fmaxf(sacc[nt][0], sacc[nt][1]));
        mx_hi = fmaxf(mx_hi, fmaxf(sacc[nt][2], sacc[nt][3]));
      }
      mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
      mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
      mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
      const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
      const float ms_lo = (mn_lo == -INFINITY) ? 0.f : mn_lo, ms_hi = (mn_hi == -INFINITY) ? 0.f : mn_hi;
      const float c_lo = fast_exp2(m_lo - ms_lo), c_hi = fast_exp2(m_hi - ms_hi);
      m_lo = mn_lo;
      m_hi = mn_hi;
      l_lo *= c_lo;
      l_hi *= c_hi;
#pragma unroll
      for (int i = 0; i < D / 8; ++i) {
        oacc[i][0] *= c_lo;
        oacc[i][1] *= c_lo;
        oacc[i][2] *= c_hi;
        oacc[i][3] *= c_hi;
      }
#pragma unroll
      for (int nt = 0; nt < BN / 8; ++nt) {
        sacc[nt][0] = fast_exp2(sacc[nt][0] - ms_lo);
        sacc[nt][1] = fast_exp2(sacc[nt][1] - ms_lo);
        sacc[nt][2] = fast_exp2(sacc[nt][2] - ms_hi);
        sacc[nt][3] = fast_exp2(sacc[nt][3] - ms_hi);
        l_lo += sacc[nt][0] + sacc[nt][1];
        l_hi += sacc[nt][2] + sacc[nt][3];
      }
      // ---- O += P V ----
      const uint32_t vs_base = ks_base + TILE_BYTES;
#pragma unroll
      for (int kt = 0; kt < BN / 16; ++kt) {
        uint32_t pa[4];
        pa[0] = pack_bf16(sacc[2 * kt][0], sacc[2 * kt][1]);
        pa[1] = pack_bf16(sacc[2 * kt][2], sacc[2 * kt][3]);
        pa[2] = pack_bf16(sacc[2 * kt + 1][0], sacc[2 * kt + 1][1]);
        pa[3] = pack_bf16(sacc[2 * kt + 1][2], sacc[2 * kt + 1][3]);
        const int token = kt * 16 + (mi & 1) * 8 + rr;
#pragma unroll
        for (int nd = 0; nd < D / 16; ++nd) {
          const int chunk = nd * 2 + (mi >> 1);
          uint32_t b[4];
          ldmatrix_x4_trans(b, vs_base + token * ROW_BYTES + ((chunk ^ rr) << 4));
          mma_bf16_16816(oacc[2 * nd], pa, b[0], b[1]);
          mma_bf16_16816(oacc[2 * nd + 1], pa, b[2], b[3]);
        }
      }
    } else {
      // ---- mass: column sums of exp2(s - lse2) over this warp's 16 rows ----
#pragma unroll
      for (int nt = 0; nt < BN / 8; ++nt) {
        float ca = fast_exp2(sacc[nt][0] - lse2_lo) + fast_exp2(sacc[nt][2] - lse2_hi);
        float cb = fast_exp2(sacc[nt][1] - lse2_lo) + fast_exp2(sacc[nt][3] - lse2_hi);
#pragma unroll
        for (int sh = 4; sh <= 16; sh <<= 1) {
          ca += __shfl_xor_sync(0xffffffffu, ca, sh);
          cb += __shfl_xor_sync(0xffffffffu, cb, sh);
        }
        if (lane < 4) {
          colsum[warp * BN + nt * 8 + 2 * lane] = ca;
          colsum[warp * BN + nt * 8 + 2 * lane + 1] = cb;
        }
      }
      __syncthreads();
      for (int t = threadIdx.x; t < BN; t += blockDim.x) {       // a CTA may be a single warp
        if (j0 + t >= a.T) break;
        float acc = 0.f;
        const int nw = blockDim.x >> 5;
        for (int w = 0; w < nw; ++w) acc += colsum[w * BN + t];
        a.part_mass[((long long)zrow * a.Hkv + kvh) * a.T_pad + j0 + t] = acc;
      }
    }
  }
  cp_async_wait<0>();

  if (MODE == 0) {
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
    if (a.splits == 1) {
      const float inv_lo = 1.f / l_lo, inv_hi = 1.f / l_hi;
      __nv_bfloat16* ob = a.o + (long long)layer * a.q_ls;
      if (ok_lo) {
        __nv_bfloat16* dst = ob + ((long long)r_lo * a.Hq + kvh * a.G + g_lo) * D + 2 * (lane & 3);
#pragma unroll
        for (int i = 0; i < D / 8; ++i)
          *reinterpret_cast<uint32_t*>(dst + i * 8) = pack_bf16(oacc[i][0] * inv_lo, oacc[i][1] * inv_lo);
      }
      if (ok_hi) {
        __nv_bfloat16* dst = ob + ((long long)r_hi * a.Hq + kvh * a.G + g_hi) * D + 2 * (lane & 3);
#pragma unroll
        for (int i = 0; i < D / 8; ++i)
          *reinterpret_cast<uint32_t*>(dst + i * 8) = pack_bf16(oacc[i][2] * inv_hi, oacc[i][3] * inv_hi);
      }
      if ((lane & 3) == 0) {
        const long long lb = (long long)layer * a.Hq * a.R;
        if (ok_lo) {
          const float v2 = m_lo + log2f(l_lo);
          a.lse2[lb + (kvh * a.G + g_lo) * a.R + r_lo] = v2;
          if (a.lse) a.lse[lb + (kvh * a.G + g_lo) * a.R + r_lo] = v2 * kLn2;
        }
        if (ok_hi) {
          const float v2 = m_hi + log2f(l_hi);
          a.lse2[lb + (kvh * a.G + g_hi) * a.R + r_hi] = v2;
          if (a.lse) a.lse[lb + (kvh * a.G + g_hi) * a.R + r_hi] = v2 * kLn2;
        }
      }
    } else {
      const long long slot = (((long long)layer * a.Hkv + kvh) * a.splits + split) * a.rows_pad;
      float* po_lo = a.part_o + (slot + row_lo) * D + 2 * (lane & 3);
      float* po_hi = a.part_o + (slot + row_hi) * D + 2 * (lane & 3);
#pragma unroll
      for (int i = 0; i < D / 8; ++i) {
        *reinterpret_cast<float2*>(po_lo + i * 8) = make_float2(oacc[i][0], oacc[i][1]);
        *reinterpret_cast<float2*>(po_hi + i * 8) = make_float2(oacc[i][2], oacc[i][3]);
      }
      if ((lane & 3) == 0) {
        *reinterpret_cast<float2*>(a.part_ml + (slot + row_lo) * 2) = make_float2(m_lo, l_lo);
        *reinterpret_cast<float2*>(a.part_ml + (slot + row_hi) * 2) = make_float2(m_hi, l_hi);
      }
    }
  }
}

// Merge the key-range partials of one query row: grid (rows, Hkv, n_layers), D threads.
template <int D>
__global__ void __launch_bounds__(D) attn_combine_kernel(const AttnArgs a) {
  const int row = blockIdx.x, kvh = blockIdx.y, layer = blockIdx.z, d = threadIdx.x;
  const long long slot0 = ((long long)layer * a.Hkv + kvh) * a.splits * a.rows_pad + row;
  float mstar = -INFINITY;
  for (int s = 0; s < a.splits; ++s) mstar = fmaxf(mstar, a.part_ml[(slot0 + (long long)s * a.rows_pad) * 2]);
  float l = 0.f, acc = 0.f;
  for (int s = 0; s < a.splits; ++s) {
    const long long sl = slot0 + (long long)s * a.rows_pad;
    const float2 ml = *reinterpret_cast<const float2*>(a.part_ml + sl * 2);
    const float w = fast_exp2(ml.x - mstar);       // exp2(-inf) = 0 for ranges the row cannot see
    l += ml.y * w;
    acc += a.part_o[sl * D + d] * w;
  }
  const int r = row / a.G, g = row % a.G;
  a.o[(long long)layer * a.q_ls + ((long long)r * a.Hq + kvh * a.G + g) * D + d] = __float2bfloat16_rn(acc / l);
  if (d == 0) {
    const long long li = (long long)layer * a.Hq * a.R + (kvh * a.G + g) * a.R + r;
    const float v2 = mstar + log2f(l);
    a.lse2[li] = v2;
    if (a.lse) a.lse[li] = v2 * kLn2;
  }
}

// mass[layer][j] = sum over KV heads (fixed order) of the per-head partial.
__global__ void mass_reduce_kernel(const AttnArgs a) {
  const int layer = blockIdx.y;
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= a.T) return;
  float acc = 0.f;
  for (int h = 0; h < a.Hkv; ++h) acc += a.part_mass[((long long)layer * a.Hkv + h) * a.T_pad + j];
  a.mass[(long long)layer * a.mass_ls + j] = acc;
}

template <int D, int MAXW>
pvlm_status launch_dw(const AttnArgs& a, const pvlm_attn_params& p, const AttnPlan& plan, cudaStream_t s) {
  const dim3 grid(plan.splits, p.Hkv, p.n_layers);
  const int threads = plan.n_warps * 32;
  const int smem0 = kStages * 2 * kAttnBN * D * 2;
  cudaFuncSetAttribute(attn_kernel<D, 0, MAXW>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem0);
  cudaFuncSetAttribute(attn_kernel<D, 0, MAXW>, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
  if (!plan.use_tc) {
    if (p.prof_event_begin) cudaEventRecord((cudaEvent_t)p.prof_event_begin, s);
    attn_kernel<D, 0, MAXW><<<grid, threads, smem0, s>>>(a);
    if (p.prof_event_end) cudaEventRecord((cudaEvent_t)p.prof_event_end, s);
    if (plan.splits > 1) attn_combine_kernel<D><<<dim3(plan.rows, p.Hkv, p.n_layers), D, 0, s>>>(a);
  }
  if (p.mass) {
    const int smem1 = kStages * kAttnBN * D * 2 + 8 * kAttnBN * 4;
    cudaFuncSetAttribute(attn_kernel<D, 1, MAXW>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem1);
    cudaFuncSetAttribute(attn_kernel<D, 1, MAXW>, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
    attn_kernel<D, 1, MAXW><<<dim3(plan.splits, p.Hkv, a.n_mass), threads, smem1, s>>>(a);
    mass_reduce_kernel<<<dim3(ceil_div(plan.T, 256), a.n_mass), 256, 0, s>>>(a);
  }
  return check_launch();
}

template <int D>
pvlm_status launch_d(const AttnArgs& a, const pvlm_attn_params& p, const AttnPlan& plan, cudaStream_t s) {
  return plan.n_warps <= 6 ? launch_dw<D, 6>(a, p, plan, s) : launch_dw<D, 8>(a, p, plan, s);
}

}  // namespace

bool make_attn_plan(const pvlm_attn_params& p, AttnPlan& plan) {
  if (p.Hkv <= 0 || p.Hq <= 0 || p.Hq % p.Hkv != 0 || p.R < 1 || p.n_ctx < 0 || p.n_layers < 1) return false;
  if (p.D != 64 && p.D != 128) return false;
  const int G = p.Hq / p.Hkv;
  if ((long long)G * p.R > 128) return false;
  plan.rows = G * p.R;
  plan.n_warps = ceil_div(plan.rows, 16);
  plan.rows_pad = plan.n_warps * 16;
  plan.T = p.n_ctx + p.R;
  plan.tiles = ceil_div(plan.T, kAttnBN);
  const long long items = (long long)p.Hkv * p.n_layers;
  long long want = ceil_div((long long)kNumSMs * 2 * 8, items);
  const int max_splits = plan.tiles / 8 > 1 ? plan.tiles / 8 : 1;
  int splits = (int)(want < 1 ? 1 : (want > max_splits ? max_splits : want));
  plan.tiles_per_split = ceil_div(plan.tiles, splits);
  plan.splits = ceil_div(plan.tiles, plan.tiles_per_split);
  size_t off = 0;
  plan.off_part_o = off;
  if (plan.splits > 1) off += align_up((size_t)items * plan.splits * plan.rows_pad * p.D * 4, 256);
  plan.off_part_ml = off;
  if (plan.splits > 1) off += align_up((size_t)items * plan.splits * plan.rows_pad * 2 * 4, 256);
  plan.off_lse2 = off;
  off += align_up((size_t)p.n_layers * p.Hq * p.R * 4, 256);
  plan.off_part_mass = off;
  if (p.mass) {
    if (p.mass_layers && (p.n_mass_layers < 1 || p.n_mass_layers > 8)) return false;
    const int n_mass = p.mass_layers ? p.n_mass_layers : p.n_layers;
    // per-KV-head partial sums; two per head where the tensor-core mass pass splits the query rows between its groups
    const int parts = (plan.rows_pad == 96 || plan.rows_pad == 128) ? 2 : 1;
    off += align_up((size_t)n_mass * p.Hkv * parts * align_up(plan.T, kAttnBN) * 4, 256);
  }
  // main pass on the tcgen05 kernel whenever it applies (PVLM_ATTN_IMPL=mma forces the mma.sync kernel)
  const bool force_mma = option_value(PVLM_OPT_ATTN_MMA_SYNC) != 0;
  plan.use_tc = (p.D == 128 || p.D == 64) && !force_mma && make_attn_tc_plan(p, plan.tc);
  plan.off_tc = off;
  if (plan.use_tc) off += align_up(plan.tc.total, 256);
  plan.total = off;
  return true;
}

pvlm_status launch_verify_attn(const pvlm_attn_params& p, const AttnPlan& plan, cudaStream_t s) {
  AttnArgs a;
  a.q = (const __nv_bfloat16*)p.q;
  a.k = (const __nv_bfloat16*)p.k;
  a.v = (const __nv_bfloat16*)p.v;
  a.o = (__nv_bfloat16*)p.o;
  a.lse = p.lse;
  a.mass = p.mass;
  char* ws = (char*)p.workspace;
  a.part_o = (float*)(ws + plan.off_part_o);
  a.part_ml = (float*)(ws + plan.off_part_ml);
  a.lse2 = (float*)(ws + plan.off_lse2);
  a.part_mass = (float*)(ws + plan.off_part_mass);
  a.R = p.R; a.Hq = p.Hq; a.Hkv = p.Hkv; a.G = p.Hq / p.Hkv; a.n_ctx = p.n_ctx;
  a.T = plan.T; a.T_pad = (int)align_up(plan.T, kAttnBN);
  a.rows = plan.rows; a.rows_pad = plan.rows_pad;
  a.splits = plan.splits; a.tiles_per_split = plan.tiles_per_split; a.tiles = plan.tiles;
  a.q_ls = p.q_layer_stride; a.kv_ls = p.kv_layer_stride; a.kv_ts = p.kv_token_stride; a.kv_hs = p.kv_head_stride;
  a.mass_ls = p.mass_layer_stride;
  const float scale = (p.softmax_scale == 0.f) ? 1.0f / sqrtf((float)p.D) : p.softmax_scale;
  a.scale_log2 = scale * kLog2e;
  a.mass_listed = p.mass_layers != nullptr;
  a.n_mass = a.mass_listed ? p.n_mass_layers : p.n_layers;
  for (int i = 0; i < 8; ++i) a.mass_layer[i] = (a.mass_listed && i < p.n_mass_layers) ? p.mass_layers[i] : 0;
  if (plan.use_tc) {
    const pvlm_status st = launch_verify_attn_tc(p, plan.tc, ws + plan.off_tc, a.lse2, s);
    if (st != PVLM_OK) return st;
    if (!p.mass) return PVLM_OK;
    return launch_attn_mass_tc(p, a.lse2, a.part_mass, (int*)(ws + plan.off_tc + plan.tc.off_status), s);
  }
  return p.D == 64 ? launch_d<64>(a, p, plan, s) : launch_d<128>(a, p, plan, s);
}

}  // namespace pvlm
