// Window-verify GQA attention on the 5th-generation tensor cores (tcgen05 + TMEM + TMA), D = 128.
//
// Work decomposition ("stream-K"): the (layer, KV head) items are cut into 128-key tiles, the
// flattened tile sequence is divided evenly among one persistent CTA per SM, and a CTA walks its
// contiguous range segment by segment (a segment = its tiles of one item).  Every segment ends in a
// partial (O, m, l) written to the workspace; a small combine kernel merges an item's segments.
//
// Inside a CTA (10 warps):
//   warp 0      TMA producer: K and V tiles (two 64-channel boxes each, 128-byte swizzle) into
//               separate 2-deep shared-memory rings, completion on mbarriers.
//   warp 1      MMA issuer (one thread): S^T = K . Q^T  (M = 128 keys, N = padded query rows,
//               K = 128 channels) into one of two TMEM score buffers, then O^T += V^T . P^T
//               (M = 128 channels, N = rows, K = 128 keys) into the TMEM output accumulator.
//   warps 2..9  softmax: each thread owns one key (TMEM lane) and half of the query-row columns,
//               so exp2, the running row sums and the bf16 pack are thread-local; P is written to
//               shared memory in the MN-major core-matrix layout the second MMA reads.
// The transposed orientation keeps all 128 TMEM lanes busy although only G*R <= 128 (typically
// 65..88) query rows exist, and makes N (not M) the padded dimension: N = 80 instead of M = 128.
//
// Softmax reference m per row is updated lazily: a tile whose scores stay below m + 8 (log2 units)
// reuses m; otherwise (and on the first tile of a segment) all softmax threads take a slow path that
// reduces the tile's row maxima, rescales the running sums and the TMEM accumulator, and goes on.
// Every mbarrier wait is bounded: on expiry the CTA sets a status word and leaves cleanly.
#include "pvlm_common.cuh"

#include <cuda.h>

namespace pvlm {

namespace {

constexpr int kTile = 128;                 // keys per tile
constexpr int kKStages = 2, kVStages = 2;
// P buffers: two, except for the widest row counts where shared memory only has room for one
__host__ __device__ constexpr int p_bufs(int nrp) { return nrp > 96 ? 1 : 2; }
constexpr int kBoxBytes = kTile * 128;     // one 64-channel box of a 128-key tile: 16 KB
constexpr int kTileBytes = 2 * kBoxBytes;  // 32 KB
constexpr int kSoftmaxThreads = 256;
constexpr int kThreads = 64 + kSoftmaxThreads;
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr float kRescaleThreshold = 8.0f;  // log2 units
constexpr float kNegBig = -1.0e30f;        // "no key seen yet" reference: finite, so differences never give NaN

struct TcArgs {
  const __nv_bfloat16* q;
  float *part_o, *part_ml;
  int* status;
  int R, Hq, Hkv, G, n_ctx, T, rows, n_layers;
  long long q_ls;
  float scale_log2;
  int tiles_per_item;        // Tt
  long long total_tiles;     // W = items * Tt
  int seg_max;               // partial slots per CTA
  int n_cta;
};

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait: false if the phase did not complete within the spin limit or another thread gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
    if (*abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&r)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr));
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t (&r)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// Makes the compiler treat the registers as written here, i.e. after the preceding wait::ld.
__device__ __forceinline__ void reg_fence8(uint32_t (&r)[8]) {
  asm volatile("" : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]));
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}
__device__ __forceinline__ void softmax_bar_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ bool softmax_bar_or(bool pred) {
  uint32_t out;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 p, %1, 0;\n\t"
      "bar.red.or.pred q, 1, 256, p;\n\t"
      "selp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(out)
      : "r"((uint32_t)pred)
      : "memory");
  return out != 0;
}
// monotone float <-> int map for shared-memory atomicMax on floats
__device__ __forceinline__ int f2ord(float f) {
  const int i = __float_as_int(f);
  return i >= 0 ? i : i ^ 0x7fffffff;
}
__device__ __forceinline__ float ord2f(int i) { return __int_as_float(i >= 0 ? i : i ^ 0x7fffffff); }

// shared-memory matrix descriptor (version 1); offsets in bytes
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo, uint32_t layout) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) |
         (1ull << 46) | ((uint64_t)layout << 61);
}

// ---------------------------------------------------------------------------------------------
// The kernel.  NRP = query rows per KV head padded to a multiple of 16 (MMA N).
// ---------------------------------------------------------------------------------------------
template <int NRP>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, const TcArgs a) {
  constexpr int HALF = NRP / 2;            // columns per softmax thread
  constexpr int NCH = HALF / 8;            // 8-column chunks per thread
  constexpr int QBOX = NRP * 128;          // bytes of one 64-channel box of Q
  constexpr int PBYTES = NRP * 256;        // one P buffer: NRP/8 row groups x 2048 B
  constexpr int kPBufs = p_bufs(NRP);
  constexpr uint32_t TMEM_COLS = (3 * NRP <= 32) ? 32 : (3 * NRP <= 64) ? 64 : (3 * NRP <= 128) ? 128 : (3 * NRP <= 256) ? 256 : 512;
  constexpr uint32_t IDESC_QK = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NRP >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
  constexpr uint32_t IDESC_PV = IDESC_QK | (1u << 15) | (1u << 16);

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* sK = smem;
  unsigned char* sV = sK + kKStages * kTileBytes;
  unsigned char* sQ = sV + kVStages * kTileBytes;
  unsigned char* sP = sQ + 2 * QBOX;
  int* s_newmax = reinterpret_cast<int*>(sP + kPBufs * PBYTES);      // [128]
  float* s_lsum = reinterpret_cast<float*>(s_newmax + 128);          // [4][128]
  uint64_t* bars = reinterpret_cast<uint64_t*>(s_lsum + 4 * 128);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 24);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);

  enum { K_FULL = 0, K_EMPTY = 2, V_FULL = 4, V_EMPTY = 6, S_FULL = 8, S_FREE = 10, P_FULL = 12, P_FREE = 14,
         Q_READY = 16, O_FULL = 17, O_FREE = 18 };
  auto bar = [&](int i) { return smem_addr(bars + i); };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // ---- this CTA's range of the flattened tile sequence ----
  const long long W = a.total_tiles;
  const long long f_begin = (W * blockIdx.x) / a.n_cta, f_end = (W * (blockIdx.x + 1)) / a.n_cta;
  const int Tt = a.tiles_per_item;
  const int item_first = (int)(f_begin / Tt);

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar(K_FULL + i), 1); mbar_init(bar(K_EMPTY + i), 1);
      mbar_init(bar(V_FULL + i), 1); mbar_init(bar(V_EMPTY + i), 1);
      mbar_init(bar(S_FULL + i), 1); mbar_init(bar(S_FREE + i), kSoftmaxThreads);
      mbar_init(bar(P_FULL + i), kSoftmaxThreads); mbar_init(bar(P_FREE + i), 1);
    }
    mbar_init(bar(Q_READY), kSoftmaxThreads);
    mbar_init(bar(O_FULL), 1);
    mbar_init(bar(O_FREE), kSoftmaxThreads);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(s_tmem)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // zero Q (its padding rows are never written again) and the slow-path scratch
  for (int i = tid; i < 2 * QBOX / 16; i += kThreads) reinterpret_cast<uint4*>(sQ)[i] = make_uint4(0, 0, 0, 0);
  if (tid < 128) s_newmax[tid] = f2ord(-INFINITY);
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;
  const uint32_t tmem_S0 = tmem, tmem_O = tmem + 2 * NRP;

  if (f_end > f_begin) {
    if (warp == 0) {
      // =========================== TMA producer ===========================
      if (lane == 0) {
        uint32_t jt = 0;
        for (long long f = f_begin; f < f_end; ++f, ++jt) {
          const int item = (int)(f / Tt), tile = (int)(f - (long long)item * Tt);
          const int layer = item / a.Hkv, kvh = item - layer * a.Hkv;
          const uint32_t ks = jt % kKStages, vs = jt % kVStages;
          if (jt >= kKStages && !mbar_wait(bar(K_EMPTY + ks), ((jt / kKStages) - 1) & 1, s_abort)) break;
          mbar_expect_tx(bar(K_FULL + ks), kTileBytes);
          tma_load_4d(smem_addr(sK + ks * kTileBytes), &tm_k, bar(K_FULL + ks), 0, kvh, tile * kTile, layer);
          tma_load_4d(smem_addr(sK + ks * kTileBytes + kBoxBytes), &tm_k, bar(K_FULL + ks), 64, kvh, tile * kTile, layer);
          if (jt >= kVStages && !mbar_wait(bar(V_EMPTY + vs), ((jt / kVStages) - 1) & 1, s_abort)) break;
          mbar_expect_tx(bar(V_FULL + vs), kTileBytes);
          tma_load_4d(smem_addr(sV + vs * kTileBytes), &tm_v, bar(V_FULL + vs), 0, kvh, tile * kTile, layer);
          tma_load_4d(smem_addr(sV + vs * kTileBytes + kBoxBytes), &tm_v, bar(V_FULL + vs), 64, kvh, tile * kTile, layer);
        }
      }
    } else if (warp == 1) {
      // =========================== MMA issuer ===========================
      if (lane == 0) {
        const uint32_t q_base = smem_addr(sQ);
        bool ok = true;
        uint32_t jt = 0;           // tiles issued by this CTA so far (ring phases run across segments)
        int seg = 0;
        auto issue_qk = [&](uint32_t j) -> bool {
          const uint32_t ks = j % kKStages, sb = j & 1;
          if (!mbar_wait(bar(K_FULL + ks), (j / kKStages) & 1, s_abort)) return false;
          if (j >= 2 && !mbar_wait(bar(S_FREE + sb), ((j >> 1) - 1) & 1, s_abort)) return false;
          tc_fence_after();
          const uint32_t k_base = smem_addr(sK + ks * kTileBytes);
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t off = (kk >> 2) * kBoxBytes + (kk & 3) * 32, qoff = (kk >> 2) * QBOX + (kk & 3) * 32;
            tc_mma(tmem_S0 + sb * NRP, make_desc(k_base + off, 16, 1024, 2), make_desc(q_base + qoff, 16, 1024, 2), IDESC_QK, kk > 0);
          }
          tc_commit(bar(S_FULL + sb));
          tc_commit(bar(K_EMPTY + ks));
          return true;
        };
        for (long long f = f_begin; f < f_end && ok; ++seg) {
          const int item = (int)(f / Tt);
          const long long seg_end = min(f_end, (long long)(item + 1) * Tt);
          const int n = (int)(seg_end - f);
          if (!mbar_wait(bar(Q_READY), seg & 1, s_abort)) { ok = false; break; }
          tc_fence_after();
          if (!issue_qk(jt)) { ok = false; break; }
          for (int i = 0; i < n; ++i) {
            const uint32_t j = jt + i;
            if (i + 1 < n && !issue_qk(j + 1)) { ok = false; break; }
            const uint32_t vs = j % kVStages, pb = j % kPBufs;
            if (i == 0 && seg > 0 && !mbar_wait(bar(O_FREE), (seg - 1) & 1, s_abort)) { ok = false; break; }
            if (!mbar_wait(bar(V_FULL + vs), (j / kVStages) & 1, s_abort)) { ok = false; break; }
            if (!mbar_wait(bar(P_FULL + pb), (j / kPBufs) & 1, s_abort)) { ok = false; break; }
            tc_fence_after();
            const uint32_t v_base = smem_addr(sV + vs * kTileBytes), p_base = smem_addr(sP + pb * PBYTES);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
              tc_mma(tmem_O, make_desc(v_base + kk * 2048, kBoxBytes, 1024, 2), make_desc(p_base + kk * 256, 128, 2048, 0),
                     IDESC_PV, (i > 0 || kk > 0));
            tc_commit(bar(V_EMPTY + vs));
            tc_commit(bar(P_FREE + pb));
          }
          if (!ok) break;
          tc_commit(bar(O_FULL));
          jt += n;
          f = seg_end;
        }
      }
    } else {
      // =========================== softmax warps ===========================
      const int q4 = warp & 3;                 // TMEM lane quarter this warp may access
      const int wg = (warp - 2) >> 2;          // column half
      const int t = q4 * 32 + lane;            // key within the tile == TMEM lane; channel d in the epilogue
      const int st = tid - 64;                 // 0..255
      const int col0 = wg * HALF;
      const uint32_t lane_addr = (uint32_t)(q4 * 32) << 16;
      float m_loc[HALF], l_loc[HALF];
      uint32_t jt = 0;
      int seg = 0;
      bool ok = true;
      for (long long f = f_begin; f < f_end; ++seg) {
        const int item = (int)(f / Tt), tile0 = (int)(f - (long long)item * Tt);
        const long long seg_end = min(f_end, (long long)(item + 1) * Tt);
        const int n = (int)(seg_end - f);
        const int layer = item / a.Hkv, kvh = item - layer * a.Hkv;
        // ---- stage Q of this (layer, KV head) in the K-major 128B-swizzled layout ----
        {
          const __nv_bfloat16* qb = a.q + (long long)layer * a.q_ls + (long long)kvh * a.G * 128;
          for (int idx = st; idx < a.rows * 16; idx += kSoftmaxThreads) {
            const int row = idx >> 4, c = idx & 15;
            const int r = row / a.G, g = row - r * a.G;
            const uint4 val = *reinterpret_cast<const uint4*>(qb + ((long long)r * a.Hq + g) * 128 + c * 8);
            *reinterpret_cast<uint4*>(sQ + (c >> 3) * QBOX + row * 128 + (((c & 7) ^ (row & 7)) << 4)) = val;
          }
          fence_proxy_async();
          mbar_arrive(bar(Q_READY));
        }
#pragma unroll
        for (int i = 0; i < HALF; ++i) { m_loc[i] = kNegBig; l_loc[i] = 0.f; }

        bool aborted = false;
        for (int i = 0; i < n; ++i) {
          const uint32_t j = jt + i, sb = j & 1, pb = j % kPBufs;
          const int tile = tile0 + i;
          const int key = tile * kTile + t;
          const bool need_mask = (tile * kTile + kTile - 1 > a.n_ctx);
          // A failed wait never leaves this loop on its own (the other softmax threads would be left
          // at a named barrier): it clears `ok`, and the vote below takes all 256 threads out together.
          ok &= mbar_wait(bar(S_FULL + sb), (j >> 1) & 1, s_abort);
          tc_fence_after();
          float x[HALF];
          auto load_scores = [&](bool subtract_m) {
            uint32_t raw[NCH][8];
#pragma unroll
            for (int c = 0; c < NCH; ++c) tmem_ld8(tmem_S0 + lane_addr + sb * NRP + col0 + c * 8, raw[c]);
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
              reg_fence8(raw[c]);
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const int idx = c * 8 + e;
                float v = __uint_as_float(raw[c][e]) * a.scale_log2;
                if (need_mask && key > a.n_ctx + (col0 + idx) / a.G) v = -INFINITY;
                x[idx] = subtract_m ? v - m_loc[idx] : v;
              }
            }
          };
          load_scores(true);
          bool exceed = false;
#pragma unroll
          for (int k = 0; k < HALF; ++k) exceed |= (x[k] > kRescaleThreshold);
          if (softmax_bar_or(exceed || !ok)) {
            if (softmax_bar_or(!ok)) { aborted = true; break; }        // uniform across the 256 threads
            // ------- slow path: new per-row reference, rescale sums and accumulator -------
            load_scores(false);
#pragma unroll
            for (int k = 0; k < HALF; ++k) {
              float v = x[k];
#pragma unroll
              for (int sh = 16; sh >= 1; sh >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, sh));
              if (lane == 0) atomicMax(&s_newmax[col0 + k], f2ord(v));
            }
            softmax_bar_sync();
            float fac[HALF];
#pragma unroll
            for (int k = 0; k < HALF; ++k) {
              const float mn = fmaxf(m_loc[k], ord2f(s_newmax[col0 + k]));
              fac[k] = ex2(m_loc[k] - mn);             // 0 when the row had seen nothing, 1 when nothing changed
              l_loc[k] *= fac[k];
              m_loc[k] = mn;
            }
            if (i > 0) {
              // the accumulator holds tiles < i: wait until the last of them has been added
              ok &= mbar_wait(bar(P_FREE + ((j - 1) % kPBufs)), ((j - 1) / kPBufs) & 1, s_abort);
              tc_fence_after();
#pragma unroll
              for (int c = 0; c < NCH; ++c) {
                uint32_t o[8];
                tmem_ld8(tmem_O + lane_addr + col0 + c * 8, o);
                tmem_wait_ld();
                reg_fence8(o);
#pragma unroll
                for (int e = 0; e < 8; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * fac[c * 8 + e]);
                tmem_st8(tmem_O + lane_addr + col0 + c * 8, o);
              }
              tmem_wait_st();
            }
            softmax_bar_sync();                      // everyone has read s_newmax
            if (st < NRP) s_newmax[st] = f2ord(-INFINITY);
#pragma unroll
            for (int k = 0; k < HALF; ++k) x[k] = x[k] - m_loc[k];
          }
          tc_fence_before();
          mbar_arrive(bar(S_FREE + sb));
          // ---- probabilities, running sums, bf16 P in the MN-major core-matrix layout ----
          if (j >= kPBufs) ok &= mbar_wait(bar(P_FREE + pb), ((j / kPBufs) - 1) & 1, s_abort);
          unsigned char* pdst = sP + pb * PBYTES + (col0 >> 3) * 2048 + t * 16;
#pragma unroll
          for (int c = 0; c < NCH; ++c) {
            float p[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              p[e] = ex2(x[c * 8 + e]);
              l_loc[c * 8 + e] += p[e];
            }
            *reinterpret_cast<uint4*>(pdst + c * 2048) =
                make_uint4(pack2(p[0], p[1]), pack2(p[2], p[3]), pack2(p[4], p[5]), pack2(p[6], p[7]));
          }
          fence_proxy_async();
          mbar_arrive(bar(P_FULL + pb));
        }
        if (aborted) break;
        // ---- segment epilogue: partial O (fp32), and (m, l) per row ----
        ok &= mbar_wait(bar(O_FULL), seg & 1, s_abort);
        tc_fence_after();
        const long long slot = (long long)blockIdx.x * a.seg_max + (item - item_first);
        float* po = a.part_o + slot * NRP * 128;
#pragma unroll
        for (int c = 0; c < NCH; ++c) {
          uint32_t o[8];
          tmem_ld8(tmem_O + lane_addr + col0 + c * 8, o);
          tmem_wait_ld();
          reg_fence8(o);
#pragma unroll
          for (int e = 0; e < 8; ++e) po[(long long)(col0 + c * 8 + e) * 128 + t] = __uint_as_float(o[e]);
        }
        tc_fence_before();
        mbar_arrive(bar(O_FREE));
#pragma unroll
        for (int k = 0; k < HALF; ++k) {
          float v = l_loc[k];
#pragma unroll
          for (int sh = 16; sh >= 1; sh >>= 1) v += __shfl_xor_sync(0xffffffffu, v, sh);
          if (lane == 0) s_lsum[q4 * 128 + col0 + k] = v;
        }
        // m is identical in all threads of a column half; thread with t == 0 publishes it
        if (t == 0) {
#pragma unroll
          for (int k = 0; k < HALF; ++k) a.part_ml[(slot * NRP + col0 + k) * 2] = m_loc[k];
        }
        softmax_bar_sync();
        if (st < NRP) {
          const float l = ((s_lsum[st] + s_lsum[128 + st]) + s_lsum[256 + st]) + s_lsum[384 + st];
          a.part_ml[(slot * NRP + st) * 2 + 1] = l;
        }
        softmax_bar_sync();
        jt += n;
        f = seg_end;
      }
    }
  }

  // ---- teardown (every loop above is bounded, so every thread gets here) ----
  tc_fence_before();
  __syncthreads();
  if (*s_abort) {
    if (tid == 0) atomicExch(a.status, 1);
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);     // let copies / MMAs in flight land before TMEM is released
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
  }
}

// Merge the segments of one (item, row): grid (rows, items), 128 threads (channel d).
struct CombineArgs {
  const float *part_o, *part_ml;
  __nv_bfloat16* o;
  float *lse, *lse2;
  int R, Hq, Hkv, G, rows, nrp, tiles_per_item, seg_max, n_cta;
  long long total_tiles, q_ls;
};

__global__ void __launch_bounds__(128) attn_tc_combine_kernel(const CombineArgs a) {
  const int row = blockIdx.x, item = blockIdx.y, d = threadIdx.x;
  const long long W = a.total_tiles, C = a.n_cta;
  const long long lo = (long long)item * a.tiles_per_item, hi = lo + a.tiles_per_item;
  auto b = [&](long long c) { return (W * c) / C; };
  long long c0 = (lo * C) / W;
  while (c0 + 1 < C && b(c0 + 1) <= lo) ++c0;
  while (c0 > 0 && b(c0) > lo) --c0;
  float mstar = -INFINITY;
  for (long long c = c0; c < C && b(c) < hi; ++c) {
    if (b(c + 1) <= lo || b(c + 1) == b(c)) continue;
    const long long slot = c * a.seg_max + (item - (int)(b(c) / a.tiles_per_item));
    mstar = fmaxf(mstar, a.part_ml[(slot * a.nrp + row) * 2]);
  }
  float l = 0.f, acc = 0.f;
  for (long long c = c0; c < C && b(c) < hi; ++c) {
    if (b(c + 1) <= lo || b(c + 1) == b(c)) continue;
    const long long slot = c * a.seg_max + (item - (int)(b(c) / a.tiles_per_item));
    const float m = a.part_ml[(slot * a.nrp + row) * 2], ls = a.part_ml[(slot * a.nrp + row) * 2 + 1];
    const float w = ex2(m - mstar);                     // 0 for a segment in which the row saw no key
    l += ls * w;
    acc += a.part_o[(slot * a.nrp + row) * 128 + d] * w;
  }
  const int layer = item / a.Hkv, kvh = item - layer * a.Hkv;
  const int r = row / a.G, g = row - r * a.G;
  a.o[(long long)layer * a.q_ls + ((long long)r * a.Hq + kvh * a.G + g) * 128 + d] = __float2bfloat16_rn(acc / l);
  if (d == 0) {
    const long long li = (long long)layer * a.Hq * a.R + (kvh * a.G + g) * a.R + r;
    const float v2 = mstar + log2f(l);
    a.lse2[li] = v2;
    if (a.lse) a.lse[li] = v2 * kLn2;
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
        qr == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

bool make_kv_map(CUtensorMap* map, const void* base, const pvlm_attn_params& p, int T) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {128, (cuuint64_t)p.Hkv, (cuuint64_t)T, (cuuint64_t)p.n_layers};
  const cuuint64_t layer_stride = p.n_layers > 1 ? (cuuint64_t)p.kv_layer_stride : (cuuint64_t)T * p.kv_token_stride;
  const cuuint64_t strides[3] = {(cuuint64_t)p.kv_head_stride * 2, (cuuint64_t)p.kv_token_stride * 2, layer_stride * 2};
  const cuuint32_t box[4] = {64, 1, (cuuint32_t)kTile, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int NRP>
constexpr int tc_smem_bytes() {
  return 1024 /*alignment slack*/ + (kKStages + kVStages) * kTileBytes + 2 * NRP * 128 + p_bufs(NRP) * NRP * 256 + 128 * 4 +
         4 * 128 * 4 + 24 * 8 + 64;
}

template <int NRP>
void launch_tc(const CUtensorMap& mk, const CUtensorMap& mv, const TcArgs& a, cudaStream_t s) {
  constexpr int smem = tc_smem_bytes<NRP>();
  cudaFuncSetAttribute(attn_tc_kernel<NRP>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  attn_tc_kernel<NRP><<<a.n_cta, kThreads, smem, s>>>(mk, mv, a);
}

}  // namespace

bool make_attn_tc_plan(const pvlm_attn_params& p, AttnTcPlan& plan) {
  if (p.D != 128 || p.Hkv <= 0 || p.Hq % p.Hkv != 0) return false;
  const int G = p.Hq / p.Hkv;
  const int rows = G * p.R;
  if (rows > 128) return false;
  plan.nrp = (rows + 15) / 16 * 16;
  plan.T = p.n_ctx + p.R;
  plan.tiles_per_item = ceil_div(plan.T, kTile);
  plan.total_tiles = (long long)plan.tiles_per_item * p.Hkv * p.n_layers;
  plan.n_cta = (int)(plan.total_tiles < kNumSMs ? plan.total_tiles : kNumSMs);
  const long long per_cta = (plan.total_tiles + plan.n_cta - 1) / plan.n_cta;
  plan.seg_max = (int)((per_cta + plan.tiles_per_item - 1) / plan.tiles_per_item) + 1;
  size_t off = 0;
  plan.off_part_o = off;  off += align_up((size_t)plan.n_cta * plan.seg_max * plan.nrp * 128 * 4, 256);
  plan.off_part_ml = off; off += align_up((size_t)plan.n_cta * plan.seg_max * plan.nrp * 2 * 4, 256);
  plan.off_status = off;  off += 256;
  plan.total = off;
  return true;
}

pvlm_status launch_verify_attn_tc(const pvlm_attn_params& p, const AttnTcPlan& plan, char* ws, float* lse2, cudaStream_t s) {
  CUtensorMap mk, mv;
  if (!make_kv_map(&mk, p.k, p, plan.T) || !make_kv_map(&mv, p.v, p, plan.T)) return PVLM_ERR_UNSUPPORTED;
  TcArgs a;
  a.q = (const __nv_bfloat16*)p.q;
  a.part_o = (float*)(ws + plan.off_part_o);
  a.part_ml = (float*)(ws + plan.off_part_ml);
  a.status = (int*)(ws + plan.off_status);
  a.R = p.R; a.Hq = p.Hq; a.Hkv = p.Hkv; a.G = p.Hq / p.Hkv; a.n_ctx = p.n_ctx; a.T = plan.T;
  a.rows = a.G * p.R; a.n_layers = p.n_layers;
  a.q_ls = p.q_layer_stride;
  const float scale = (p.softmax_scale == 0.f) ? 1.0f / sqrtf((float)p.D) : p.softmax_scale;
  a.scale_log2 = scale * kLog2e;
  a.tiles_per_item = plan.tiles_per_item; a.total_tiles = plan.total_tiles; a.seg_max = plan.seg_max; a.n_cta = plan.n_cta;
  cudaMemsetAsync(a.status, 0, 4, s);
  switch (plan.nrp) {
    case 16: launch_tc<16>(mk, mv, a, s); break;
    case 32: launch_tc<32>(mk, mv, a, s); break;
    case 48: launch_tc<48>(mk, mv, a, s); break;
    case 64: launch_tc<64>(mk, mv, a, s); break;
    case 80: launch_tc<80>(mk, mv, a, s); break;
    case 96: launch_tc<96>(mk, mv, a, s); break;
    case 112: launch_tc<112>(mk, mv, a, s); break;
    case 128: launch_tc<128>(mk, mv, a, s); break;
    default: return PVLM_ERR_UNSUPPORTED;
  }
  CombineArgs c;
  c.part_o = a.part_o; c.part_ml = a.part_ml; c.o = (__nv_bfloat16*)p.o; c.lse = p.lse; c.lse2 = lse2;
  c.R = p.R; c.Hq = p.Hq; c.Hkv = p.Hkv; c.G = a.G; c.rows = a.rows; c.nrp = plan.nrp;
  c.tiles_per_item = plan.tiles_per_item; c.seg_max = plan.seg_max; c.n_cta = plan.n_cta;
  c.total_tiles = plan.total_tiles; c.q_ls = p.q_layer_stride;
  attn_tc_combine_kernel<<<dim3(a.rows, p.Hkv * p.n_layers), 128, 0, s>>>(c);
  return check_launch();
}

}  // namespace pvlm
