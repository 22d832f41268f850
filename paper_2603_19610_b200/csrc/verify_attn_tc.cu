// Window-verify GQA attention on the 5th-generation tensor cores (tcgen05 + TMEM + TMA), D = 128 or 64.
// (D = 64 runs the same kernels on channels padded to 128: the tensor map knows 64 channels, so the TMA
// box of channels 64..127 is out of range and arrives as zeros without touching memory; Q's upper half stays
// zero in shared memory; only the global reads of Q and the writes of O know the real row length.)
//
// Work decomposition ("stream-K"): the (layer, KV head) items are cut into 128-key tiles, the
// flattened tile sequence is divided evenly among one persistent CTA per SM, and a CTA walks its
// contiguous range segment by segment (a segment = its tiles of one item).  Every segment ends in a
// partial (O, m, l) written to the workspace; a small combine kernel merges an item's segments.
//
// Inside a CTA (12 warps = 3 warpgroups; registers are moved from warpgroup 0 to the softmax
// warpgroups with setmaxnreg):
//   warp 0       TMA producer (one lane): K and V tiles (two 64-channel boxes each, 128-byte swizzle)
//                into ONE shared ring of 3 to 5 slots of 32 KB, in the order the issuer consumes them
//                (K(0..lookahead), V(0), K(lookahead+1), V(1), ...); completion on mbarriers.
//   warp 1       MMA issuer: the whole warp walks the tile loop converged (counters, barrier
//                addresses and descriptors are warp-uniform) and one elected lane issues
//                S^T = K . Q^T  (M = 128 keys, N = padded query rows, K = 128 channels) into one of up
//                to four TMEM score buffers, then O^T += V^T . P^T  (M = 128 channels, N = rows,
//                K = 128 keys) into a TMEM output accumulator, and commits the barriers that free
//                the ring slots.  (Two separate issuer threads were tried: they let the two softmax
//                groups fall into step, which loses the overlap between them.)
//   warps 4..11  two softmax groups working on alternate tiles, each with its own accumulator,
//                reference and row sums (two interleaved online-softmax streams).  A thread owns
//                one key (TMEM lane) of its group's tile and all query-row columns, so exp2, the
//                running row sums and the bf16 pack are thread-local; P is written to shared
//                memory in the MN-major core-matrix layout the second MMA reads.
// The transposed orientation keeps all 128 TMEM lanes busy although only G*R <= 128 (typically
// 65..88) query rows exist, and makes N (not M) the padded dimension: N = 80 instead of M = 128.
//
// Softmax reference m per row is updated lazily: a tile whose scores stay below m + 8 (log2 units)
// reuses m; otherwise (and on the first tile of a segment) all softmax threads take a slow path that
// reduces the tile's row maxima, rescales the running sums and the TMEM accumulator, and goes on.
// Every mbarrier wait is bounded: on expiry the CTA sets a status word and leaves cleanly.
#include <atomic>

#include "pvlm_common.cuh"

#include <cuda.h>


namespace pvlm {

namespace {

constexpr int kTile = 128;                 // keys per tile
constexpr int kBoxBytes = kTile * 128;     // one 64-channel box of a 128-key tile: 16 KB
constexpr int kTileBytes = 2 * kBoxBytes;  // 32 KB
constexpr int kSoftmaxThreads = 256;
constexpr int kGroupThreads = 128;         // one softmax group
constexpr int kThreads = 128 + kSoftmaxThreads;   // warpgroup 0: TMA + MMA (+2 idle warps); warpgroups 1, 2: softmax
#ifndef PVLM_SUSPEND_NS
#define PVLM_SUSPEND_NS 20000
#endif
constexpr uint32_t kSuspendHintNs = PVLM_SUSPEND_NS;        // upper bound of one sleep inside try_wait
constexpr uint64_t kWaitLimitNs = 1000000000ull;   // a wait that lasts a second has failed
constexpr float kRescaleThreshold = 8.0f;  // log2 units
constexpr float kNegBig = -1.0e30f;        // "no key seen yet" reference: finite, so differences never give NaN

struct TcArgs {
  const __nv_bfloat16* q;
  float *part_o, *part_ml;
  int* status;
  int R, Hq, Hkv, G, n_ctx, T, rows, n_layers;
  int D;                     // real head dimension (64 or 128)
  long long q_ls;
  float scale_log2;
  int tiles_per_item;        // Tt
  long long total_tiles;     // W = items * Tt
  int seg_max;               // partial slots per CTA
  int n_cta;
  uint32_t g_magic;          // ceil(2^16 / G): row / G == (row * g_magic) >> 16 for row < 128
  int lookahead;             // score tiles the issuer keeps in flight past the tile whose PV it issues next
  int l2_hints;              // 1: a mass pass over the same layers follows: K is asked to stay in L2, V to leave first
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
// Bounded wait: false if the phase did not complete within the time limit or another thread gave up.
// A first non-blocking test_wait serves the common case of a phase that completed long ago.  After
// that the thread sleeps inside try_wait (suspend-time hint) instead of polling: 300 spinning threads
// per SM cost enough power to pull the SM clock down under the board's power cap.
__device__ __forceinline__ uint64_t global_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  if (ok) return true;
  const uint64_t t0 = global_ns();
  for (;;) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(kSuspendHintNs)
        : "memory");
    if (ok) return true;
    if (*abort_flag) return false;
    if (global_ns() - t0 > kWaitLimitNs) break;
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
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld8_lo(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr));
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
// Makes the compiler treat the registers as written here, i.e. after the preceding wait::ld.
__device__ __forceinline__ void reg_fence16(uint32_t (&r)[16]) {
  asm volatile("" : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                    "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]));
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
// The same load with an L2 eviction-priority hint (a policy word made by l2_policy_*).
__device__ __forceinline__ void tma_load_4d_hint(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3,
                                                 uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy)
      : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
// One lane of a converged warp (the same lane every time).
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xffffffff;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(pred));
  return pred != 0;
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
__device__ __forceinline__ bool softmax_bar_or(bool pred) {
  uint32_t out;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 p, %1, 0;\n\t"
      "bar.red.or.pred q, 3, 256, p;\n\t"
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
// The kernel.  NRP = query rows per KV head padded to a multiple of 16 (MMA N), NRP <= 96.
// ---------------------------------------------------------------------------------------------
// K and V tiles share one ring of 32 KB slots, filled and drained in the order the issuer consumes them.
// Five slots fit beside Q and the two P buffers up to 80 padded rows.
__host__ __device__ constexpr int ring_slots(int nrp) { return nrp <= 80 ? 5 : nrp <= 112 ? 4 : 3; }
// Wide row groups (96 or 128 padded rows) run in SPLIT-COLUMN mode: both softmax groups work on EVERY tile, each on
// half of the query-row columns, instead of on alternate tiles.  A thread then holds half as many scores and running
// row sums (2 x 48 or 2 x 64 registers instead of 2 x 96 / 2 x 128, which spilled), there is one output accumulator
// and one partial per segment instead of two, and the freed TMEM columns hold one more score buffer.
__host__ __device__ constexpr bool split_cols(int nrp) { return nrp == 96 || nrp == 128; }
__host__ __device__ constexpr int s_bufs(int nrp) {
  return split_cols(nrp) ? ((512 - nrp) / nrp >= 4 ? 4 : (512 - nrp) / nrp)
                         : ((512 - 2 * nrp) / nrp >= 4 ? 4 : (512 - 2 * nrp) / nrp);
}

// HT: the last 16-column chunk holds at most 8 real query rows, so only its first 8 columns are processed.
template <int NRP, bool HT>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, const TcArgs a) {
  constexpr bool SC = split_cols(NRP);     // both groups on every tile, half of the columns each
  constexpr int NCH = SC ? NRP / 32 : NRP / 16;            // 16-column chunks per thread
  static_assert(!(SC && HT), "split-column mode processes whole chunks");
  auto CW = [](int c) constexpr { return (HT && c == NRP / 16 - 1) ? 8 : 16; };   // processed columns of chunk c
  constexpr int QBOX = NRP * 128;          // bytes of one 64-channel box of Q
  constexpr int PBYTES = NRP * 256;        // one P buffer: NRP/8 row groups x 2048 B
  constexpr int NSB = s_bufs(NRP);         // score buffers in TMEM
  constexpr int NS = ring_slots(NRP);      // K/V ring slots
  constexpr uint32_t NEED = ((SC ? 1 : 2) + NSB) * NRP;
  constexpr uint32_t TMEM_COLS = NEED <= 32 ? 32 : NEED <= 64 ? 64 : NEED <= 128 ? 128 : NEED <= 256 ? 256 : 512;
  constexpr uint32_t IDESC_QK = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NRP >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
  constexpr uint32_t IDESC_PV = IDESC_QK | (1u << 15) | (1u << 16);
  static_assert(NRP % 16 == 0 && NRP <= 128 && NSB >= 2, "row padding");

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* sRing = smem;
  unsigned char* sQ = sRing + NS * kTileBytes;
  unsigned char* sP = sQ + 2 * QBOX;                                  // one P buffer per softmax group
  float* s_m = reinterpret_cast<float*>(sP + 2 * PBYTES);            // [2][128] running reference per group
  float* s_fac = s_m + 256;                                           // [2][128] rescale factors (slow path)
  int* s_newmax = reinterpret_cast<int*>(s_fac + 256);               // [2][128]
  uint64_t* bars = reinterpret_cast<uint64_t*>(s_newmax + 256);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 32);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);

  // K_FULL and P_FULL are indexed by tile % 4.  P_FULL(j) completes when the group's 128 threads have stored
  // P(j) AND the V tile has landed (the producer arrives on it with the tile's byte count), so the issuer
  // needs one wait per MMA group.  EMPTY(slot) is committed behind the MMAs that read the slot.
  // There is no "score buffer free" barrier: score tile j+lookahead is issued after P_FULL(j-1) was seen,
  // and a group arrives there only after it has read its scores, which frees every buffer up to j-1.
  enum { K_FULL = 0, P_FULL = 4, P_FREE = 8, Q_READY = 10, O_FULL = 11, O_FREE = 12, S_FULL = 13, EMPTY = 17 };
  auto bar = [&](int i) { return smem_addr(bars + i); };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // ---- this CTA's range of the flattened tile sequence ----
  const long long W = a.total_tiles;
  const long long f_begin = (W * blockIdx.x) / a.n_cta, f_end = (W * (blockIdx.x + 1)) / a.n_cta;
  const int Tt = a.tiles_per_item;
  const int item_first = (int)(f_begin / Tt);

  if (tid == 0) {
    for (int i = 0; i < 4; ++i) { mbar_init(bar(K_FULL + i), 1); mbar_init(bar(P_FULL + i), (SC ? kSoftmaxThreads : kGroupThreads) + 1); }
    for (int i = 0; i < 2; ++i) mbar_init(bar(P_FREE + i), 1);
    for (int i = 0; i < NSB; ++i) mbar_init(bar(S_FULL + i), 1);
    for (int i = 0; i < NS; ++i) mbar_init(bar(EMPTY + i), 1);
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
  for (int i = tid; i < (2 * QBOX + 2 * PBYTES) / 16; i += kThreads) reinterpret_cast<uint4*>(sQ)[i] = make_uint4(0, 0, 0, 0);   // Q and both P buffers (contiguous)
  if (tid < 256) s_newmax[tid] = f2ord(-INFINITY);
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;
  // The launch is a programmatic dependent of whatever kernel precedes it in the stream (the merge of the previous decode
  // step, the gather of the previous round): the set-up above overlaps that kernel's tail; everything below reads
  // tensors it may have produced (Q, K, V) or writes a workspace it may still read, so it comes after this wait.
  pdl_wait();
  // The call's status word is cleared here instead of by a memset in front of the launch (one stream operation less per
  // call, and nothing between this launch and the kernel before it).  A CTA reports an expired wait at its teardown, at
  // least kWaitLimitNs after it started, and CTA 0 is the first CTA of the grid to be dispatched, so this store comes
  // before any report of this call.
  if (blockIdx.x == 0 && tid == 0) *a.status = 0;
  const uint32_t tmem_O = tmem;                    // O accumulators of the two softmax groups: columns [g*NRP, (g+1)*NRP)
  const uint32_t tmem_S = tmem + (SC ? 1 : 2) * NRP;   // score buffers (split-column mode has one accumulator)

  if (f_end > f_begin) {
    if (warp < 4) asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
    if (warp == 0) {
      // =========================== TMA producer ===========================
      // Walks the same loop as the MMA issuer, so tiles enter the ring in the order they leave it:
      // per segment K(0..lookahead), V(0), K(lookahead+1), V(1), ...  It runs ahead across segment
      // boundaries as far as free slots allow.
      if (lane == 0) {
        uint32_t u = 0;                          // loads issued so far (ring position)
        uint32_t jt = 0;
        bool ok = true;
        // K tiles of a call whose mass pass re-reads them are asked to stay in L2, V tiles (read once) to leave first
        const uint64_t pol_k = l2_policy_evict_last(), pol_v = l2_policy_evict_first();
        auto load = [&](const CUtensorMap* map, uint32_t full_bar, long long f) -> bool {
          const uint32_t slot = u % NS;
          if (u >= NS && !mbar_wait(bar(EMPTY + slot), ((u / NS) - 1) & 1, s_abort)) return false;
          const int item = (int)(f / Tt), tile = (int)(f - (long long)item * Tt);
          const int layer = item / a.Hkv, kvh = item - layer * a.Hkv;
          const uint32_t dst = smem_addr(sRing + slot * kTileBytes);
          mbar_expect_tx(full_bar, kTileBytes);
          if (a.l2_hints) {
            const uint64_t pol = map == &tm_k ? pol_k : pol_v;
            tma_load_4d_hint(dst, map, full_bar, 0, kvh, tile * kTile, layer, pol);
            tma_load_4d_hint(dst + kBoxBytes, map, full_bar, 64, kvh, tile * kTile, layer, pol);
          } else {
            tma_load_4d(dst, map, full_bar, 0, kvh, tile * kTile, layer);
            tma_load_4d(dst + kBoxBytes, map, full_bar, 64, kvh, tile * kTile, layer);
          }
          ++u;
          return true;
        };
        for (long long f = f_begin; f < f_end && ok;) {
          const int item = (int)(f / Tt);
          const long long seg_end = min(f_end, (long long)(item + 1) * Tt);
          const int n = (int)(seg_end - f);
          int issued = 0;
          for (int i = 0; i < n && ok; ++i) {
            while (ok && issued < n && issued <= i + a.lookahead) {
              ok = load(&tm_k, bar(K_FULL + ((jt + issued) & 3)), f + issued);
              ++issued;
            }
            if (ok) ok = load(&tm_v, bar(P_FULL + ((jt + i) & 3)), f + i);
          }
          jt += n;
          f = seg_end;
        }
      }
    } else if (warp == 1) {
      // =========================== MMA issuer ===========================
      // The whole warp walks the loop (so tile counters, barrier addresses and descriptors are
      // warp-uniform values) and one elected lane issues the MMAs and commits.  Score tiles run
      // `lookahead` tiles ahead of the PV tiles; the fixed interleave of the two streams keeps the
      // two softmax groups half a period apart.
      {
        const uint32_t q_base = smem_addr(sQ);
        // descriptor constants: only the 14-bit start-address field changes from MMA to MMA
        const uint64_t desc_k0 = make_desc(smem_addr(sRing), 16, 1024, 2), desc_q0 = make_desc(q_base, 16, 1024, 2);
        const uint64_t desc_v0 = make_desc(smem_addr(sRing), kBoxBytes, 1024, 2), desc_p0 = make_desc(smem_addr(sP), 128, 2048, 0);
        uint32_t u = 0;            // ring position (same sequence as the producer's)
        bool ok = true;
        uint32_t jt = 0;           // tiles issued by this CTA so far (ring phases run across segments)
        int seg = 0;
        auto wait_all = [&](uint32_t b, uint32_t parity) -> bool {     // a vote makes the outcome provably warp-uniform
          return __all_sync(0xffffffffu, mbar_wait(b, parity, s_abort));
        };
        auto issue_qk = [&](uint32_t j) -> bool {
          const uint32_t slot = u % NS, sb = j % NSB;
          ++u;
          if (!wait_all(bar(K_FULL + (j & 3)), (j >> 2) & 1)) return false;
          tc_fence_after();
          const uint64_t dk = desc_k0 + (uint64_t)((slot * kTileBytes) >> 4);
          const uint32_t d_tmem = tmem_S + sb * NRP;
          if (elect_one()) {
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              const uint32_t off = (kk >> 2) * kBoxBytes + (kk & 3) * 32, qoff = (kk >> 2) * QBOX + (kk & 3) * 32;
              tc_mma(d_tmem, dk + (off >> 4), desc_q0 + (qoff >> 4), IDESC_QK, kk > 0);
            }
            tc_commit(bar(S_FULL + sb));
            tc_commit(bar(EMPTY + slot));
          }
          __syncwarp();
          return true;
        };
        for (long long f = f_begin; f < f_end && ok; ++seg) {
          const int item = (int)(f / Tt);
          const long long seg_end = min(f_end, (long long)(item + 1) * Tt);
          const int n = (int)(seg_end - f);
          if (!wait_all(bar(Q_READY), seg & 1)) { ok = false; break; }
          tc_fence_after();
          int issued = 0;                                  // score tiles of this segment already issued
          for (int i = 0; i < n; ++i) {
            const uint32_t j = jt + i;
            while (issued < n && issued <= i + a.lookahead) {  // look-ahead: score tiles in flight past tile i
              if (!issue_qk(jt + issued)) { ok = false; break; }
              ++issued;
            }
            if (!ok) break;
            const uint32_t slot = u % NS, g = j & 1;
            ++u;
            if (i == 0 && seg > 0 && !wait_all(bar(O_FREE), (seg - 1) & 1)) { ok = false; break; }
            if (!wait_all(bar(P_FULL + (j & 3)), (j >> 2) & 1)) { ok = false; break; }     // P stored and V landed
            tc_fence_after();
            const uint64_t dv = desc_v0 + (uint64_t)((slot * kTileBytes) >> 4), dp = desc_p0 + (uint64_t)((g * PBYTES) >> 4);
            const uint32_t d_tmem = tmem_O + (SC ? 0 : g * NRP);
            const uint32_t acc0 = i >= (SC ? 1 : 2);       // each accumulator starts afresh in every segment
            if (elect_one()) {
#pragma unroll
              for (int kk = 0; kk < 8; ++kk)
                tc_mma(d_tmem, dv + (uint64_t)((kk * 2048) >> 4), dp + (uint64_t)((kk * 256) >> 4), IDESC_PV, (kk > 0) ? 1u : acc0);
              tc_commit(bar(P_FREE + g));
              tc_commit(bar(EMPTY + slot));
            }
            __syncwarp();
          }
          if (!ok) break;
          if (elect_one()) tc_commit(bar(O_FULL));
          __syncwarp();
          jt += n;
          f = seg_end;
        }
      }
    } else if (warp >= 4) {
      // =========================== softmax warps ===========================
      asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
      // Two groups of four warps work on alternate tiles (group = tile parity), each with its own
      // accumulator, reference m and row sums: two independent online-softmax streams whose
      // partials the combine kernel merges.  A thread owns one key of its group's tile.
      const int q4 = warp & 3;                 // TMEM lane quarter this warp may access
      const int g = (warp - 4) >> 2;           // softmax group
      const int t = q4 * 32 + lane;            // key within the tile == TMEM lane; channel d in the epilogue
      const int st = tid - 128;                // 0..255
      const uint32_t lane_addr = (uint32_t)(q4 * 32) << 16;
      constexpr int NR = NCH * 16;             // query-row columns this thread handles
      const int r0 = SC ? g * NR : 0;          // the first of them (split-column mode: group 1 takes the upper half)
      // per-row state: one set per group, or one set indexed by absolute row in split-column mode
      float* m_s = s_m + (SC ? 0 : g * 128);
      float* fac_s = s_fac + (SC ? 0 : g * 128);
      int* newmax_s = s_newmax + (SC ? 0 : g * 128);
      // per-warp row sums of the epilogue live in the first row group (2 KB) of the group's P buffer: the last
      // PV of the segment has been waited for by then, and every tile rewrites that row group
      float* lsum_s = reinterpret_cast<float*>(sP + g * PBYTES);
      float l_loc[NR];
      uint32_t jt = 0;
      int seg = 0;
      bool ok = true;
      auto group_sync = [&]() { asm volatile("bar.sync %0, 128;" ::"r"(1 + g) : "memory"); };
      auto group_or = [&](bool pred) -> bool {
        uint32_t out;
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t"
            "setp.ne.u32 p, %1, 0;\n\t"
            "bar.red.or.pred q, %2, 128, p;\n\t"
            "selp.u32 %0, 1, 0, q;\n\t}"
            : "=r"(out)
            : "r"((uint32_t)pred), "r"(1 + g)
            : "memory");
        return out != 0;
      };
      // Q of one (layer, KV head) item goes into the K-major 128B-swizzled layout in two steps, so that the global loads
      // can be in flight while the thread does something else: q_load issues them, q_store writes shared memory and
      // tells the issuer.
      constexpr int QP = (NRP * 16 + kSoftmaxThreads - 1) / kSoftmaxThreads;
      uint4 qval[QP];
      auto q_load = [&](int item) {
        const int layer = item / a.Hkv, kvh = item - layer * a.Hkv;
        const __nv_bfloat16* qb = a.q + (long long)layer * a.q_ls + (long long)kvh * a.G * a.D;
        const int cpr = a.D >> 3;                        // 16-byte pieces per query row: 16, or 8 when D = 64
#pragma unroll
        for (int k = 0; k < QP; ++k) {
          const int idx = st + k * kSoftmaxThreads;
          if (idx < a.rows * cpr) {
            const int row = a.D == 128 ? idx >> 4 : idx >> 3, c = idx & (cpr - 1);
            const int r = (int)(((uint32_t)row * a.g_magic) >> 16), gq = row - r * a.G;
            qval[k] = *reinterpret_cast<const uint4*>(qb + ((long long)r * a.Hq + gq) * a.D + c * 8);
          }
        }
      };
      auto q_store = [&]() {
        const int cpr = a.D >> 3;
#pragma unroll
        for (int k = 0; k < QP; ++k) {
          const int idx = st + k * kSoftmaxThreads;
          if (idx < a.rows * cpr) {
            const int row = a.D == 128 ? idx >> 4 : idx >> 3, c = idx & (cpr - 1);
            *reinterpret_cast<uint4*>(sQ + (c >> 3) * QBOX + row * 128 + (((c & 7) ^ (row & 7)) << 4)) = qval[k];
          }
        }
        fence_proxy_async();
        mbar_arrive(bar(Q_READY));
      };
      q_load((int)(f_begin / Tt));
      q_store();
      for (long long f = f_begin; f < f_end; ++seg) {
        const int item = (int)(f / Tt), tile0 = (int)(f - (long long)item * Tt);
        const long long seg_end = min(f_end, (long long)(item + 1) * Tt);
        const int n = (int)(seg_end - f);
        if (t < NR) m_s[r0 + t] = kNegBig;
#pragma unroll
        for (int i = 0; i < NR; ++i) l_loc[i] = 0.f;
        group_sync();

        bool aborted = false;
        const int i_first = SC ? 0 : (((jt & 1) == (uint32_t)g) ? 0 : 1);      // this group's first tile in the segment
        for (int i = i_first; i < n; i += (SC ? 1 : 2)) {
          const uint32_t j = jt + i, sb = j % NSB;
          const uint32_t pb = SC ? (j & 1) : (uint32_t)g;            // P buffer of this tile
          const int tile = tile0 + i;
          const int rel = tile * kTile + t - a.n_ctx;                 // row r sees this key iff rel <= r
          const bool need_mask = (tile * kTile + kTile - 1 > a.n_ctx);
          const uint32_t s_addr = tmem_S + lane_addr + sb * NRP + r0;
          // A failed wait never leaves this loop on its own (the rest of the group would be left at a
          // named barrier): it clears `ok`, and the vote below takes all 128 threads out together.
          ok &= mbar_wait(bar(S_FULL + sb), (j / NSB) & 1, s_abort);
          tc_fence_after();
          if (i == i_first) {
            // First tile of this group's stream: instead of going through the reference-replacement path (row
            // maxima over the tile, two group barriers), guess the reference from ONE key of the tile, its first:
            // m = that key's score + 2 x threshold.  Any reference is valid; if another key of the tile beats the
            // guess by more than the threshold (or the first key is masked for a row: then the "nothing seen"
            // reference stays), the usual test below sends the group through the replacement path after all.
            if (q4 == 0) {                             // the whole warp issues the (warp-collective) TMEM loads; lane 0 = the tile's first key
#pragma unroll 1
              for (int c = 0; c < NCH; ++c) {
                uint32_t raw[16];
                tmem_ld16(s_addr + c * 16, raw);
                tmem_wait_ld();
                reg_fence16(raw);
                if (lane == 0) {
#pragma unroll
                  for (int e = 0; e < 16; ++e) {
                    const bool masked = need_mask && rel > (int)(((uint32_t)(r0 + c * 16 + e) * a.g_magic) >> 16);
                    if (!masked) m_s[r0 + c * 16 + e] = fmaf(__uint_as_float(raw[e]), a.scale_log2, 2.f * kRescaleThreshold);
                  }
                }
                __syncwarp();
              }
            }
            group_sync();
          }
          // ---- scores of this key against all rows: x = s * scale - m (log2 domain), masked ----
          uint32_t xr[NCH][16];                       // TMEM loads land here and are converted in place
          float xmax;
          auto load_x = [&]() {
#pragma unroll
            for (int c = 0; c < NCH; ++c)
              if (CW(c) == 16) tmem_ld16(s_addr + c * 16, xr[c]); else tmem_ld8_lo(s_addr + c * 16, xr[c]);
            tmem_wait_ld();
            float xm[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
            const float4* m4 = reinterpret_cast<const float4*>(m_s + r0);
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
              {
                reg_fence16(xr[c]);
#pragma unroll
                for (int q = 0; q < CW(c) / 4; ++q) {
                  const float4 mq = m4[c * 4 + q];
                  const float v0 = fmaf(__uint_as_float(xr[c][4 * q + 0]), a.scale_log2, -mq.x);
                  const float v1 = fmaf(__uint_as_float(xr[c][4 * q + 1]), a.scale_log2, -mq.y);
                  const float v2 = fmaf(__uint_as_float(xr[c][4 * q + 2]), a.scale_log2, -mq.z);
                  const float v3 = fmaf(__uint_as_float(xr[c][4 * q + 3]), a.scale_log2, -mq.w);
                  xr[c][4 * q + 0] = __float_as_uint(v0);
                  xr[c][4 * q + 1] = __float_as_uint(v1);
                  xr[c][4 * q + 2] = __float_as_uint(v2);
                  xr[c][4 * q + 3] = __float_as_uint(v3);
                  xm[0] = fmaxf(xm[0], v0);
                  xm[1] = fmaxf(xm[1], v1);
                  xm[2] = fmaxf(xm[2], v2);
                  xm[3] = fmaxf(xm[3], v3);
                }
              }
            }
            xmax = fmaxf(fmaxf(xm[0], xm[1]), fmaxf(xm[2], xm[3]));
            if (need_mask) {                          // cold: only the last tile(s) of an item hold keys past a row's horizon
              xmax = -INFINITY;
#pragma unroll 1
              for (int r = 0; r < 1; ++r) {           // (kept in its own block so that it stays out of the hot instruction stream)
#pragma unroll
                for (int c = 0; c < NCH; ++c) {
#pragma unroll
                  for (int e = 0; e < CW(c); ++e) {
                    {
                      if (rel > (int)(((uint32_t)(r0 + c * 16 + e) * a.g_magic) >> 16)) xr[c][e] = __float_as_uint(-INFINITY);
                      xmax = fmaxf(xmax, __uint_as_float(xr[c][e]));
                    }
                  }
                }
              }
            }
          };
          // Attempt 0 converts against the current reference and votes; if the group needs a new reference
          // the slow path installs it and attempt 1 converts again.  (One copy of the conversion code, and
          // the slow path's chunk loops stay rolled: it is cold code and should stay small.)
#pragma unroll 1
          for (int attempt = 0; attempt < 2; ++attempt) {
            load_x();
            if (attempt == 1) break;
            const bool slow = group_or((xmax > kRescaleThreshold) || !ok);
            if (!slow) break;
            if (group_or(!ok)) { aborted = true; break; }              // uniform across the group
            // ------- slow path: new per-row reference, rescale row sums and the accumulator -------
#pragma unroll 1
            for (int c = 0; c < NCH; ++c) {
              const int cw = (HT && c == NCH - 1) ? 8 : 16;
              uint32_t raw[16];
              tmem_ld16(s_addr + c * 16, raw);
              tmem_wait_ld();
              reg_fence16(raw);
#pragma unroll
              for (int e = 0; e < 16; ++e) {
                float v = __uint_as_float(raw[e]) * a.scale_log2;
                if (e >= cw || (need_mask && rel > (int)(((uint32_t)(r0 + c * 16 + e) * a.g_magic) >> 16))) v = -INFINITY;
                // warp maximum in one instruction on the order-preserving integer image of the float
                const int ov = __reduce_max_sync(0xffffffffu, f2ord(v));
                if (lane == 0 && e < cw) atomicMax(&newmax_s[r0 + c * 16 + e], ov);
              }
            }
            group_sync();
            if (t < NR) {
              const int row = r0 + t;
              const float mo = m_s[row], mn = fmaxf(mo, ord2f(newmax_s[row]));
              fac_s[row] = ex2(mo - mn);               // 0 when the row had seen nothing, 1 when nothing changed
              m_s[row] = mn;
              newmax_s[row] = f2ord(-INFINITY);
            }
            group_sync();
#pragma unroll
            for (int k = 0; k < NR; ++k) l_loc[k] *= fac_s[r0 + k];
            if (i >= (SC ? 1 : 2)) {
              // the accumulator holds earlier tiles of the segment: wait until the last of them has been added
              // (split-column mode: the tile before this one, whose P buffer is the other one)
              const uint32_t jp = SC ? j - 1 : j - 2;
              ok &= mbar_wait(bar(P_FREE + (SC ? (jp & 1) : (uint32_t)g)), (jp >> 1) & 1, s_abort);
              tc_fence_after();
#pragma unroll 1
              for (int c = 0; c < NCH; ++c) {
                uint32_t o[16];
                tmem_ld16(tmem_O + lane_addr + (SC ? 0 : g * NRP) + r0 + c * 16, o);
                tmem_wait_ld();
                reg_fence16(o);
#pragma unroll
                for (int e = 0; e < 16; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * fac_s[r0 + c * 16 + e]);
                tmem_st16(tmem_O + lane_addr + (SC ? 0 : g * NRP) + r0 + c * 16, o);
              }
              tmem_wait_st();
            }
          }
          if (aborted) break;
          // ---- probabilities, running sums, bf16 P in the MN-major core-matrix layout ----
          if (i >= 2) ok &= mbar_wait(bar(P_FREE + pb), ((j >> 1) - 1) & 1, s_abort);     // the buffer's last reader: tile j - 2
          unsigned char* pdst = sP + pb * PBYTES + (r0 >> 3) * 2048 + t * 16;
#pragma unroll
          for (int c = 0; c < NCH; ++c) {
            {
              float p[16];
#pragma unroll
              for (int e = 0; e < CW(c); ++e) {
                p[e] = ex2(__uint_as_float(xr[c][e]));
                l_loc[c * 16 + e] += p[e];
              }
              *reinterpret_cast<uint4*>(pdst + (2 * c) * 2048) =
                  make_uint4(pack2(p[0], p[1]), pack2(p[2], p[3]), pack2(p[4], p[5]), pack2(p[6], p[7]));
              if (CW(c) == 16)                       // (the padding row group of a half chunk stays zero from start-up)
                *reinterpret_cast<uint4*>(pdst + (2 * c + 1) * 2048) =
                    make_uint4(pack2(p[8], p[9]), pack2(p[10], p[11]), pack2(p[12], p[13]), pack2(p[14], p[15]));
            }
          }
          fence_proxy_async();
          tc_fence_before();                    // the score buffer has been read: this arrival also releases it
          mbar_arrive(bar(P_FULL + (j & 3)));
        }
        // both groups leave together: the exit vote is per group, so agree across groups here
        if (softmax_bar_or(aborted)) break;
        // Both groups have read the scores of their last tiles, so every score MMA of this segment is done and Q is
        // free: the next item's Q goes in now, and the issuer starts that segment's score MMAs while the epilogue
        // below drains this segment's accumulators.
        if (seg_end < f_end) q_load(item + 1);             // in flight during the wait below
        // ---- segment epilogue: this group's partial O (fp32), and (m, l) per row ----
        ok &= mbar_wait(bar(O_FULL), seg & 1, s_abort);
        tc_fence_after();
        if (seg_end < f_end) q_store();
        // (split-column mode: both groups fill the segment's first slot, each its own rows; the second slot is marked empty)
        const long long slot = ((long long)blockIdx.x * a.seg_max + (item - item_first)) * 2 + (SC ? 0 : g);
        float* po = a.part_o + slot * NRP * 128;
        const bool has_tiles = i_first < n;
        if (has_tiles) {
#pragma unroll
          for (int c = 0; c < NCH; ++c) {
            uint32_t o[16];
            tmem_ld16(tmem_O + lane_addr + (SC ? 0 : g * NRP) + r0 + c * 16, o);
            tmem_wait_ld();
            reg_fence16(o);
#pragma unroll
            for (int e = 0; e < 16; ++e) po[(long long)(r0 + c * 16 + e) * 128 + t] = __uint_as_float(o[e]);
          }
        }
        tc_fence_before();
        mbar_arrive(bar(O_FREE));
#pragma unroll
        for (int k = 0; k < NR; ++k) {
          float v = l_loc[k];
#pragma unroll
          for (int sh = 16; sh >= 1; sh >>= 1) v += __shfl_xor_sync(0xffffffffu, v, sh);
          if (lane == 0) lsum_s[q4 * 128 + k] = v;
        }
        group_sync();
        if (t < NR) {
          const float* ls = lsum_s;
          const float l = ((ls[t] + ls[128 + t]) + ls[256 + t]) + ls[384 + t];
          a.part_ml[(slot * NRP + r0 + t) * 2] = has_tiles ? m_s[r0 + t] : kNegBig;
          a.part_ml[(slot * NRP + r0 + t) * 2 + 1] = has_tiles ? l : 0.f;
        }
        if (SC && g == 1 && t < NRP) {           // the slot of the segment that nobody fills: "saw no key"
          a.part_ml[((slot + 1) * NRP + t) * 2] = kNegBig;
          a.part_ml[((slot + 1) * NRP + t) * 2 + 1] = 0.f;
        }
        group_sync();
        jt += n;
        f = seg_end;
      }
    }
  }

  // ---- teardown (every loop above is bounded, so every thread gets here) ----
  tc_fence_before();
  __syncthreads();
  // This CTA's work is done: the kernel behind this one may be scheduled once every CTA got here (it waits before it
  // reads).  Not earlier: its CTAs would sit on SM slots for the whole run of this kernel and keep another stream's
  // kernels off the SMs this launch leaves free.
  pdl_launch_dependents();
  if (*s_abort) {
    if (tid == 0) atomicExch(a.status, 1);
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);     // let copies / MMAs in flight land before TMEM is released
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
  }
}

struct CombineArgs {
  const float *part_o, *part_ml;
  __nv_bfloat16* o;
  float *lse, *lse2;
  int R, Hq, Hkv, G, rows, nrp, tiles_per_item, seg_max, n_cta;
  int D;                     // real head dimension; partials are always 128 wide
  long long total_tiles, q_ls;
};

// Grid (items, rows): one block per query row.  Warp 0 lists the partial slots of the item; the four
// warps then share the slots round-robin (a lane owns four channels) and their sums are merged in
// fixed order through shared memory, so the result does not depend on timing.
__global__ void __launch_bounds__(128) attn_tc_combine_kernel(const CombineArgs a) {
  const int item = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  __shared__ long long s_slot[2 * kNumSMs + 4];          // at most every CTA contributes two partials
  __shared__ int s_n;
  __shared__ float s_m[4], s_l[4];
  __shared__ float4 s_acc[4][32];
  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    const long long W = a.total_tiles, C = a.n_cta;
    const long long lo = (long long)item * a.tiles_per_item, hi = lo + a.tiles_per_item;
    auto b = [&](long long c) { return (W * c) / C; };
    long long c0 = (lo * C) / W;
    while (c0 + 1 < C && b(c0 + 1) <= lo) ++c0;
    while (c0 > 0 && b(c0) > lo) --c0;
    int n = 0;
    for (long long c = c0; c < C && b(c) < hi && n < 2 * kNumSMs; ++c) {
      if (b(c + 1) <= lo || b(c + 1) == b(c)) continue;
      const long long slot = (c * a.seg_max + (item - (int)(b(c) / a.tiles_per_item))) * 2;
      s_slot[n++] = slot;
      s_slot[n++] = slot + 1;
    }
    s_n = n;
  }
  __syncthreads();
  pdl_wait();                                            // the partials come from the main kernel
  const int n = s_n;
  if (n <= 8) {
    // few partials per item (long tile runs): a warp merges whole rows on its own, no block barriers
    const int layer = item / a.Hkv, kvh = item - layer * a.Hkv;
    for (int row = blockIdx.y * 4 + warp; row < a.rows; row += 4 * gridDim.y) {
      // all (m, l) pairs first, then every partial's row piece in flight at once, then a fixed-order sum
      float2 ml[8];
#pragma unroll
      for (int i = 0; i < 8; ++i)
        ml[i] = i < n ? *reinterpret_cast<const float2*>(a.part_ml + (s_slot[i] * a.nrp + row) * 2) : make_float2(kNegBig, 0.f);
      float mstar = -INFINITY;
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if (ml[i].y > 0.f) mstar = fmaxf(mstar, ml[i].x);
      float4 o[8];
#pragma unroll
      for (int i = 0; i < 8; ++i)
        o[i] = (i < n && ml[i].y > 0.f) ? *reinterpret_cast<const float4*>(a.part_o + (s_slot[i] * a.nrp + row) * 128 + lane * 4)
                                         : make_float4(0.f, 0.f, 0.f, 0.f);
      float l = 0.f;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (!(i < n && ml[i].y > 0.f)) continue;
        const float w = ex2(ml[i].x - mstar);
        l += ml[i].y * w;
        acc.x += o[i].x * w; acc.y += o[i].y * w; acc.z += o[i].z * w; acc.w += o[i].w * w;
      }
      const float inv = 1.f / l;
      const int r = row / a.G, g = row - r * a.G;
      __nv_bfloat16* dst = a.o + (long long)layer * a.q_ls + ((long long)r * a.Hq + kvh * a.G + g) * a.D + lane * 4;
      if (lane * 4 < a.D)
        *reinterpret_cast<uint2*>(dst) = make_uint2(pack2(acc.x * inv, acc.y * inv), pack2(acc.z * inv, acc.w * inv));
      if (lane == 0) {
        const long long li = (long long)layer * a.Hq * a.R + (kvh * a.G + g) * a.R + r;
        const float v2 = mstar + log2f(l);
        a.lse2[li] = v2;
        if (a.lse) a.lse[li] = v2 * kLn2;
      }
    }
    return;
  }
  for (int row = blockIdx.y; row < a.rows; row += gridDim.y) {
  // reference = largest m among the partials that saw a key (every lane scans a strided share)
  float mstar = -INFINITY;
  for (int i = threadIdx.x; i < n; i += 128) {
    const float2 ml = *reinterpret_cast<const float2*>(a.part_ml + (s_slot[i] * a.nrp + row) * 2);
    if (ml.y > 0.f) mstar = fmaxf(mstar, ml.x);
  }
#pragma unroll
  for (int sh = 16; sh >= 1; sh >>= 1) mstar = fmaxf(mstar, __shfl_xor_sync(0xffffffffu, mstar, sh));
  if (lane == 0) s_m[warp] = mstar;
  __syncthreads();
  mstar = fmaxf(fmaxf(s_m[0], s_m[1]), fmaxf(s_m[2], s_m[3]));
  float l = 0.f;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int i = warp; i < n; i += 4) {
    const float2 ml = *reinterpret_cast<const float2*>(a.part_ml + (s_slot[i] * a.nrp + row) * 2);
    if (!(ml.y > 0.f)) continue;                        // a stream in which the row saw no key (or that had no tile)
    const float w = ex2(ml.x - mstar);
    l += ml.y * w;
    const float4 o = *reinterpret_cast<const float4*>(a.part_o + (s_slot[i] * a.nrp + row) * 128 + lane * 4);
    acc.x += o.x * w; acc.y += o.y * w; acc.z += o.z * w; acc.w += o.w * w;
  }
  s_acc[warp][lane] = acc;
  if (lane == 0) s_l[warp] = l;
  __syncthreads();
  if (warp == 0) {
    const float lt = ((s_l[0] + s_l[1]) + s_l[2]) + s_l[3];
    float4 t = s_acc[0][lane];
#pragma unroll
    for (int w = 1; w < 4; ++w) { t.x += s_acc[w][lane].x; t.y += s_acc[w][lane].y; t.z += s_acc[w][lane].z; t.w += s_acc[w][lane].w; }
    const float inv = 1.f / lt;
    const int layer = item / a.Hkv, kvh = item - layer * a.Hkv;
    const int r = row / a.G, g = row - r * a.G;
    __nv_bfloat16* dst = a.o + (long long)layer * a.q_ls + ((long long)r * a.Hq + kvh * a.G + g) * a.D + lane * 4;
    if (lane * 4 < a.D)
      *reinterpret_cast<uint2*>(dst) = make_uint2(pack2(t.x * inv, t.y * inv), pack2(t.z * inv, t.w * inv));
    if (lane == 0) {
      const long long li = (long long)layer * a.Hq * a.R + (kvh * a.G + g) * a.R + r;
      const float v2 = mstar + log2f(lt);
      a.lse2[li] = v2;
      if (a.lse) a.lse[li] = v2 * kLn2;
    }
  }
  __syncthreads();                                       // the shared staging arrays are reused by the next row
  }
}

// The merge for items that many CTAs contributed to (short tile runs: few layers, long contexts).  Grid (items, rows):
// a block per query row.  One thread per contributing CTA works out that CTA's slot; the row's (m, l) pairs go to
// shared memory once, and the four warps take every fourth partial with four loads in flight.  Sums run in a fixed
// order, so the result does not depend on timing.
__global__ void __launch_bounds__(128) attn_tc_combine_many_kernel(const CombineArgs a) {
  const int item = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  __shared__ long long s_slot[2 * kNumSMs + 4];          // at most every CTA contributes two partials (-1: none)
  __shared__ int s_n, s_c0;
  __shared__ float s_m[4], s_l[4];
  __shared__ float4 s_acc[4][32];
  __shared__ float2 s_ml[2 * kNumSMs + 4];
  pdl_launch_dependents();
  {
    // The CTAs whose tile ranges meet this item are consecutive: thread 0 finds the first and the last with a few
    // divisions, then one thread per CTA works out that CTA's slot (-1: a CTA without tiles, possible when there
    // are fewer tiles than CTAs).
    const long long W = a.total_tiles, C = a.n_cta;
    const long long lo = (long long)item * a.tiles_per_item, hi = lo + a.tiles_per_item;
    auto bnd = [&](long long c) { return (W * c) / C; };
    if (threadIdx.x == 0) {
      long long c0 = (lo * C) / W;
      while (c0 + 1 < C && bnd(c0 + 1) <= lo) ++c0;
      while (c0 > 0 && bnd(c0) > lo) --c0;
      long long c1 = ((hi - 1) * C) / W;
      while (c1 + 1 < C && bnd(c1 + 1) < hi) ++c1;
      while (c1 > c0 && bnd(c1) >= hi) --c1;
      s_c0 = (int)c0;
      s_n = 2 * (int)(c1 - c0 + 1);
    }
    __syncthreads();
    const int cnt = s_n >> 1;
    for (int k = threadIdx.x; k < cnt; k += 128) {
      const long long c = s_c0 + k;
      const long long b0 = bnd(c), b1 = bnd(c + 1);
      const long long base = (b1 > b0 && b0 < hi && b1 > lo) ? (c * a.seg_max + (item - (int)(b0 / a.tiles_per_item))) * 2 : -1;
      s_slot[2 * k] = base;
      s_slot[2 * k + 1] = base < 0 ? -1 : base + 1;
    }
    __syncthreads();
  }
  pdl_wait();                                            // the partials come from the main kernel
  const int n = s_n;
  const int layer = item / a.Hkv, kvh = item - layer * a.Hkv;
  auto store_row = [&](int row, float4 acc, float l, float mstar) {       // called by one warp
    const float inv = 1.f / l;
    const int r = row / a.G, g = row - r * a.G;
    __nv_bfloat16* dst = a.o + (long long)layer * a.q_ls + ((long long)r * a.Hq + kvh * a.G + g) * a.D + lane * 4;
    if (lane * 4 < a.D)
      *reinterpret_cast<uint2*>(dst) = make_uint2(pack2(acc.x * inv, acc.y * inv), pack2(acc.z * inv, acc.w * inv));
    if (lane == 0) {
      const long long li = (long long)layer * a.Hq * a.R + (kvh * a.G + g) * a.R + r;
      const float v2 = mstar + log2f(l);
      a.lse2[li] = v2;
      if (a.lse) a.lse[li] = v2 * kLn2;
    }
  };
  for (int row = blockIdx.y; row < a.rows; row += gridDim.y) {
    // (m, l) of every partial of this row into shared memory; reference = largest m among those that saw a key
    float mstar = -INFINITY;
    for (int i = threadIdx.x; i < n; i += 128) {
      const float2 ml = s_slot[i] >= 0 ? *reinterpret_cast<const float2*>(a.part_ml + (s_slot[i] * a.nrp + row) * 2)
                                       : make_float2(kNegBig, 0.f);
      s_ml[i] = ml;
      if (ml.y > 0.f) mstar = fmaxf(mstar, ml.x);
    }
#pragma unroll
    for (int sh = 16; sh >= 1; sh >>= 1) mstar = fmaxf(mstar, __shfl_xor_sync(0xffffffffu, mstar, sh));
    if (lane == 0) s_m[warp] = mstar;
    __syncthreads();
    mstar = fmaxf(fmaxf(s_m[0], s_m[1]), fmaxf(s_m[2], s_m[3]));
    float l = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int i0 = warp; i0 < n; i0 += 16) {               // a warp takes every fourth partial, four loads in flight
      float4 o[4];
      float w[4], lw[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int i = i0 + 4 * k;
        const bool live = i < n && s_ml[i < n ? i : 0].y > 0.f;
        w[k] = live ? ex2(s_ml[i].x - mstar) : 0.f;
        lw[k] = live ? s_ml[i].y * w[k] : 0.f;
        o[k] = live ? *reinterpret_cast<const float4*>(a.part_o + (s_slot[i] * a.nrp + row) * 128 + lane * 4)
                    : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        l += lw[k];
        acc.x += o[k].x * w[k]; acc.y += o[k].y * w[k]; acc.z += o[k].z * w[k]; acc.w += o[k].w * w[k];
      }
    }
    s_acc[warp][lane] = acc;
    if (lane == 0) s_l[warp] = l;
    __syncthreads();
    if (warp == 0) {
      const float lt = ((s_l[0] + s_l[1]) + s_l[2]) + s_l[3];
      float4 t = s_acc[0][lane];
#pragma unroll
      for (int w = 1; w < 4; ++w) { t.x += s_acc[w][lane].x; t.y += s_acc[w][lane].y; t.z += s_acc[w][lane].z; t.w += s_acc[w][lane].w; }
      store_row(row, t, lt, mstar);
    }
    __syncthreads();
  }
}

// ---------------------------------------------------------------------------------------------
// Mass pass on the same machinery: S^T = K . Q^T only (no V, no P, no accumulator).  With the final
// lse of every row known, a thread turns its key's scores into probabilities and adds them over the
// query rows, which in this orientation is a thread-local sum: mass_part[kv head][key].
// ---------------------------------------------------------------------------------------------
constexpr int kMassKStages = 6;             // K tiles in flight: the kernel holds no V, P or accumulators, so shared memory allows six

struct TcMassArgs {
  const __nv_bfloat16* q;
  const float* lse2;         // [n_layers][Hq][R], log2 domain
  float* part_mass;          // [n_mass][Hkv][T_pad]
  int* status;
  int R, Hq, Hkv, G, n_ctx, T, T_pad, rows;
  int D;                     // real head dimension (64 or 128)
  long long q_ls;
  float scale_log2;
  int tiles_per_item, n_cta;
  long long total_tiles;
  uint32_t g_magic;
  int mass_listed;
  int mass_layer[8];
};

template <int NRP>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_mass_kernel(const __grid_constant__ CUtensorMap tm_k, const TcMassArgs a) {
  constexpr bool SC = split_cols(NRP);     // both groups on every tile, half of the query-row columns each (two partial sums per key)
  constexpr int NCH = SC ? NRP / 32 : NRP / 16;
  constexpr int QBOX = NRP * 128;
  constexpr int NSB = (512 / NRP) >= 4 ? 4 : (512 / NRP);
  constexpr uint32_t NEED = NSB * NRP;
  constexpr uint32_t TMEM_COLS = NEED <= 32 ? 32 : NEED <= 64 ? 64 : NEED <= 128 ? 128 : NEED <= 256 ? 256 : 512;
  constexpr uint32_t IDESC_QK = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NRP >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);

  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* sK = smem;
  unsigned char* sQ = sK + kMassKStages * kTileBytes;
  float* s_lse = reinterpret_cast<float*>(sQ + 2 * QBOX);            // [128] lse2 per row (pad rows: +big => p = 0)
  uint64_t* bars = reinterpret_cast<uint64_t*>(s_lse + 128);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 24);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  enum { K_FULL = 0, K_EMPTY = kMassKStages, S_FULL = 2 * kMassKStages, S_FREE = 2 * kMassKStages + 4, Q_READY = 2 * kMassKStages + 8 };
  static_assert(2 * kMassKStages + 9 <= 24, "barrier storage");
  auto bar = [&](int i) { return smem_addr(bars + i); };
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const long long W = a.total_tiles;
  const long long f_begin = (W * blockIdx.x) / a.n_cta, f_end = (W * (blockIdx.x + 1)) / a.n_cta;
  const int Tt = a.tiles_per_item;

  if (tid == 0) {
    for (int i = 0; i < kMassKStages; ++i) { mbar_init(bar(K_FULL + i), 1); mbar_init(bar(K_EMPTY + i), 1); }
    for (int i = 0; i < 4; ++i) { mbar_init(bar(S_FULL + i), 1); mbar_init(bar(S_FREE + i), SC ? kSoftmaxThreads : kGroupThreads); }
    mbar_init(bar(Q_READY), kSoftmaxThreads);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(s_tmem)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  for (int i = tid; i < 2 * QBOX / 16; i += kThreads) reinterpret_cast<uint4*>(sQ)[i] = make_uint4(0, 0, 0, 0);
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  if (f_end > f_begin) {
    const uint32_t total = (uint32_t)(f_end - f_begin);
    if (warp == 0) {
      if (lane == 0) {
        // A CTA walks its tile range BACKWARDS: when this pass covers the same layers as the main pass (a one-layer
        // call) its range is the one that CTA streamed there, and the tiles it read last are the likeliest to be in L2 still.
        for (uint32_t j = 0; j < total; ++j) {
          const long long f = f_end - 1 - j;
          const int item = (int)(f / Tt), tile = (int)(f - (long long)item * Tt);
          const int zrow = item / a.Hkv, kvh = item - zrow * a.Hkv;
          const int layer = a.mass_listed ? a.mass_layer[zrow] : zrow;
          const uint32_t ks = j % kMassKStages;
          if (j >= kMassKStages && !mbar_wait(bar(K_EMPTY + ks), ((j / kMassKStages) - 1) & 1, s_abort)) break;
          mbar_expect_tx(bar(K_FULL + ks), kTileBytes);
          tma_load_4d(smem_addr(sK + ks * kTileBytes), &tm_k, bar(K_FULL + ks), 0, kvh, tile * kTile, layer);
          tma_load_4d(smem_addr(sK + ks * kTileBytes + kBoxBytes), &tm_k, bar(K_FULL + ks), 64, kvh, tile * kTile, layer);
        }
      }
    } else if (warp == 1) {
      if (lane == 0) {
        const uint32_t q_base = smem_addr(sQ);
        uint32_t jt = 0;
        int seg = 0;
        bool ok = true;
        for (long long fh = f_end - 1; fh >= f_begin && ok; ++seg) {        // fh: the segment's highest tile, processed first
          const int item = (int)(fh / Tt);
          const long long seg_lo = max(f_begin, (long long)item * Tt);
          const int n = (int)(fh - seg_lo + 1);
          if (!mbar_wait(bar(Q_READY), seg & 1, s_abort)) break;
          tc_fence_after();
          for (int i = 0; i < n; ++i) {
            const uint32_t j = jt + i, ks = j % kMassKStages, sb = j % NSB;
            if (!mbar_wait(bar(K_FULL + ks), (j / kMassKStages) & 1, s_abort)) { ok = false; break; }
            if (j >= NSB && !mbar_wait(bar(S_FREE + sb), ((j / NSB) - 1) & 1, s_abort)) { ok = false; break; }
            tc_fence_after();
            const uint32_t k_base = smem_addr(sK + ks * kTileBytes);
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              const uint32_t off = (kk >> 2) * kBoxBytes + (kk & 3) * 32, qoff = (kk >> 2) * QBOX + (kk & 3) * 32;
              tc_mma(tmem + sb * NRP, make_desc(k_base + off, 16, 1024, 2), make_desc(q_base + qoff, 16, 1024, 2), IDESC_QK, kk > 0);
            }
            tc_commit(bar(S_FULL + sb));
            tc_commit(bar(K_EMPTY + ks));
          }
          jt += n;
          fh = seg_lo - 1;
        }
      }
    } else if (warp >= 4) {
      const int q4 = warp & 3, g = (warp - 4) >> 2;
      const int t = q4 * 32 + lane, st = tid - 128;
      const uint32_t lane_addr = (uint32_t)(q4 * 32) << 16;
      const int r0 = SC ? g * (NCH * 16) : 0;                    // first query-row column of this thread's share
      const int nch_valid = min(NCH, max(0, (a.rows - r0 + 15) >> 4));
      uint32_t jt = 0;
      int seg = 0;
      bool ok = true;
      for (long long fh = f_end - 1; fh >= f_begin; ++seg) {
        const int item = (int)(fh / Tt), tile_hi = (int)(fh - (long long)item * Tt);
        const long long seg_lo = max(f_begin, (long long)item * Tt);
        const int n = (int)(fh - seg_lo + 1);
        const int zrow = item / a.Hkv, kvh = item - zrow * a.Hkv;
        const int layer = a.mass_listed ? a.mass_layer[zrow] : zrow;
        {
          const __nv_bfloat16* qb = a.q + (long long)layer * a.q_ls + (long long)kvh * a.G * a.D;
          const int cpr = a.D >> 3;                        // 16-byte pieces per query row: 16, or 8 when D = 64
          constexpr int QP = (NRP * 16 + kSoftmaxThreads - 1) / kSoftmaxThreads;
          uint4 val[QP];                                   // all of a thread's pieces are in flight before the first store
#pragma unroll
          for (int k = 0; k < QP; ++k) {
            const int idx = st + k * kSoftmaxThreads;
            if (idx < a.rows * cpr) {
              const int row = a.D == 128 ? idx >> 4 : idx >> 3, c = idx & (cpr - 1);
              const int r = (int)(((uint32_t)row * a.g_magic) >> 16), gq = row - r * a.G;
              val[k] = *reinterpret_cast<const uint4*>(qb + ((long long)r * a.Hq + gq) * a.D + c * 8);
            }
          }
#pragma unroll
          for (int k = 0; k < QP; ++k) {
            const int idx = st + k * kSoftmaxThreads;
            if (idx < a.rows * cpr) {
              const int row = a.D == 128 ? idx >> 4 : idx >> 3, c = idx & (cpr - 1);
              *reinterpret_cast<uint4*>(sQ + (c >> 3) * QBOX + row * 128 + (((c & 7) ^ (row & 7)) << 4)) = val[k];
            }
          }
          pdl_wait();                                      // lse2 comes from the merge kernel (Q, K are the call's inputs)
          if (st < 128) {
            float v = 1.0e30f;
            if (st < a.rows) {
              const int r = (int)(((uint32_t)st * a.g_magic) >> 16), gq = st - r * a.G;
              v = a.lse2[((long long)layer * a.Hq + kvh * a.G + gq) * a.R + r];
            }
            s_lse[st] = v;
          }
          fence_proxy_async();
          mbar_arrive(bar(Q_READY));
        }
        softmax_bar_or(false);                     // s_lse visible to both groups
        const int i_first = SC ? 0 : (((jt & 1) == (uint32_t)g) ? 0 : 1);
        float* out = a.part_mass + (((long long)zrow * a.Hkv + kvh) * (SC ? 2 : 1) + (SC ? g : 0)) * a.T_pad;
        for (int i = i_first; i < n; i += (SC ? 1 : 2)) {
          const uint32_t j = jt + i, sb = j % NSB;
          const int tile = tile_hi - i;
          const int key = tile * kTile + t;
          const int rel = key - a.n_ctx;
          const bool need_mask = (tile * kTile + kTile - 1 > a.n_ctx);
          ok &= mbar_wait(bar(S_FULL + sb), (j / NSB) & 1, s_abort);
          tc_fence_after();
          const uint32_t s_addr = tmem + lane_addr + sb * NRP + r0;
          uint32_t xr[NCH][16];
#pragma unroll
          for (int c = 0; c < NCH; ++c)
            if (c < nch_valid) tmem_ld16(s_addr + c * 16, xr[c]);
          tmem_wait_ld();
          tc_fence_before();
          mbar_arrive(bar(S_FREE + sb));
          // x = s * scale - lse (log2 domain) in place, then the exponentials.  The hot path (every chunk real, no key past a
          // row's horizon) is one straight block, so that the loads of lse, the multiply-adds, the exponentials and the
          // sums of different elements overlap (with the mask test inside the element loop every group of four was a basic
          // block of its own: 0.86 us of arithmetic per tile at 96 padded rows, 0.5 us as one block); masking lives in
          // a cold block of its own.
          float acc[4] = {0.f, 0.f, 0.f, 0.f};
          const float4* l4 = reinterpret_cast<const float4*>(s_lse + r0);
          auto to_x = [&](int c) {
            reg_fence16(xr[c]);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const float4 lq = l4[c * 4 + q];
              xr[c][4 * q + 0] = __float_as_uint(fmaf(__uint_as_float(xr[c][4 * q + 0]), a.scale_log2, -lq.x));
              xr[c][4 * q + 1] = __float_as_uint(fmaf(__uint_as_float(xr[c][4 * q + 1]), a.scale_log2, -lq.y));
              xr[c][4 * q + 2] = __float_as_uint(fmaf(__uint_as_float(xr[c][4 * q + 2]), a.scale_log2, -lq.z));
              xr[c][4 * q + 3] = __float_as_uint(fmaf(__uint_as_float(xr[c][4 * q + 3]), a.scale_log2, -lq.w));
            }
          };
          auto add_p = [&](int c) {
#pragma unroll
            for (int e = 0; e < 16; ++e) acc[e & 3] += ex2(__uint_as_float(xr[c][e]));
          };
          if (nch_valid == NCH && !need_mask) {
#pragma unroll
            for (int c = 0; c < NCH; ++c) to_x(c);
#pragma unroll
            for (int c = 0; c < NCH; ++c) add_p(c);
          } else {
#pragma unroll 1
            for (int r = 0; r < 1; ++r) {                 // (its own block: stays out of the hot instruction stream)
#pragma unroll
              for (int c = 0; c < NCH; ++c) {
                if (c < nch_valid) {
                  to_x(c);
                  if (need_mask) {
#pragma unroll
                    for (int e = 0; e < 16; ++e)
                      if (rel > (int)(((uint32_t)(r0 + c * 16 + e) * a.g_magic) >> 16)) xr[c][e] = __float_as_uint(-INFINITY);
                  }
                  add_p(c);
                }
              }
            }
          }
          if (key < a.T) out[key] = (acc[0] + acc[1]) + (acc[2] + acc[3]);
        }
        // all score MMAs of the segment have been consumed by one of the groups: Q may be replaced
        if (softmax_bar_or(!ok)) break;
        jt += n;
        fh = seg_lo - 1;
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  pdl_launch_dependents();                 // at the end, as in the main kernel
  if (*s_abort) {
    if (tid == 0) atomicExch(a.status, 1);
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
  }
}

// part: [n_mass][n_part][T_pad] with n_part = KV heads (x 2 in split-column mode), summed in fixed order
__global__ void mass_reduce_tc_kernel(const float* part, float* mass, int Hkv, int T, int T_pad, long long mass_ls) {
  pdl_launch_dependents();
  pdl_wait();
  const int zrow = blockIdx.y;
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= T) return;
  float acc = 0.f;
  for (int h = 0; h < Hkv; ++h) acc += part[((long long)zrow * Hkv + h) * T_pad + j];      // fixed order
  mass[(long long)zrow * mass_ls + j] = acc;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Looked up once per process; the initialisation of a function-local static is thread-safe, so host threads
// that make their first attention call at the same time all see the finished pointer.
EncodeTiledFn encode_tiled_fn() {
  static const EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
        qr == cudaDriverEntryPointSuccess)
      return reinterpret_cast<EncodeTiledFn>(p);
    return nullptr;
  }();
  return fn;
}

bool make_kv_map(CUtensorMap* map, const void* base, const pvlm_attn_params& p, int T) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {(cuuint64_t)p.D, (cuuint64_t)p.Hkv, (cuuint64_t)T, (cuuint64_t)p.n_layers};   // D = 64: box 1 is all fill
  const cuuint64_t layer_stride = p.n_layers > 1 ? (cuuint64_t)p.kv_layer_stride : (cuuint64_t)T * p.kv_token_stride;
  const cuuint64_t strides[3] = {(cuuint64_t)p.kv_head_stride * 2, (cuuint64_t)p.kv_token_stride * 2, layer_stride * 2};
  const cuuint32_t box[4] = {64, 1, (cuuint32_t)kTile, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// cudaFuncSetAttribute once per kernel and device instead of on every launch (the attribute belongs to the device's
// copy of the function; devices beyond the 64th set it every time).  The kernel is a template argument, so that every
// instantiation has a flag word of its own.
template <auto Kernel>
void set_max_dynamic_smem_once(int bytes) {
  static std::atomic<unsigned long long> done{0};
  int dev = 0;
  cudaGetDevice(&dev);
  const unsigned long long bit = (dev >= 0 && dev < 64) ? 1ull << dev : 0ull;
  if (bit && (done.load(std::memory_order_acquire) & bit)) return;
  cudaFuncSetAttribute(Kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (bit) done.fetch_or(bit, std::memory_order_release);
}

template <int NRP>
constexpr int tc_smem_bytes() {
  return 1024 /*alignment slack*/ + ring_slots(NRP) * kTileBytes + 2 * NRP * 128 + 2 * NRP * 256 + 3 * 256 * 4 + 32 * 8 + 64;
}

template <int NRP>
void launch_tc(const CUtensorMap& mk, const CUtensorMap& mv, const TcArgs& a, cudaStream_t s) {
  constexpr int smem = tc_smem_bytes<NRP>();
  if constexpr (!split_cols(NRP)) {
    if (a.rows <= NRP - 8) {
      set_max_dynamic_smem_once<attn_tc_kernel<NRP, true>>(smem);
      const cudaError_t e = launch_dependent(attn_tc_kernel<NRP, true>, dim3(a.n_cta), dim3(kThreads), smem, s, mk, mv, a);
      if (e != cudaSuccess) set_cuda_error((int)e);
      return;
    }
  }
  {
    set_max_dynamic_smem_once<attn_tc_kernel<NRP, false>>(smem);
    const cudaError_t e = launch_dependent(attn_tc_kernel<NRP, false>, dim3(a.n_cta), dim3(kThreads), smem, s, mk, mv, a);
    if (e != cudaSuccess) set_cuda_error((int)e);
  }
}

template <int NRP>
void launch_tc_mass(const CUtensorMap& mk, const TcMassArgs& a, cudaStream_t s) {
  constexpr int smem = 1024 + kMassKStages * kTileBytes + 2 * NRP * 128 + 128 * 4 + 24 * 8 + 64;
  set_max_dynamic_smem_once<attn_tc_mass_kernel<NRP>>(smem);
  const cudaError_t e = launch_dependent(attn_tc_mass_kernel<NRP>, dim3(a.n_cta), dim3(kThreads), smem, s, mk, a);
  if (e != cudaSuccess) set_cuda_error((int)e);
}

}  // namespace

pvlm_status launch_attn_mass_tc(const pvlm_attn_params& p, const float* lse2, float* part_mass, int* status, cudaStream_t s) {
  const int G = p.Hq / p.Hkv, rows = G * p.R, nrp = (rows + 15) / 16 * 16;
  const int T = p.n_ctx + p.R;
  CUtensorMap mk;
  if (!make_kv_map(&mk, p.k, p, T)) return PVLM_ERR_UNSUPPORTED;
  TcMassArgs a;
  a.q = (const __nv_bfloat16*)p.q; a.lse2 = lse2; a.part_mass = part_mass; a.status = status;
  a.R = p.R; a.Hq = p.Hq; a.Hkv = p.Hkv; a.G = G; a.n_ctx = p.n_ctx; a.T = T; a.T_pad = (int)align_up(T, kAttnBN); a.rows = rows;
  a.D = p.D;
  a.q_ls = p.q_layer_stride;
  const float scale = (p.softmax_scale == 0.f) ? 1.0f / sqrtf((float)p.D) : p.softmax_scale;
  a.scale_log2 = scale * kLog2e;
  a.mass_listed = p.mass_layers != nullptr;
  const int n_mass = a.mass_listed ? p.n_mass_layers : p.n_layers;
  for (int i = 0; i < 8; ++i) a.mass_layer[i] = (a.mass_listed && i < p.n_mass_layers) ? p.mass_layers[i] : 0;
  a.tiles_per_item = ceil_div(T, kTile);
  a.total_tiles = (long long)a.tiles_per_item * p.Hkv * n_mass;
  a.n_cta = (int)(a.total_tiles < kNumSMs ? a.total_tiles : kNumSMs);
  if (p.max_ctas > 0 && p.max_ctas < a.n_cta) a.n_cta = p.max_ctas;
  a.g_magic = (65536u + G - 1) / G;
  switch (nrp) {
    case 16: launch_tc_mass<16>(mk, a, s); break;
    case 32: launch_tc_mass<32>(mk, a, s); break;
    case 48: launch_tc_mass<48>(mk, a, s); break;
    case 64: launch_tc_mass<64>(mk, a, s); break;
    case 80: launch_tc_mass<80>(mk, a, s); break;
    case 96: launch_tc_mass<96>(mk, a, s); break;
    case 112: launch_tc_mass<112>(mk, a, s); break;
    case 128: launch_tc_mass<128>(mk, a, s); break;
    default: return PVLM_ERR_UNSUPPORTED;
  }
  const cudaError_t e = launch_dependent(mass_reduce_tc_kernel, dim3(ceil_div(T, 256), n_mass), dim3(256), 0, s,
                                         (const float*)part_mass, p.mass, p.Hkv * (split_cols(nrp) ? 2 : 1), T, a.T_pad,
                                         p.mass_layer_stride);
  if (e != cudaSuccess) set_cuda_error((int)e);
  return check_launch();
}

bool make_attn_tc_plan(const pvlm_attn_params& p, AttnTcPlan& plan) {
  if ((p.D != 128 && p.D != 64) || p.Hkv <= 0 || p.Hq % p.Hkv != 0) return false;
  const int G = p.Hq / p.Hkv;
  const int rows = G * p.R;
  if (rows > 128) return false;                  // one tile row per TMEM lane: at most 128 query rows per KV head
  plan.nrp = (rows + 15) / 16 * 16;
  plan.T = p.n_ctx + p.R;
  plan.tiles_per_item = ceil_div(plan.T, kTile);
  plan.total_tiles = (long long)plan.tiles_per_item * p.Hkv * p.n_layers;
  plan.n_cta = (int)(plan.total_tiles < kNumSMs ? plan.total_tiles : kNumSMs);
  if (p.max_ctas > 0 && p.max_ctas < plan.n_cta) plan.n_cta = p.max_ctas;
  // test switch: fewer CTAs => longer tile runs and more segments per CTA
  const int opt_ctas = option_value(PVLM_OPT_ATTN_MAX_CTAS);
  if (opt_ctas >= 1 && opt_ctas < plan.n_cta) plan.n_cta = opt_ctas;
  const long long per_cta = (plan.total_tiles + plan.n_cta - 1) / plan.n_cta;
  plan.seg_max = (int)((per_cta + plan.tiles_per_item - 1) / plan.tiles_per_item) + 1;
  size_t off = 0;
  // two partial slots (one per softmax group) per segment
  plan.off_part_o = off;  off += align_up((size_t)plan.n_cta * plan.seg_max * 2 * plan.nrp * 128 * 4, 256);
  plan.off_part_ml = off; off += align_up((size_t)plan.n_cta * plan.seg_max * 2 * plan.nrp * 2 * 4, 256);
  plan.off_status = off;  off += 8192;
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
  a.D = p.D;
  a.q_ls = p.q_layer_stride;
  const float scale = (p.softmax_scale == 0.f) ? 1.0f / sqrtf((float)p.D) : p.softmax_scale;
  a.scale_log2 = scale * kLog2e;
  a.tiles_per_item = plan.tiles_per_item; a.total_tiles = plan.total_tiles; a.seg_max = plan.seg_max; a.n_cta = plan.n_cta;
  a.g_magic = (65536u + a.G - 1) / a.G;
  {
    a.lookahead = s_bufs(plan.nrp) - 1;
    // worth it only where the mass pass re-reads a sizeable share of what this launch streams: every layer's mass wanted
    a.l2_hints = (p.mass != nullptr && (p.mass_layers == nullptr || p.n_mass_layers == p.n_layers)) ? 1 : 0;
  }
  if (p.prof_event_begin) cudaEventRecord((cudaEvent_t)p.prof_event_begin, s);
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
  if (p.prof_event_end) cudaEventRecord((cudaEvent_t)p.prof_event_end, s);
  if (cudaEvent_t ev = take_after_main_event()) cudaEventRecord(ev, s);     // lets a caller queue other work behind the main kernel
  CombineArgs c;
  c.part_o = a.part_o; c.part_ml = a.part_ml; c.o = (__nv_bfloat16*)p.o; c.lse = p.lse; c.lse2 = lse2;
  c.R = p.R; c.Hq = p.Hq; c.Hkv = p.Hkv; c.G = a.G; c.rows = a.rows; c.nrp = plan.nrp;
  c.tiles_per_item = plan.tiles_per_item; c.seg_max = plan.seg_max; c.n_cta = plan.n_cta;
  c.total_tiles = plan.total_tiles; c.q_ls = p.q_layer_stride;
  c.D = p.D;
  {
    const int items = p.Hkv * p.n_layers;
    int rows_y = 2048 / items;                            // enough blocks to fill the GPU, not tens of thousands (1024 / 4096 / 8192
                                                          // blocks measured 23.7 / 26.8 / 31.7 us against 24.9 at the 64-layer config)
    rows_y = rows_y < 1 ? 1 : (rows_y > a.rows ? a.rows : rows_y);
    // an item's tiles are spread over at most this many CTAs, each with two partials
    const long long ctas_per_item = ((long long)plan.tiles_per_item * plan.n_cta + plan.total_tiles - 1) / plan.total_tiles + 1;
    const cudaError_t e = 2 * ctas_per_item <= 8 ? launch_dependent(attn_tc_combine_kernel, dim3(items, rows_y), dim3(128), 0, s, c)
                                                 : launch_dependent(attn_tc_combine_many_kernel, dim3(items, rows_y), dim3(128), 0, s, c);
    if (e != cudaSuccess) set_cuda_error((int)e);
  }
  return check_launch();
}

}  // namespace pvlm
