// UV-Prune: variation score, deterministic Top-K (radix select with
// lower-index tie break, ascending output) and the row gather that builds the
// compacted draft cache.
#include "pvlm_common.cuh"
#include <cooperative_groups.h>
#include <mutex>

namespace pvlm {

namespace {

constexpr int kSelThreads = 1024;
#ifndef PVLM_WIDE_SELECT_MIN
#define PVLM_WIDE_SELECT_MIN 32769
#endif
constexpr int kWideSelectMinTokens = PVLM_WIDE_SELECT_MIN;   // from this many tokens on the selection uses a 16-CTA cluster
constexpr int kSelWarps = kSelThreads / 32;

// Order-preserving map fp32 -> uint32 (larger float => larger key); -0.0 maps
// with +0.0; NaN maps to 0 (below every number, -inf included).
__device__ __forceinline__ uint32_t score_key(float s) {
  if (s != s) return 0u;
  uint32_t b = __float_as_uint(s + 0.0f);          // -0.0 + 0.0 = +0.0
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

struct SelArgs {
  const float *cur, *ref;
  float* score;
  uint32_t* keys;     // workspace [m]
  int* kept;
  int m, k;
};

// Single CTA: m <= 2^24 elements, 4 radix passes of 8 bits over keys kept in
// global/L2, then an ordered compaction.
__global__ void __launch_bounds__(kSelThreads) uvprune_select_kernel(const SelArgs a) {
  pdl_wait();                  // the masses may come from the kernel right before (programmatic dependent launch)
  __shared__ unsigned int hist[256];
  __shared__ unsigned int s_prefix, s_remaining;
  __shared__ int warp_eq[kSelWarps], warp_sel[kSelWarps];
  __shared__ int base_eq, base_sel;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // pass 0: scores and keys
  for (int i = tid; i < a.m; i += kSelThreads) {
    const float s = a.ref ? __fsub_rn(a.cur[i], a.ref[i]) : a.cur[i];
    if (a.score) a.score[i] = s;
    a.keys[i] = score_key(s);
  }
  if (tid == 0) { s_prefix = 0u; s_remaining = (unsigned)a.k; }
  __syncthreads();
  if (a.k == 0) return;

  uint32_t mask = 0u;
  for (int shift = 24; shift >= 0; shift -= 8) {
    if (tid < 256) hist[tid] = 0u;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    for (int i0 = 0; i0 < a.m; i0 += kSelThreads) {      // uniform trip count: every lane reaches the ballot
      const int i = i0 + tid;
      const uint32_t key = (i < a.m) ? a.keys[i] : 0u;
      const bool in = (i < a.m) && (key & mask) == prefix;
      // warp-aggregated histogram update: lanes with the same digit elect one adder
      const unsigned digit = (key >> shift) & 0xFFu;
      const unsigned active = __ballot_sync(0xffffffffu, in);
      if (in) {
        const unsigned peers = __match_any_sync(active, digit);
        if ((int)(__ffs(peers) - 1) == lane) atomicAdd(&hist[digit], (unsigned)__popc(peers));
      }
    }
    __syncthreads();
    if (tid == 0) {
      unsigned remaining = s_remaining, cum = 0u;
      int d = 255;
      for (; d > 0; --d) {
        if (cum + hist[d] >= remaining) break;
        cum += hist[d];
      }
      s_remaining = remaining - cum;           // how many to take from digit d's bucket
      s_prefix = prefix | ((uint32_t)d << shift);
    }
    mask |= (0xFFu << shift);
    __syncthreads();
  }
  const uint32_t tau = s_prefix;               // key of the k-th largest score
  const int take_eq = (int)s_remaining;        // equals to keep, lowest indices first

  if (tid == 0) { base_eq = 0; base_sel = 0; }
  __syncthreads();
  for (int i0 = 0; i0 < a.m; i0 += kSelThreads) {
    const int i = i0 + tid;
    const uint32_t key = (i < a.m) ? a.keys[i] : 0u;
    const bool gt = (i < a.m) && key > tau;
    const bool eq = (i < a.m) && key == tau;
    const unsigned eq_b = __ballot_sync(0xffffffffu, eq);
    if (lane == 0) warp_eq[warp] = __popc(eq_b);
    __syncthreads();
    int eq_before = base_eq + __popc(eq_b & ((1u << lane) - 1u));
    for (int w = 0; w < warp; ++w) eq_before += warp_eq[w];
    const bool sel = gt || (eq && eq_before < take_eq);
    const unsigned sel_b = __ballot_sync(0xffffffffu, sel);
    if (lane == 0) warp_sel[warp] = __popc(sel_b);
    __syncthreads();
    int pos = base_sel + __popc(sel_b & ((1u << lane) - 1u));
    for (int w = 0; w < warp; ++w) pos += warp_sel[w];
    if (sel) a.kept[pos] = i;
    __syncthreads();
    if (tid == kSelThreads - 1) {
      base_eq = eq_before + (eq ? 1 : 0);
      base_sel = pos + (sel ? 1 : 0);
    }
    __syncthreads();
  }
}

// Block-wide exclusive prefix sum over 1024 threads; `total` receives the block sum.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_sums, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int sh = 1; sh < 32; sh <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, sh);
    if (lane >= sh) incl += t;
  }
  __syncthreads();                       // warp_sums may still be read from a previous call
  if (lane == 31) warp_sums[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int w = warp_sums[lane], wi = w;
#pragma unroll
    for (int sh = 1; sh < 32; sh <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, wi, sh);
      if (lane >= sh) wi += t;
    }
    warp_sums[lane] = wi - w;            // exclusive offset of each warp
    if (lane == 31) warp_sums[32] = wi;  // block total
  }
  __syncthreads();
  total = warp_sums[32];
  return warp_sums[warp] + incl - v;
}

// Register-resident variant for m <= ITEMS * 1024.  Warp w owns the ITEMS*32 consecutive scores
// starting at w*ITEMS*32; lane l holds elements w*ITEMS*32 + i*32 + l (coalesced loads), so index
// order inside a warp is (i, lane) and ordered compaction needs only ballots plus two block scans.
template <int ITEMS>
__global__ void __launch_bounds__(kSelThreads) uvprune_select_reg_kernel(const SelArgs a) {
  pdl_wait();                  // the masses may come from the kernel right before (programmatic dependent launch)
  __shared__ unsigned int hist[256];
  __shared__ unsigned int hist_l[256 * 32];              // one histogram column per lane: bank = lane, so the
                                                         // atomics of a warp never collide, whatever the digits
  __shared__ unsigned int s_prefix, s_remaining;
  __shared__ int wsum[33];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int base = warp * (ITEMS * 32) + lane;
  uint32_t key[ITEMS];
  uint32_t valid = 0u;
#pragma unroll
  for (int i = 0; i < ITEMS; ++i) {
    const int idx = base + i * 32;
    key[i] = 0u;
    if (idx < a.m) {
      const float s = a.ref ? __fsub_rn(a.cur[idx], a.ref[idx]) : a.cur[idx];
      if (a.score) a.score[idx] = s;
      key[i] = score_key(s);
      valid |= 1u << i;
    }
  }
  if (a.k == 0) return;
  if (tid == 0) { s_prefix = 0u; s_remaining = (unsigned)a.k; }
  uint32_t mask = 0u;
  for (int shift = 24; shift >= 0; shift -= 8) {
    for (int i = tid; i < 256 * 32; i += kSelThreads) hist_l[i] = 0u;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    const unsigned remaining = s_remaining;
#pragma unroll
    for (int i = 0; i < ITEMS; ++i)
      if (((valid >> i) & 1u) && (key[i] & mask) == prefix) atomicAdd(&hist_l[(((key[i] >> shift) & 0xFFu) << 5) + lane], 1u);
    __syncthreads();
    if (tid < 256) {
      unsigned t = 0;
#pragma unroll 8
      for (int j = 0; j < 32; ++j) t += hist_l[(tid << 5) + ((j + tid) & 31)];     // rotated: conflict-free
      hist[tid] = t;
    }
    __syncthreads();
    // bins in descending digit order across threads 0..255: find the bin where the running count reaches `remaining`
    unsigned v = 0, incl = 0;
    if (tid < 256) {
      v = hist[255 - tid];
      incl = v;
#pragma unroll
      for (int sh = 1; sh < 32; sh <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, incl, sh);
        if (lane >= sh) incl += t;
      }
      if (lane == 31) wsum[warp] = (int)incl;
    }
    __syncthreads();
    if (tid < 256) {
      for (int w = 0; w < warp; ++w) incl += (unsigned)wsum[w];
      const unsigned excl = incl - v;
      if (excl < remaining && incl >= remaining) {
        s_prefix = prefix | ((uint32_t)(255 - tid) << shift);
        s_remaining = remaining - excl;
      }
    }
    mask |= (0xFFu << shift);
    __syncthreads();
  }
  const uint32_t tau = s_prefix;
  const int take_eq = (int)s_remaining;
  const unsigned lt_mask = (1u << lane) - 1u;
  // equals per warp -> rank of every equal element in index order
  int warp_eq = 0;
#pragma unroll
  for (int i = 0; i < ITEMS; ++i) warp_eq += __popc(__ballot_sync(0xffffffffu, ((valid >> i) & 1u) && key[i] == tau));
  int total;
  int eq_run = block_exclusive_scan(lane == 31 ? warp_eq : 0, wsum, total);   // lane 31 carries the warp's count
  eq_run = __shfl_sync(0xffffffffu, eq_run, 31);                              // equals in all earlier warps
  uint32_t selbits = 0u;
  int warp_sel = 0;
#pragma unroll
  for (int i = 0; i < ITEMS; ++i) {
    const bool v = (valid >> i) & 1u;
    const bool eq = v && key[i] == tau;
    const unsigned eq_b = __ballot_sync(0xffffffffu, eq);
    const int rank = eq_run + __popc(eq_b & lt_mask);
    const bool sel = v && (key[i] > tau || (eq && rank < take_eq));
    eq_run += __popc(eq_b);
    const unsigned sel_b = __ballot_sync(0xffffffffu, sel);
    if (sel) selbits |= 1u << i;
    warp_sel += __popc(sel_b);
  }
  int pos = block_exclusive_scan(lane == 31 ? warp_sel : 0, wsum, total);
  pos = __shfl_sync(0xffffffffu, pos, 31);                                    // selected in all earlier warps
#pragma unroll
  for (int i = 0; i < ITEMS; ++i) {
    const unsigned sel_b = __ballot_sync(0xffffffffu, (selbits >> i) & 1u);
    if ((selbits >> i) & 1u) a.kept[pos + __popc(sel_b & lt_mask)] = base + i * 32;
    pos += __popc(sel_b);
  }
}

// Cluster variant: 8 CTAs (one thread-block cluster, 8 SMs) share the selection.  CTA r owns the
// ITEMS*1024 consecutive scores starting at r*ITEMS*1024 (keys in registers, warp-coalesced as
// above); per radix pass every CTA builds its own histogram, the cluster synchronises, and every CTA
// adds up all eight histograms through distributed shared memory, so all CTAs derive the same
// threshold without any global-memory round trip.  The ordered compaction needs one more exchange
// (per-CTA counts of greater and of equal keys).  m <= 8 * 1024 * ITEMS.
// kSelCluster: CTAs per cluster, 8 (portable) or 16 (needs the non-portable cluster size attribute at launch).
template <int ITEMS, int kSelCluster>
__global__ void __cluster_dims__(kSelCluster, 1, 1) __launch_bounds__(kSelThreads)
uvprune_select_cluster_kernel(const SelArgs a) {
  pdl_wait();                  // the masses may come from the kernel right before (programmatic dependent launch)
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  const unsigned rank = cluster.block_rank();
  __shared__ unsigned int hist[2][256];                  // this CTA's histogram of the pass (read remotely); two buffers, so
                                                         // that one cluster barrier per pass is enough (see below)
  __shared__ unsigned int hist_l[256 * 32];
  __shared__ unsigned int s_prefix, s_remaining;
  __shared__ int s_cnt[kSelCluster];                     // (greater << 16 | equal) counts of every CTA, each written by its owner
  __shared__ int wsum[33];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int base = (int)rank * (ITEMS * kSelThreads) + warp * (ITEMS * 32) + lane;
  uint32_t key[ITEMS];
  uint32_t valid = 0u;
#pragma unroll
  for (int i = 0; i < ITEMS; ++i) {
    const int idx = base + i * 32;
    key[i] = 0u;
    if (idx < a.m) {
      const float s = a.ref ? __fsub_rn(a.cur[idx], a.ref[idx]) : a.cur[idx];
      if (a.score) a.score[idx] = s;
      key[i] = score_key(s);
      valid |= 1u << i;
    }
  }
  if (a.k == 0) return;                                  // uniform over the cluster: nobody reaches a cluster barrier
  if (tid == 0) { s_prefix = 0u; s_remaining = (unsigned)a.k; }
  uint32_t mask = 0u;
  int pass = 0;
  for (int shift = 24; shift >= 0; shift -= 8, ++pass) {
    unsigned int* hist_p = hist[pass & 1];
    for (int i = tid; i < 256 * 32; i += kSelThreads) hist_l[i] = 0u;
    __syncthreads();
    const uint32_t prefix = s_prefix;
    const unsigned remaining = s_remaining;
#pragma unroll
    for (int i = 0; i < ITEMS; ++i)
      if (((valid >> i) & 1u) && (key[i] & mask) == prefix) atomicAdd(&hist_l[(((key[i] >> shift) & 0xFFu) << 5) + lane], 1u);
    __syncthreads();
    if (tid < 256) {
      unsigned t = 0;
#pragma unroll 8
      for (int j = 0; j < 32; ++j) t += hist_l[(tid << 5) + ((j + tid) & 31)];
      hist_p[tid] = t;
    }
    // Every CTA's histogram of this pass is complete.  No second barrier after the remote reads: the next pass writes the
    // OTHER buffer, and this one is written again two passes on, behind the next pass's barrier, which a CTA reaches only
    // after its reads here.
    cluster.sync();
    unsigned v = 0, incl = 0;
    if (tid < 256) {
#pragma unroll
      for (int r = 0; r < kSelCluster; ++r) v += cluster.map_shared_rank(hist_p, r)[255 - tid];   // descending digit order
      incl = v;
#pragma unroll
      for (int sh = 1; sh < 32; sh <<= 1) {
        const unsigned t = __shfl_up_sync(0xffffffffu, incl, sh);
        if (lane >= sh) incl += t;
      }
      if (lane == 31) wsum[warp] = (int)incl;
    }
    __syncthreads();
    if (tid < 256) {
      for (int w = 0; w < warp; ++w) incl += (unsigned)wsum[w];
      const unsigned excl = incl - v;
      if (excl < remaining && incl >= remaining) {
        s_prefix = prefix | ((uint32_t)(255 - tid) << shift);
        s_remaining = remaining - excl;
      }
    }
    mask |= (0xFFu << shift);
    __syncthreads();                                     // s_prefix / s_remaining are visible to the whole CTA
  }
  const uint32_t tau = s_prefix;
  const int take_eq = (int)s_remaining;
  const unsigned lt_mask = (1u << lane) - 1u;
  int warp_eq = 0, warp_gt = 0;
#pragma unroll
  for (int i = 0; i < ITEMS; ++i) {
    const bool vld = (valid >> i) & 1u;
    warp_eq += __popc(__ballot_sync(0xffffffffu, vld && key[i] == tau));
    warp_gt += __popc(__ballot_sync(0xffffffffu, vld && key[i] > tau));
  }
  // one scan for both counts: a CTA holds at most ITEMS * 1024 <= 32768 keys, so (greater, equal) fit the halves of a word
  static_assert(ITEMS * kSelThreads <= 32768, "packed counts");
  int cta_cnt;
  int run = block_exclusive_scan(lane == 31 ? ((warp_gt << 16) | warp_eq) : 0, wsum, cta_cnt);
  int eq_run = __shfl_sync(0xffffffffu, run, 31) & 0xFFFF;
  // every CTA stores its counts into every member's shared memory (distributed shared memory), so that after ONE cluster
  // barrier all reads are local and nobody's shared memory is touched again
  if (tid < kSelCluster) *cluster.map_shared_rank(&s_cnt[rank], tid) = cta_cnt;
  cluster.sync();
  // counts of the CTAs before this one: equals before => how many of mine are kept; kept before => output offset
  int eq_base = 0, sel_base = 0;
#pragma unroll
  for (int r = 0; r < kSelCluster; ++r) {
    if (r < (int)rank) {
      const unsigned c = (unsigned)s_cnt[r];
      const int g = (int)(c >> 16), e = (int)(c & 0xFFFFu);
      const int kept_eq = min(max(take_eq - eq_base, 0), e);
      sel_base += g + kept_eq;
      eq_base += e;
    }
  }
  eq_run += eq_base;
  uint32_t selbits = 0u;
  int warp_sel = 0;
#pragma unroll
  for (int i = 0; i < ITEMS; ++i) {
    const bool vld = (valid >> i) & 1u;
    const bool eq = vld && key[i] == tau;
    const unsigned eq_b = __ballot_sync(0xffffffffu, eq);
    const int rnk = eq_run + __popc(eq_b & lt_mask);
    const bool sel = vld && (key[i] > tau || (eq && rnk < take_eq));
    eq_run += __popc(eq_b);
    const unsigned sel_b = __ballot_sync(0xffffffffu, sel);
    if (sel) selbits |= 1u << i;
    warp_sel += __popc(sel_b);
  }
  int total;
  int pos = block_exclusive_scan(lane == 31 ? warp_sel : 0, wsum, total);
  pos = __shfl_sync(0xffffffffu, pos, 31) + sel_base;
#pragma unroll
  for (int i = 0; i < ITEMS; ++i) {
    const unsigned sel_b = __ballot_sync(0xffffffffu, (selbits >> i) & 1u);
    if ((selbits >> i) & 1u) a.kept[pos + __popc(sel_b & lt_mask)] = base + i * 32;
    pos += __popc(sel_b);
  }
}

struct GatherArgs {
  const int4 *src_k, *src_v;
  int4 *dst_k, *dst_v;
  const int* kept;
  int vis_start, m, k, dst_len, n_layers;
  int seg0_lo, seg0_len, seg1_lo, seg1_len;   // the destination rows this launch writes: two runs, rows = their sum
  int rows;
  int row_vec;                       // 16-byte units per row
  long long src_ls_vec, dst_ls_vec;  // layer strides in 16-byte units
};

// One thread moves 16 bytes of K and 16 bytes of V per step; a destination row
// maps to its source row through the kept-index list.
__global__ void __launch_bounds__(256) uvprune_gather_kernel(const GatherArgs a) {
  const long long per_layer = (long long)a.rows * a.row_vec;
  const long long total = per_layer * a.n_layers;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x; u < total; u += stride) {
    const int layer = (int)(u / per_layer);
    const long long w = u - (long long)layer * per_layer;
    const int r = (int)(w / a.row_vec);
    const int c = (int)(w - (long long)r * a.row_vec);
    const int drow = r < a.seg0_len ? a.seg0_lo + r : a.seg1_lo + (r - a.seg0_len);
    int srow;
    if (drow < a.vis_start) srow = drow;
    else if (drow < a.vis_start + a.k) srow = a.vis_start + __ldg(a.kept + (drow - a.vis_start));
    else srow = drow - a.k + a.m;
    const long long so = (long long)layer * a.src_ls_vec + (long long)srow * a.row_vec + c;
    const long long dof = (long long)layer * a.dst_ls_vec + (long long)drow * a.row_vec + c;
    const int4 kk = __ldg(a.src_k + so);
    const int4 vv = __ldg(a.src_v + so);
    a.dst_k[dof] = kk;
    a.dst_v[dof] = vv;
  }
}

}  // namespace

size_t uvprune_workspace(const pvlm_prune_params& p) { return align_up((size_t)(p.m > 0 ? p.m : 1) * 4, 256); }

pvlm_status launch_uvprune(const pvlm_prune_params& p, cudaStream_t s) { return launch_uvprune_parts(p, true, 0, s); }

// part 0: all destination rows; 1: only the rows that do not depend on the selection (before and after the
// visual span); 2: only the selected visual rows; 3: no gather.
pvlm_status launch_uvprune_parts(const pvlm_prune_params& p, bool select, int part, cudaStream_t s) {
  SelArgs sa;
  sa.cur = p.mass_cur + p.vis_start;
  sa.ref = p.mass_ref ? p.mass_ref + p.vis_start : nullptr;
  sa.score = p.score;
  sa.keys = (uint32_t*)p.workspace;
  sa.kept = p.kept_idx;
  sa.m = p.m;
  sa.k = p.k;
  if (select && p.m > 0) {
    const bool one_cta = option_value(PVLM_OPT_SELECT_ONE_CTA) != 0;    // single-CTA kernels only: the tests' second implementation
    const dim3 cl8(8), cl16(16), one(1), th(kSelThreads);
    cudaError_t e = cudaErrorUnknown;
    bool launched = false;
    // Larger token counts go to a 16-CTA cluster (half the keys per thread).  That size is not portable, so the kernel is
    // told that it is allowed: a per-device function attribute, hence set with the launch, not once per process.
    if (!one_cta && p.m >= kWideSelectMinTokens && p.m <= 16 * kSelThreads * 16) {
      auto wide = [&](auto kernel) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
          (void)cudaGetLastError();
          return;                                           // this device will not have it: the 8-CTA kernels below
        }
        e = launch_dependent(kernel, cl16, th, 0, s, sa);
        launched = true;
      };
      if (p.m <= 16 * kSelThreads * 8) wide(uvprune_select_cluster_kernel<8, 16>);
      else wide(uvprune_select_cluster_kernel<16, 16>);
    }
    if (!launched) {
      if (!one_cta && p.m <= 8 * kSelThreads * 4) e = launch_dependent(uvprune_select_cluster_kernel<4, 8>, cl8, th, 0, s, sa);
      else if (!one_cta && p.m <= 8 * kSelThreads * 16) e = launch_dependent(uvprune_select_cluster_kernel<16, 8>, cl8, th, 0, s, sa);
      else if (!one_cta && p.m <= 8 * kSelThreads * 32) e = launch_dependent(uvprune_select_cluster_kernel<32, 8>, cl8, th, 0, s, sa);
      else if (p.m <= 32 * kSelThreads) e = launch_dependent(uvprune_select_reg_kernel<32>, one, th, 0, s, sa);
      else e = launch_dependent(uvprune_select_kernel, one, th, 0, s, sa);
    }
    if (e != cudaSuccess) set_cuda_error((int)e);
  }
  if (p.src_k && part != 3) {
    GatherArgs g;
    g.src_k = (const int4*)p.src_k;
    g.src_v = (const int4*)p.src_v;
    g.dst_k = (int4*)p.dst_k;
    g.dst_v = (int4*)p.dst_v;
    g.kept = p.kept_idx;
    g.vis_start = p.vis_start; g.m = p.m; g.k = p.k;
    g.dst_len = p.src_len - p.m + p.k;
    g.n_layers = p.n_layers;
    g.row_vec = (int)(p.row_bytes / 16);
    g.src_ls_vec = p.src_layer_stride_bytes / 16;
    g.dst_ls_vec = p.dst_layer_stride_bytes / 16;
    g.seg1_lo = g.seg1_len = 0;
    if (part == 0) { g.seg0_lo = 0; g.seg0_len = g.dst_len; }
    else if (part == 1) { g.seg0_lo = 0; g.seg0_len = p.vis_start; g.seg1_lo = p.vis_start + p.k; g.seg1_len = g.dst_len - g.seg1_lo; }
    else { g.seg0_lo = p.vis_start; g.seg0_len = p.k; }
    g.rows = g.seg0_len + g.seg1_len;
    const long long total = (long long)g.rows * g.row_vec * g.n_layers;
    if (total > 0) {
      long long blocks = (total + 255) / 256;
      // Short-lived CTAs (four K + V copies per thread) measured faster than a resident grid that loops (419 vs 440 µs on
      // the 64-layer gather), and they give SM slots back quickly when the launch runs beside another stream's kernels.
      const long long cap = (blocks + 3) / 4;
      if (blocks > cap) blocks = cap;
      uvprune_gather_kernel<<<(int)blocks, 256, 0, s>>>(g);
    }
  }
  return check_launch();
}

// ---- selection without caller-provided scratch -------------------------------------------
// The key buffer of the selection kernel, held in the library's device image so that callers
// who cannot allocate device memory can still select.  In host code this name is only a
// handle for the symbol: the kernel must be given the address cudaGetSymbolAddress returns.
static __device__ __align__(256) uint32_t g_select_static_keys[PVLM_SELECT_STATIC_MAX_M];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
uint32_t* g_static_keys_addr[kMaxDevices] = {};

// Device address of the static key buffer on the current device; looked up once per device.
pvlm_status static_keys_for_current_device(uint32_t** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) { set_cuda_error((int)e); return PVLM_ERR_CUDA; }
  if (dev < 0 || dev >= kMaxDevices) return PVLM_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_mu);
  if (!g_static_keys_addr[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_select_static_keys);
    if (e != cudaSuccess || !ptr) { set_cuda_error((int)e); return PVLM_ERR_CUDA; }
    g_static_keys_addr[dev] = static_cast<uint32_t*>(ptr);
  }
  *out = g_static_keys_addr[dev];
  return PVLM_OK;
}
}  // namespace

}  // namespace pvlm

extern "C" pvlm_status pvlm_uvprune_select_static(const float* mass_cur, const float* mass_ref, int vis_start, int m,
                                                  int k, int* kept_idx, float* score, void* stream) {
  using namespace pvlm;
  if (m < 0 || k < 0 || k > m || vis_start < 0) return PVLM_ERR_INVALID_ARG;
  if (m > PVLM_SELECT_STATIC_MAX_M) return PVLM_ERR_TOO_LARGE;
  if (m > 0 && !mass_cur) return PVLM_ERR_INVALID_ARG;
  if (k > 0 && !kept_idx) return PVLM_ERR_INVALID_ARG;
  if (m == 0) return PVLM_OK;
  uint32_t* keys = nullptr;
  const pvlm_status st = static_keys_for_current_device(&keys);
  if (st != PVLM_OK) return st;
  SelArgs sa;
  sa.cur = mass_cur + vis_start;
  sa.ref = mass_ref ? mass_ref + vis_start : nullptr;
  sa.score = score;
  sa.keys = keys;
  sa.kept = kept_idx;
  sa.m = m;
  sa.k = k;
  uvprune_select_kernel<<<1, kSelThreads, 0, (cudaStream_t)stream>>>(sa);
  return check_launch();
}
