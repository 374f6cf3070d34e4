// Token-level top-k (Eq. 3, second half) as an exact MSB-first radix select.
//
// One thread-block cluster per (sequence, query) row. The row's visible scores are cut into
// contiguous slices, one per block; each block converts its slice once to order-preserving 32-bit
// keys held in shared memory, so nothing goes back to global memory afterwards.
//
// First digit: 12 key bits (sign, exponent, three mantissa bits). fp32 scores crowd into a few
// sign/exponent patterns, so a wide first digit is what keeps the shared-memory histogram atomics
// from serialising on a handful of bins; a warp whose lanes all hit one bin adds once. The
// histogram is built in the same sweep that loads the scores. Each block adds its non-empty bins
// into every block's copy of the row histogram with distributed-shared-memory atomics; after one
// cluster barrier every block scans its own copy from the top bin down and finds, redundantly and
// identically, the bin that contains the k-th largest key.
//
// Remaining 20 bits, common case: that bin holds few keys (a fraction of a percent of the row). A
// second sweep counts, per warp, the keys above the bin and collects the keys inside it
// ("candidates") with their positions; the blocks read each other's short candidate lists through
// distributed shared memory and each finishes the select locally with two 10-bit passes over the
// candidates only. Rare case (more than kCandCap keys share the first 12 bits, e.g. long runs of
// equal scores): two more full radix passes (12 + 8 bits) with the same cluster-wide histograms.
//
// Either way the exact threshold key and the number of threshold-equal keys still needed are
// known, and a block's output offset is the number of selected keys in lower-ranked blocks. Common
// case: the ballots of the second sweep (keys above the threshold's bin) were kept as a position
// bitmap of the slice; the selected candidates add their bits, and a prefix count over the bitmap
// words writes the positions in ascending order -- no third sweep over the keys. Rare case: an
// index-ordered compaction sweep (a warp's offset is the number selected in lower warps). In both,
// among keys equal to the threshold the lowest positions win.
// No atomics touch global memory and nothing spins.
//
// Launches with more rows than clusters that are resident at once (a prefill chunk's thousands of
// rows, but also a decode batch of 34 or more 128K-token sequences) first go through the one-sweep
// kernel in topk_filter.cu, if the shape fits it; this kernel then runs once more, one block per 16
// rows, for the rows that kernel marked as unfinished (count = -1).
#include <cooperative_groups.h>

#include <mutex>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace clsa {
namespace {

// 1024 threads per block for latency hiding (the sweeps are chains of votes and shared-memory atomics), clusters
// of 1 to 8 blocks: 8 for launches of up to 8 rows, 6 for up to 22, 4 beyond -- as many as are all resident at once
// (a block fills an SM; a B200 holds 33 clusters of 4 and 22 of 6, but only 15 of 7, 8 or 9).
constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxBins = 4096;
constexpr int kMaxCluster = 8;       // the largest cluster make_topk_plan chooses
constexpr int kCandCap = 2048;  // candidates (row-wide) the short path handles

struct alignas(16) Shared {  // the keys follow it in shared memory and are written 16 bytes at a time
  uint32_t local_hist[kMaxBins];       // this block's slice; later: gathered candidates + 1024-bin histogram
  uint32_t cluster_hist[2][kMaxBins];  // whole row, one copy per block; [1] later: this block's candidate list
  uint32_t warp_tot[kWarps];
  uint32_t warp_gt[kWarps], warp_eq[kWarps];
  uint32_t block_gt_eq[2];             // read remotely (long path)
  uint32_t cand_count;                 // read remotely
  uint32_t block_gt0;                  // keys of this block above the threshold's 12-bit bin; read remotely
  uint32_t rank_gt[kMaxCluster], rank_eq[kMaxCluster];  // per block of the cluster: candidates above / equal to the threshold
  uint32_t digit, k_rem, bin_count;
  uint32_t out_base, eq_base;
  uint32_t eq_n, use_bitmap, pad_[2];
};

// Split cluster barrier: arrive early, wait late, so the barrier's latency hides behind independent work.
static_assert(kWarps == 32, "lane l reads warp l's total");
static_assert(sizeof(Shared) % 16 == 0, "the key array behind Shared must stay 16-byte aligned");

__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t score_key(float x) {
  uint32_t u = __float_as_uint(x);
  if (u == 0x80000000u) u = 0u;  // -0.0 ranks equal to +0.0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Adds one to hist[bin] for every lane with `in`; a warp whose voters all share one bin adds once.
__device__ __forceinline__ void hist_add(uint32_t* hist, bool in, uint32_t bin, int lane) {
  // one vote decides whether the whole warp agrees on one bin
  int same = 0;
  const uint32_t voters = __match_all_sync(0xffffffffu, in ? bin : 0xffffffffu, &same);
  (void)voters;
  if (same) {
    if (in && lane == 0) atomicAdd(&hist[bin], 32u);
  } else if (in) {
    atomicAdd(&hist[bin], 1u);
  }
}

// Block-wide scan of hist[0..NB) from the top bin down: finds the bin in which the running count
// reaches k_rem. On return (after a __syncthreads) sh.digit is that bin, sh.k_rem what is still
// needed inside it, sh.bin_count its population. If `clear`, the histogram is zeroed on the way.
template <int NB>
__device__ __forceinline__ void scan_from_top(Shared& sh, uint32_t* hist, uint32_t k_rem, bool clear) {
  constexpr int PT = (NB + kThreads - 1) / kThreads;  // bins per thread
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t own[PT];
  uint32_t tot = 0;
#pragma unroll
  for (int j = 0; j < PT; ++j) {
    const int pos = tid * PT + j;  // thread t owns bins NB-1-(t*PT+j)
    own[j] = pos < NB ? hist[NB - 1 - pos] : 0u;
    tot += own[j];
  }
  uint32_t incl = tot;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t up = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += up;
  }
  if (lane == 31) sh.warp_tot[warp] = incl;
  __syncthreads();
  uint32_t before = 0;
  for (int w = 0; w < warp; ++w) before += sh.warp_tot[w];
  incl += before;
  const uint32_t excl = incl - tot;
  if (excl < k_rem && k_rem <= incl) {
    uint32_t acc = excl;
#pragma unroll
    for (int j = 0; j < PT; ++j) {
      if (acc < k_rem && k_rem <= acc + own[j]) {
        sh.digit = (uint32_t)(NB - 1 - (tid * PT + j));
        sh.k_rem = k_rem - acc;
        sh.bin_count = own[j];
      }
      acc += own[j];
    }
  }
  if (clear) {
#pragma unroll
    for (int j = 0; j < PT; ++j) {
      const int pos = tid * PT + j;
      if (pos < NB) hist[NB - 1 - pos] = 0u;
    }
  }
  __syncthreads();
}

// Adds this block's non-empty local bins into every block's copy `buf` of the row histogram.
template <int NB>
__device__ __forceinline__ void push_hist(Shared& sh, cg::cluster_group& cluster, int nblk, int buf) {
  uint32_t* mine = sh.cluster_hist[buf];
  for (int bin = threadIdx.x; bin < NB; bin += kThreads) {
    const uint32_t v = sh.local_hist[bin];
    if (v != 0u)
      for (int r = 0; r < nblk; ++r) atomicAdd(cluster.map_shared_rank(mine, r) + bin, v);
  }
}

// One full radix pass over `BITS` key bits at `shift` (used by the rare long path).
template <int BITS, typename KeyAt>
__device__ __forceinline__ void radix_pass(Shared& sh, cg::cluster_group& cluster, int nblk, int cnt, int shift, int buf,
                                           uint32_t& prefix, uint32_t& prefix_mask, uint32_t& k_rem, KeyAt key_at) {
  constexpr int NB = 1 << BITS;
  const int tid = threadIdx.x, lane = tid & 31;
  for (int i = tid; i < NB; i += kThreads) sh.local_hist[i] = 0;
  __syncthreads();
  for (int i0 = 0; i0 < cnt; i0 += kThreads) {
    const int i = i0 + tid;
    const uint32_t key = i < cnt ? key_at(i) : 0u;
    hist_add(sh.local_hist, i < cnt && (key & prefix_mask) == prefix, (key >> shift) & (uint32_t)(NB - 1), lane);
  }
  __syncthreads();
  push_hist<NB>(sh, cluster, nblk, buf);
  cluster.sync();
  scan_from_top<NB>(sh, sh.cluster_hist[buf], k_rem, true);
  prefix |= sh.digit << shift;
  prefix_mask |= (uint32_t)(NB - 1) << shift;
  k_rem = sh.k_rem;
}

// One (sequence, query) row, by the calling cluster (one block when the cluster has one).
// `row`: the (sequence, query) row whose lengths apply and whose index is written; `score_row`: the row of `scores`
// that holds its scores (the same, except for rows that another route handed back into a scratch matrix).
template <bool CACHED>
__device__ __forceinline__ void topk_row(const int row, const int score_row, const float* __restrict__ scores, int64_t score_stride,
                                         const int32_t* __restrict__ seq_len, int q_per_seq, int causal, int top_k,
                                         int max_seq_len, int32_t* __restrict__ idx_out, int32_t* __restrict__ count_out,
                                         uint32_t* status, unsigned char* smem_raw) {
  Shared& sh = *reinterpret_cast<Shared*>(smem_raw);
  uint32_t* keys = reinterpret_cast<uint32_t*>(smem_raw + sizeof(Shared));

  cg::cluster_group cluster = cg::this_cluster();
  const int nblk = (int)cluster.num_blocks();
  const int rank = (int)cluster.block_rank();
  const int b = row / q_per_seq, t = row % q_per_seq;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  // Shared-memory state first: it needs nothing from global memory, so it is cleared while the kernel that
  // produces the scores may still be running (programmatic dependent launch); only then wait for that kernel.
  for (int i = tid; i < kMaxBins; i += kThreads) { sh.local_hist[i] = 0; sh.cluster_hist[0][i] = 0; }
  if (tid < kMaxCluster) { sh.rank_gt[tid] = 0; sh.rank_eq[tid] = 0; }
  if (tid == 0) { sh.cand_count = 0; sh.block_gt0 = 0; }
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // Everything up to the first cluster.sync() is uniform over the cluster (same row, same lengths).
  const int n = seq_len[b];
  int v = causal ? n - q_per_seq + t + 1 : n;
  if (n < q_per_seq || n > max_seq_len) {
    v = 0;
    if (tid == 0 && rank == 0) flag_status(status, CLSA_DEV_BAD_SEQLEN);
  }
  const int kk = min(top_k, v);
  int32_t* out = idx_out + (int64_t)row * top_k;
  if (rank == 0) {
    if (tid == 0) count_out[row] = kk;
    for (int i = kk + tid; i < top_k; i += kThreads) out[i] = -1;
  }
  const int per = ((v + nblk - 1) / nblk + 3) & ~3;  // slice length, a multiple of 4 so slices keep their 16-byte phase
  const int lo = min(v, rank * per), hi = min(v, lo + per);
  const int cnt = hi - lo;
  if (kk == v) {  // nothing to select: every visible position is taken, in order
    for (int i = tid; i < cnt; i += kThreads) out[lo + i] = lo + i;
    return;
  }
  const float* src = scores + (int64_t)score_row * score_stride + lo;
  auto key_at = [&](int i) -> uint32_t { return CACHED ? keys[i] : score_key(src[i]); };

  __syncthreads();
  // Remote adds may land in this block's histogram copy only after it has been cleared: every block arrives
  // here and waits just before it starts adding, with the whole first sweep in between.
  cluster_arrive();

  // ---- sweep 1: scores -> keys (kept in shared memory) and the 12-bit histogram of this slice --------
  if (CACHED && (reinterpret_cast<uintptr_t>(src) & 15u) == 0) {
    const float4* src4 = reinterpret_cast<const float4*>(src);
    const int n4 = cnt >> 2;
    constexpr int kBatch = 8;  // 16-byte loads a thread issues before it touches the first of them
    for (int i0 = 0; i0 < n4; i0 += kThreads * kBatch) {
      float4 f[kBatch];
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        const int i = i0 + u * kThreads + tid;
        f[u] = i < n4 ? src4[i] : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        const int i = i0 + u * kThreads + tid;
        const bool in = i < n4;
        const uint32_t k0 = score_key(f[u].x), k1 = score_key(f[u].y), k2 = score_key(f[u].z), k3 = score_key(f[u].w);
        if (in) *reinterpret_cast<uint4*>(keys + 4 * i) = make_uint4(k0, k1, k2, k3);
        if (__any_sync(0xffffffffu, in)) {
          hist_add(sh.local_hist, in, k0 >> 20, lane);
          hist_add(sh.local_hist, in, k1 >> 20, lane);
          hist_add(sh.local_hist, in, k2 >> 20, lane);
          hist_add(sh.local_hist, in, k3 >> 20, lane);
        }
      }
    }
    for (int i0 = n4 * 4; i0 < cnt; i0 += 32) {  // up to three leftover scores, handled by warp 0
      if (warp == 0) {
        const int i = i0 + lane;
        const uint32_t key = i < cnt ? score_key(src[i]) : 0u;
        if (i < cnt) keys[i] = key;
        hist_add(sh.local_hist, i < cnt, key >> 20, lane);
      }
    }
  } else {
    constexpr int kBatch = 8;
    for (int i0 = 0; i0 < cnt; i0 += kThreads * kBatch) {
      float f[kBatch];
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        const int i = i0 + u * kThreads + tid;
        f[u] = i < cnt ? src[i] : 0.f;
      }
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        const int i = i0 + u * kThreads + tid;
        const uint32_t key = score_key(f[u]);
        if (CACHED && i < cnt) keys[i] = key;
        hist_add(sh.local_hist, i < cnt, key >> 20, lane);
      }
    }
  }
  __syncthreads();   // this block's histogram is complete
  cluster_wait();    // every block has cleared its copy of the row histogram
  push_hist<4096>(sh, cluster, nblk, 0);
  cluster.sync();
  scan_from_top<4096>(sh, sh.cluster_hist[0], (uint32_t)kk, true);
  const uint32_t digit0 = sh.digit;
  uint32_t k_rem = sh.k_rem;
  const uint32_t in_bin = sh.bin_count;  // keys of the whole row that share the threshold's first 12 bits

  const int chunk = ((cnt + kWarps - 1) / kWarps + 31) & ~31;  // contiguous positions per warp in the ordered sweeps
  const int c_lo = min(cnt, warp * chunk), c_hi = min(cnt, c_lo + chunk);
  uint32_t thr, need_eq;

  // Short path only: selected positions of this slice as a bitmap (the first histogram copy is free again after
  // its scan cleared it), so that the last step is a prefix count over at most 4096 words instead of a third
  // sweep over the keys.
  uint32_t* bitmap = sh.cluster_hist[0];
  const bool use_bitmap = in_bin <= (uint32_t)kCandCap && cnt <= kMaxBins * 32;
  bool emitted = false;
  if (in_bin <= (uint32_t)kCandCap) {
    // ---- short path: sweep 2 counts keys above the bin per warp and collects the bin's keys ----------
    uint2* cand = reinterpret_cast<uint2*>(sh.cluster_hist[1]);  // (key, slice position), unordered
    uint32_t gt = 0;
    if (CACHED && use_bitmap) {
      // One thread per bitmap word: it reads its 32 consecutive keys as eight 16-byte chunks (in an order rotated by
      // its lane, so that the eight lanes of a quarter warp hit eight different bank groups), builds the word with
      // bit operations instead of one ballot per 32 keys, and then appends the few keys of the threshold's bin.
      const int words = (cnt + 31) >> 5;
      for (int w = tid; w < words; w += kThreads) {
        uint32_t above = 0, inbin = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int c = (j + lane) & 7;
          const int i = 32 * w + 4 * c;
          if (i < cnt) {  // the slice buffer is padded to a multiple of 4 keys
            const uint4 k4 = *reinterpret_cast<const uint4*>(keys + i);
            const uint32_t t0 = k4.x >> 20, t1 = k4.y >> 20, t2 = k4.z >> 20, t3 = k4.w >> 20;
            const uint32_t a4 = (t0 > digit0 ? 1u : 0u) | (t1 > digit0 ? 2u : 0u) | (t2 > digit0 ? 4u : 0u) | (t3 > digit0 ? 8u : 0u);
            const uint32_t e4 = (t0 == digit0 ? 1u : 0u) | (t1 == digit0 ? 2u : 0u) | (t2 == digit0 ? 4u : 0u) | (t3 == digit0 ? 8u : 0u);
            above |= a4 << (4 * c);
            inbin |= e4 << (4 * c);
          }
        }
        const int left = cnt - 32 * w;  // >= 1
        if (left < 32) {
          const uint32_t valid = (1u << left) - 1u;
          above &= valid;
          inbin &= valid;
        }
        bitmap[w] = above;
        gt += (uint32_t)__popc(above);
        while (inbin != 0u) {
          const int i = 32 * w + __ffs(inbin) - 1;
          inbin &= inbin - 1u;
          cand[atomicAdd(&sh.cand_count, 1u)] = make_uint2(keys[i], (uint32_t)i);
        }
      }
#pragma unroll
      for (int d = 16; d >= 1; d >>= 1) gt += __shfl_xor_sync(0xffffffffu, gt, d);
    } else
    for (int i0 = c_lo; i0 < c_hi; i0 += 128) {
      uint32_t key[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + 32 * u + lane;
        key[u] = i < c_hi ? key_at(i) : 0u;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int i = i0 + 32 * u + lane;
        const uint32_t top = key[u] >> 20;
        // keys above the threshold's bin are certainly selected: their ballot is the position bitmap's word
        const uint32_t gtb = __ballot_sync(0xffffffffu, i < c_hi && top > digit0);
        if (use_bitmap && lane == 0 && i0 + 32 * u < c_hi) bitmap[(i0 + 32 * u) >> 5] = gtb;
        gt += (uint32_t)__popc(gtb);  // the same on every lane
        const bool is_c = i < c_hi && top == digit0;
        const uint32_t cb = __ballot_sync(0xffffffffu, is_c);
        if (cb != 0u) {
          uint32_t base = 0;
          if (lane == 0) base = atomicAdd(&sh.cand_count, (uint32_t)__popc(cb));
          base = __shfl_sync(0xffffffffu, base, 0);
          if (is_c) cand[base + __popc(cb & ((1u << lane) - 1u))] = make_uint2(key[u], (uint32_t)i);
        }
      }
    }
    if (lane == 0) { sh.warp_gt[warp] = gt; sh.warp_eq[warp] = 0; atomicAdd(&sh.block_gt0, gt); }
    cluster.sync();  // every block's candidate list, candidate count and above-the-bin count are complete
    // gather the row's candidates (keys only) into local_hist[0..in_bin)
    uint32_t* allc = sh.local_hist;
    uint32_t* hist10 = sh.local_hist + kCandCap;  // 1024 bins
    uint32_t start[kMaxCluster];  // first flat index of each block's candidates (all lanes hold all of them)
    uint32_t gt0_of_lane = 0;     // lane r: keys of block r above the bin
    {
      // lane r of every warp reads block r's counts; an exclusive scan gives the blocks' offsets
      const uint32_t nr = lane < nblk ? *cluster.map_shared_rank(&sh.cand_count, lane) : 0u;
      gt0_of_lane = lane < nblk ? *cluster.map_shared_rank(&sh.block_gt0, lane) : 0u;
      uint32_t incl = nr;
#pragma unroll
      for (int d = 1; d < kMaxCluster; d <<= 1) {
        const uint32_t up = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += up;
      }
      const uint32_t excl = incl - nr;
#pragma unroll
      for (int q = 0; q < kMaxCluster; ++q) start[q] = q < nblk ? __shfl_sync(0xffffffffu, excl, q) : 0xffffffffu;
      for (uint32_t i = tid; i < in_bin; i += kThreads) {
        int r = 0;
        uint32_t off = 0;
#pragma unroll
        for (int q = 1; q < kMaxCluster; ++q)
          if (i >= start[q]) { r = q; off = start[q]; }
        const uint2* rc = reinterpret_cast<const uint2*>(cluster.map_shared_rank(&sh.cluster_hist[1][0], r));
        allc[i] = rc[i - off].x;
      }
    }
    for (int i = tid; i < 1024; i += kThreads) hist10[i] = 0;
    __syncthreads();
    // This block reads nobody's shared memory from here on: arrive now on the barrier that keeps every block
    // alive until its neighbours are done with it, and wait on it only at the very end.
    cluster_arrive();
    // two local 10-bit passes over the candidates: bits 19..10, then 9..0
    uint32_t prefix = digit0 << 20, prefix_mask = 0xfff00000u;
#pragma unroll 1
    for (int pass = 0; pass < 2; ++pass) {
      const int shift = 10 - 10 * pass;
      for (uint32_t i0 = 0; i0 < in_bin; i0 += kThreads) {
        const uint32_t i = i0 + tid;
        const uint32_t key = i < in_bin ? allc[i] : 0u;
        hist_add(hist10, i < in_bin && (key & prefix_mask) == prefix, (key >> shift) & 1023u, lane);
      }
      __syncthreads();
      scan_from_top<1024>(sh, hist10, k_rem, true);
      prefix |= sh.digit << shift;
      prefix_mask |= 1023u << shift;
      k_rem = sh.k_rem;
    }
    thr = prefix;
    need_eq = k_rem;
    // per-warp counts of this block: keys above the bin (already counted) plus candidates above / equal to thr
    const uint32_t my_n = sh.cand_count;
    if (!use_bitmap) {  // only the ordered sweep at the end needs them
      for (uint32_t i = tid; i < my_n; i += kThreads) {
        const uint2 c = cand[i];
        const int w = (int)c.y / chunk;
        if (c.x > thr) atomicAdd(&sh.warp_gt[w], 1u);
        else if (c.x == thr) atomicAdd(&sh.warp_eq[w], 1u);
      }
    }
    // the same two counts for every block of the cluster, from the gathered candidates (grouped by block):
    // with them each block derives its output offset alone, without another exchange
    for (uint32_t i = tid; i < in_bin; i += kThreads) {
      int r = 0;
#pragma unroll
      for (int q = 1; q < kMaxCluster; ++q)
        if (i >= start[q]) r = q;
      const uint32_t key = allc[i];
      if (key > thr) atomicAdd(&sh.rank_gt[r], 1u);
      else if (key == thr) atomicAdd(&sh.rank_eq[r], 1u);
    }
    __syncthreads();
    if (warp == 0) {
      // lane r holds the totals of block r; the offset of this block is a prefix over the lower-ranked ones
      const uint32_t g = lane < nblk ? gt0_of_lane + sh.rank_gt[lane] : 0u;
      const uint32_t e = lane < nblk ? sh.rank_eq[lane] : 0u;
      uint32_t eq_before = 0, sel_before = 0;
      for (int r = 0; r < rank; ++r) {
        const uint32_t gr = __shfl_sync(0xffffffffu, g, r), er = __shfl_sync(0xffffffffu, e, r);
        const uint32_t take = eq_before >= need_eq ? 0u : min(er, need_eq - eq_before);
        sel_before += gr + take;
        eq_before += er;
      }
      if (lane == 0) { sh.out_base = sel_before; sh.eq_base = eq_before; sh.eq_n = 0u; }
    }
    __syncthreads();
    if (use_bitmap) {
      // threshold-equal candidates of this block that are taken: the lowest positions, after those of lower blocks
      const uint32_t my_eq = sh.rank_eq[rank];
      const uint32_t quota = sh.eq_base >= need_eq ? 0u : min(my_eq, need_eq - sh.eq_base);
      uint32_t* eq_pos = sh.local_hist;  // the gathered candidates and their histogram are dead by now
      const bool partial = quota != 0u && quota != my_eq;  // my_eq <= kCandCap entries: they fit eq_pos
      {
        for (uint32_t i = tid; i < my_n; i += kThreads) {
          const uint2 c = cand[i];
          if (c.x > thr || (c.x == thr && quota == my_eq)) atomicOr(&bitmap[c.y >> 5], 1u << (c.y & 31u));
          else if (c.x == thr && partial) eq_pos[atomicAdd(&sh.eq_n, 1u)] = c.y;
        }
        __syncthreads();
        if (partial) {
          for (uint32_t i = tid; i < my_eq; i += kThreads) {
            const uint32_t mine = eq_pos[i];
            uint32_t lower = 0;
            for (uint32_t j = 0; j < my_eq; ++j) lower += eq_pos[j] < mine;
            if (lower < quota) atomicOr(&bitmap[mine >> 5], 1u << (mine & 31u));
          }
          __syncthreads();
        }
        // prefix count over the bitmap words, then every thread writes the positions of its own words
        const int words = (cnt + 31) >> 5;
        const int wpt = (words + kThreads - 1) / kThreads;
        const int w_lo = min(words, tid * wpt), w_hi = min(words, w_lo + wpt);
        uint32_t mine = 0;
        for (int w = w_lo; w < w_hi; ++w) mine += __popc(bitmap[w]);
        uint32_t incl = mine;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const uint32_t up = __shfl_up_sync(0xffffffffu, incl, d);
          if (lane >= d) incl += up;
        }
        if (lane == 31) sh.warp_tot[warp] = incl;
        __syncthreads();
        uint32_t tot = sh.warp_tot[lane];  // kWarps == 32: lane l holds warp l's total
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const uint32_t up = __shfl_up_sync(0xffffffffu, tot, d);
          if (lane >= d) tot += up;
        }
        const uint32_t below = __shfl_sync(0xffffffffu, tot, (warp + 31) & 31);
        uint32_t off = sh.out_base + (warp == 0 ? 0u : below) + incl - mine;
        for (int w = w_lo; w < w_hi; ++w) {
          uint32_t bits = bitmap[w];
          while (bits != 0u) {
            if (off < (uint32_t)kk) out[off] = lo + w * 32 + __ffs(bits) - 1;
            ++off;
            bits &= bits - 1u;
          }
        }
        emitted = true;
      }
    }
  } else {
    // ---- long path: two more cluster-wide radix passes, then a counting sweep ------------------------
    uint32_t prefix = digit0 << 20, prefix_mask = 0xfff00000u;
    for (int i = tid; i < kMaxBins; i += kThreads) sh.cluster_hist[1][i] = 0;
    cluster.sync();  // every block's second histogram copy is clear before anybody adds into it
    radix_pass<12>(sh, cluster, nblk, cnt, 8, 1, prefix, prefix_mask, k_rem, key_at);
    radix_pass<8>(sh, cluster, nblk, cnt, 0, 0, prefix, prefix_mask, k_rem, key_at);
    thr = prefix;
    need_eq = k_rem;
    uint32_t gt = 0, eq = 0;
    for (int i = c_lo + lane; i < c_hi; i += 32) {
      const uint32_t key = key_at(i);
      gt += key > thr;
      eq += key == thr;
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
      gt += __shfl_xor_sync(0xffffffffu, gt, d);
      eq += __shfl_xor_sync(0xffffffffu, eq, d);
    }
    if (lane == 0) { sh.warp_gt[warp] = gt; sh.warp_eq[warp] = eq; }
    __syncthreads();
    if (warp == 0) {
      uint32_t g = lane < kWarps ? sh.warp_gt[lane] : 0u, e = lane < kWarps ? sh.warp_eq[lane] : 0u;
#pragma unroll
      for (int d = 16; d >= 1; d >>= 1) {
        g += __shfl_xor_sync(0xffffffffu, g, d);
        e += __shfl_xor_sync(0xffffffffu, e, d);
      }
      if (lane == 0) { sh.block_gt_eq[0] = g; sh.block_gt_eq[1] = e; }
    }
    cluster.sync();
    if (tid == 0) {
      uint32_t eq_before = 0, sel_before = 0;
      for (int r = 0; r < rank; ++r) {
        const uint32_t* ge = cluster.map_shared_rank(sh.block_gt_eq, r);
        const uint32_t g = ge[0], e = ge[1];
        const uint32_t take = eq_before >= need_eq ? 0u : min(e, need_eq - eq_before);
        sel_before += g + take;
        eq_before += e;
      }
      sh.out_base = sel_before;
      sh.eq_base = eq_before;
    }
    __syncthreads();
    cluster_arrive();  // pairs with the wait at the very end
  }

  if (emitted) {
    cluster_wait();  // no block may exit while a neighbour can still read its shared memory (arrived earlier)
    return;
  }
  // ---- index-ordered compaction (long path, and short-path slices the bitmap route does not take) ------------
  // offsets of this warp: selected / threshold-equal keys in lower warps of this block
  uint32_t out_pos = sh.out_base, eq_rank = sh.eq_base;
  for (int w = 0; w < warp; ++w) {
    const uint32_t e = sh.warp_eq[w];
    const uint32_t take = eq_rank >= need_eq ? 0u : min(e, need_eq - eq_rank);
    out_pos += sh.warp_gt[w] + take;
    eq_rank += e;
  }
  const uint32_t lt_mask = (1u << lane) - 1u;
  for (int i0 = c_lo; i0 < c_hi; i0 += 128) {
    uint32_t key[4], eq_ballot[4], gt_ballot[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + 32 * u + lane;
      key[u] = i < c_hi ? key_at(i) : 0u;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + 32 * u + lane;
      gt_ballot[u] = __ballot_sync(0xffffffffu, i < c_hi && key[u] > thr);
      eq_ballot[u] = __ballot_sync(0xffffffffu, i < c_hi && key[u] == thr);
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int i = i0 + 32 * u + lane;
      const bool is_gt = (gt_ballot[u] >> lane) & 1u, is_eq = (eq_ballot[u] >> lane) & 1u;
      // threshold-equal keys are taken in position order until need_eq of them are in
      const bool take = is_gt || (is_eq && eq_rank + __popc(eq_ballot[u] & lt_mask) < need_eq);
      const uint32_t take_ballot = __ballot_sync(0xffffffffu, take);
      if (take) {
        const uint32_t pos = out_pos + __popc(take_ballot & lt_mask);
        if (pos < (uint32_t)kk) out[pos] = lo + i;
      }
      out_pos += __popc(take_ballot);
      eq_rank += __popc(eq_ballot[u]);
    }
  }
  cluster_wait();  // no block may exit while a neighbour can still read its shared memory (arrived earlier)
}

constexpr int kPendingRowsPerBlock = 16;  // rows a block of the pending-only launch looks after (all pending: still >= 148 blocks for 2400 rows)

template <bool CACHED>
__global__ void __launch_bounds__(kThreads, 1)
topk_radix_kernel(const float* __restrict__ scores, int64_t score_stride, const int32_t* __restrict__ seq_len,
                  int q_per_seq, int causal, int top_k, int max_seq_len, int pending_rows,
                  int32_t* __restrict__ idx_out, int32_t* __restrict__ count_out, uint32_t* status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  // Programmatic dependent launch: this grid may have been scheduled before the kernel that writes the scores
  // has finished. The kernel after this one may be scheduled early in turn (it waits for this grid itself);
  // this grid's own wait sits in topk_row, after the shared-memory clears and before the first global access.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (pending_rows == 0) {
    const int nblk = (int)cg::this_cluster().num_blocks();
    topk_row<CACHED>(blockIdx.x / nblk, blockIdx.x / nblk, scores, score_stride, seq_len, q_per_seq, causal, top_k, max_seq_len, idx_out,
                     count_out, status, smem_raw);
    return;
  }
  // Second kernel of the many-rows route (one block per kPendingRowsPerBlock rows, no clusters): the one-sweep
  // kernel before this one has done every row it could and left count = -1 on the others. All marks of this
  // block's rows are read in one round trip; the usual outcome is that none is set.
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the marks come from the kernel just before this one
  __shared__ int pending[kPendingRowsPerBlock];
  const int first = blockIdx.x * kPendingRowsPerBlock;
  int mine = 0;
  if (threadIdx.x < kPendingRowsPerBlock) {
    const int row = first + threadIdx.x;
    mine = (row < pending_rows && count_out[row] == -1) ? 1 : 0;
    pending[threadIdx.x] = mine;
  }
  if (__syncthreads_or(mine) == 0) return;
  for (int j = 0; j < kPendingRowsPerBlock; ++j) {
    if (pending[j]) {
      topk_row<CACHED>(first + j, first + j, scores, score_stride, seq_len, q_per_seq, causal, top_k, max_seq_len, idx_out,
                       count_out, status, smem_raw);
      __syncthreads();  // the next row reuses this block's shared memory
    }
  }
}

// Rows that the fused chunk routing handed back: block j takes the row listed in slot j, whose scores are row j of the
// scratch matrix (no clusters; usually there is no such row and the block returns at once). A kernel of its own, so
// that the decode kernel above is compiled exactly as it is without this route.
template <bool CACHED>
__global__ void __launch_bounds__(kThreads, 1)
topk_radix_slots_kernel(const float* __restrict__ scores, int64_t score_stride, const int32_t* __restrict__ seq_len,
                        int q_per_seq, int causal, int top_k, int max_seq_len,
                        const int32_t* __restrict__ row_of_slot, const uint32_t* __restrict__ nslots,
                        int32_t* __restrict__ idx_out, int32_t* __restrict__ count_out, uint32_t* status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (blockIdx.x >= *nslots) return;
  topk_row<CACHED>(row_of_slot[blockIdx.x], (int)blockIdx.x, scores, score_stride, seq_len, q_per_seq, causal, top_k,
                   max_seq_len, idx_out, count_out, status, smem_raw);
}

}  // namespace

// Clusters of `cluster` blocks with `smem_bytes` of dynamic shared memory that are resident at once on the current
// device (cached; a failed query falls back to one block per SM).
static int resident_clusters(int cluster, size_t smem_bytes, bool cached, const DeviceInfo& dev) {
  struct Entry { int dev, cluster, cached; size_t smem; int n; };
  static std::mutex mu;
  static Entry seen[16];
  static int used = 0;
  int d = 0;
  if (cudaGetDevice(&d) != cudaSuccess) { cudaGetLastError(); return dev.sm_count / cluster; }
  std::lock_guard<std::mutex> lock(mu);
  for (int i = 0; i < used; ++i)
    if (seen[i].dev == d && seen[i].cluster == cluster && seen[i].cached == (int)cached && seen[i].smem == smem_bytes) return seen[i].n;
  auto kernel = cached ? topk_radix_kernel<true> : topk_radix_kernel<false>;
  int n = 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)cluster * 64, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem_bytes;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)cluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes) != cudaSuccess ||
      cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess || n <= 0) {
    cudaGetLastError();
    n = dev.sm_count / cluster;
  }
  if (used < 16) seen[used++] = Entry{d, cluster, (int)cached, smem_bytes, n};
  return n;
}

// Shared memory of a block whose slice of the row is `per` scores: the keys are kept there whenever they fit,
// even if that leaves one block per SM and several waves (two waves of one block per SM beat one wave of two blocks
// per SM that re-read their slices from L2 in every sweep).
static void size_blocks(TopkPlan& plan, int max_seq_len, const DeviceInfo& dev) {
  const int per = (((max_seq_len + plan.cluster - 1) / plan.cluster) + 3) & ~3;
  const size_t want = sizeof(Shared) + (size_t)per * sizeof(uint32_t);
  if (want <= (size_t)dev.max_smem_optin) {
    plan.slice_cap = per;
    plan.smem_bytes = want;
  } else {
    plan.slice_cap = 0;  // slice too long for shared memory: keys are recomputed from global memory in every sweep
    plan.smem_bytes = sizeof(Shared);
  }
}

TopkPlan make_topk_plan(const clsa_params& p, const DeviceInfo& dev, bool one_sweep_fits) {
  TopkPlan plan;
  // One block per 32K visible scores, capped at kMaxCluster and rounded to a power of two; when there are few
  // rows, spread each over more blocks (down to 2K scores per block).
  int c = (p.max_seq_len + 32767) / 32768;
  if (c > 4) c = 4;
  int pow2 = 1;
  while (pow2 < c) pow2 <<= 1;
  const int64_t rows = (int64_t)p.num_seqs * p.q_per_seq;
  while (pow2 < 4 && rows * pow2 * 2 <= dev.sm_count && p.max_seq_len / (pow2 * 2) >= 2048) pow2 <<= 1;
  // a handful of rows (small-batch decoding): clusters of 8, all of which are resident at once up to 8 rows
  if (pow2 == 4 && rows <= 8 && p.max_seq_len / 8 >= 2048) pow2 = 8;
  plan.cluster = pow2;
  plan.one_sweep = 0;
  size_blocks(plan, p.max_seq_len, dev);
  // In between (9 to about 22 rows): clusters of 6, if they are all resident at once (22 of them on a B200, against
  // 15 of 7, 8 or 9) -- a third fewer scores per thread in the two sweeps.
  if (pow2 == 4 && rows > 8 && p.max_seq_len / 6 >= 2048) {
    TopkPlan six = plan;
    six.cluster = 6;
    size_blocks(six, p.max_seq_len, dev);
    if (six.slice_cap > 0 && rows <= resident_clusters(6, six.smem_bytes, true, dev)) plan = six;
  }
  // Many rows. Far more rows than SMs (a prefill chunk): throughput matters, not the latency of one row; one block
  // per row needs no cluster barriers and keeps more rows in flight. And whenever the clusters of this launch would
  // not all be resident at once, the one-sweep kernel (one block per row, two blocks per SM, one pass over the
  // scores) is faster than a second wave of clusters, if the shape fits it (as fast at the largest launch that one
  // wave of clusters still holds, and several times faster at a few hundred rows).
  bool many = rows >= 4 * (int64_t)dev.sm_count;
  if (!many && one_sweep_fits && rows > resident_clusters(plan.cluster, plan.smem_bytes, plan.slice_cap > 0, dev)) many = true;
  if (many) {
    plan.cluster = 1;
    plan.one_sweep = one_sweep_fits ? 1 : 0;
    size_blocks(plan, p.max_seq_len, dev);
  }
  return plan;
}

cudaError_t launch_topk(const clsa_params& p, const float* scores, int64_t score_stride, int32_t* idx, int32_t* count,
                        uint32_t* status, const DeviceInfo& dev, cudaStream_t stream) {
  const TopkPlan plan = make_topk_plan(p, dev, topk_prefilter_fits(p, scores, score_stride, dev));
  const int64_t rows = (int64_t)p.num_seqs * p.q_per_seq;
  // Many rows: a one-sweep kernel takes every row it can finish exactly and marks the rest; the general kernel
  // below then runs for the marked rows only.
  const int pending_only = plan.one_sweep;
  if (pending_only) {
    const cudaError_t pre = launch_topk_prefilter(p, scores, score_stride, idx, count, status, dev, stream);
    if (pre != cudaSuccess) return pre;
  }
  const int pending_rows = pending_only ? (int)rows : 0;
  const int64_t blocks = pending_only ? (rows + kPendingRowsPerBlock - 1) / kPendingRowsPerBlock : rows * plan.cluster;
  auto kernel = plan.slice_cap > 0 ? topk_radix_kernel<true> : topk_radix_kernel<false>;
  cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem_bytes);
  if (err != cudaSuccess) return err;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)blocks, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = plan.smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)plan.cluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, kernel, scores, score_stride, p.seq_len, (int)p.q_per_seq, (int)p.causal,
                            (int)p.top_k, (int)p.max_seq_len, pending_rows, idx, count, status);
}

cudaError_t launch_topk_slots(const clsa_params& p, const float* scores, int64_t score_stride, const int32_t* row_of_slot,
                              const uint32_t* nslots, int max_slots, int32_t* idx, int32_t* count, uint32_t* status,
                              const DeviceInfo& dev, cudaStream_t stream) {
  TopkPlan plan;
  plan.cluster = 1;
  plan.one_sweep = 0;
  size_blocks(plan, p.max_seq_len, dev);
  auto kernel = plan.slice_cap > 0 ? topk_radix_slots_kernel<true> : topk_radix_slots_kernel<false>;
  cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem_bytes);
  if (err != cudaSuccess) return err;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)max_slots, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = plan.smem_bytes;
  cfg.stream = stream;
  return cudaLaunchKernelEx(&cfg, kernel, scores, score_stride, p.seq_len, (int)p.q_per_seq, (int)p.causal, (int)p.top_k,
                            (int)p.max_seq_len, row_of_slot, nslots, idx, count, status);
}

}  // namespace clsa
