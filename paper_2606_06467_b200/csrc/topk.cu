// Token-level top-k (Eq. 3, second half) as an exact MSB-first radix select.
//
// One thread-block cluster per (sequence, query) row. The row's visible scores are cut into
// contiguous slices, one per block; each block converts its slice once to order-preserving 32-bit
// keys held in shared memory, so the radix passes never go back to global memory. Three passes
// resolve 12 + 12 + 8 key bits. fp32 scores crowd into a few sign/exponent patterns, so a wide
// first digit (sign, exponent and three mantissa bits) is what keeps the shared-memory histogram
// atomics from serialising on a handful of bins; a warp whose lanes all hit one bin adds once.
// Per pass: each block histograms its slice into shared memory, then adds its non-empty bins into
// every block's copy of the cluster-wide histogram with distributed-shared-memory atomics; after
// one cluster barrier every block scans its own copy from the top bin down and finds, redundantly
// and identically, the digit that contains the k-th largest key (the copies are double-buffered,
// so one barrier per pass is enough). After three passes the exact threshold key and the number
// of threshold-equal elements still needed are known. The compaction is index-ordered: a block's
// output offset is the number of selected elements in lower-ranked blocks, a warp's offset the
// number selected in lower warps, so positions come out ascending and, among keys equal to the
// threshold, the lowest positions win. No atomics touch global memory and nothing spins.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace clsa {
namespace {

constexpr int kThreads = 512;  // 512 threads and < 113 KiB of shared memory: two blocks per SM, so that 16+ clusters of 8 are resident at once
constexpr int kWarps = kThreads / 32;
constexpr int kMaxBins = 4096;
constexpr int kMaxCluster = 8;

struct Shared {
  uint32_t local_hist[kMaxBins];       // this block's slice
  uint32_t cluster_hist[2][kMaxBins];  // whole row, one copy per block, filled by every block of the cluster
  uint32_t warp_tot[kWarps];
  uint32_t warp_gt[kWarps], warp_eq[kWarps];
  uint32_t block_gt_eq[2];             // read remotely
  uint32_t digit, k_rem;
  uint32_t out_base, eq_base;
};

__device__ __forceinline__ uint32_t score_key(float x) {
  uint32_t u = __float_as_uint(x);
  if (u == 0x80000000u) u = 0u;  // -0.0 ranks equal to +0.0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// One radix pass over `BITS` key bits starting at `shift`. On return prefix/prefix_mask/k_rem are
// updated. `buf` selects the cluster_hist copy (alternates between passes).
template <int BITS, typename KeyAt>
__device__ __forceinline__ void radix_pass(Shared& sh, cg::cluster_group& cluster, int nblk, int cnt, int shift, int buf,
                                           uint32_t& prefix, uint32_t& prefix_mask, uint32_t& k_rem, KeyAt key_at) {
  constexpr int NB = 1 << BITS;
  constexpr int PT = (NB + kThreads - 1) / kThreads;  // bins per thread
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  for (int i = tid; i < NB; i += kThreads) sh.local_hist[i] = 0;
  __syncthreads();
  for (int i0 = 0; i0 < cnt; i0 += kThreads) {
    const int i = i0 + tid;
    const uint32_t key = i < cnt ? key_at(i) : 0u;
    const bool in = i < cnt && (key & prefix_mask) == prefix;
    const uint32_t bin = (key >> shift) & (uint32_t)(NB - 1);
    const uint32_t voters = __ballot_sync(0xffffffffu, in);
    if (voters == 0u) continue;
    // all participating lanes on one bin (long runs of equal scores): one add for the warp
    const uint32_t lead_bin = __shfl_sync(0xffffffffu, bin, __ffs(voters) - 1);
    const bool same = __all_sync(0xffffffffu, !in || bin == lead_bin);
    if (same) {
      if (lane == __ffs(voters) - 1) atomicAdd(&sh.local_hist[bin], (uint32_t)__popc(voters));
    } else if (in) {
      atomicAdd(&sh.local_hist[bin], 1u);
    }
  }
  __syncthreads();
  // add this block's non-empty bins into every block's copy of the row histogram
  uint32_t* mine = sh.cluster_hist[buf];
#pragma unroll
  for (int j = 0; j < PT; ++j) {
    const int bin = tid + j * kThreads;
    if (bin < NB) {
      const uint32_t v = sh.local_hist[bin];
      if (v != 0u)
        for (int r = 0; r < nblk; ++r) atomicAdd(cluster.map_shared_rank(mine, r) + bin, v);
    }
  }
  cluster.sync();
  // scan this block's copy from the top bin down: thread t owns bins NB-1-(t*PT+j)
  uint32_t own[PT];
  uint32_t tot = 0;
#pragma unroll
  for (int j = 0; j < PT; ++j) {
    const int pos = tid * PT + j;
    own[j] = pos < NB ? mine[NB - 1 - pos] : 0u;
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
      }
      acc += own[j];
    }
  }
  // clear the copy for its next use (two passes on); nobody else touches it before the next barrier
#pragma unroll
  for (int j = 0; j < PT; ++j) {
    const int pos = tid * PT + j;
    if (pos < NB) mine[NB - 1 - pos] = 0u;
  }
  __syncthreads();
  prefix |= sh.digit << shift;
  prefix_mask |= (uint32_t)(NB - 1) << shift;
  k_rem = sh.k_rem;
}

template <bool CACHED>
__global__ void __launch_bounds__(kThreads, 2)
topk_radix_kernel(const float* __restrict__ scores, int64_t score_stride, const int32_t* __restrict__ seq_len,
                  int q_per_seq, int causal, int top_k, int max_seq_len, int32_t* __restrict__ idx_out,
                  int32_t* __restrict__ count_out, uint32_t* status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  Shared& sh = *reinterpret_cast<Shared*>(smem_raw);
  uint32_t* keys = reinterpret_cast<uint32_t*>(smem_raw + sizeof(Shared));

  cg::cluster_group cluster = cg::this_cluster();
  const int nblk = (int)cluster.num_blocks();
  const int rank = (int)cluster.block_rank();
  const int row = blockIdx.x / nblk;
  const int b = row / q_per_seq, t = row % q_per_seq;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

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
  const int per = (v + nblk - 1) / nblk;
  const int lo = min(v, rank * per), hi = min(v, lo + per);
  const int cnt = hi - lo;
  if (kk == v) {  // nothing to select: every visible position is taken, in order
    for (int i = tid; i < cnt; i += kThreads) out[lo + i] = lo + i;
    return;
  }
  const float* src = scores + (int64_t)row * score_stride + lo;
  if (CACHED) {
    for (int i = tid; i < cnt; i += kThreads) keys[i] = score_key(src[i]);
  }
  auto key_at = [&](int i) -> uint32_t { return CACHED ? keys[i] : score_key(src[i]); };
  for (int i = tid; i < 2 * kMaxBins; i += kThreads) (&sh.cluster_hist[0][0])[i] = 0;
  // the remote adds of pass 0 may arrive as soon as a neighbour gets there: every block must have
  // cleared its copies first
  cluster.sync();

  // ---- three radix passes: bits 31..20, 19..8, 7..0 --------------------------------------------
  uint32_t prefix = 0, prefix_mask = 0, k_rem = (uint32_t)kk;
  radix_pass<12>(sh, cluster, nblk, cnt, 20, 0, prefix, prefix_mask, k_rem, key_at);
  radix_pass<12>(sh, cluster, nblk, cnt, 8, 1, prefix, prefix_mask, k_rem, key_at);
  radix_pass<8>(sh, cluster, nblk, cnt, 0, 0, prefix, prefix_mask, k_rem, key_at);
  const uint32_t thr = prefix;        // key of the kk-th largest element
  const uint32_t need_eq = k_rem;     // how many threshold-equal elements are selected (>= 1)

  // ---- index-ordered compaction ----------------------------------------------------------------
  const int chunk = ((cnt + kWarps - 1) / kWarps + 31) & ~31;  // contiguous positions per warp
  const int c_lo = min(cnt, warp * chunk), c_hi = min(cnt, c_lo + chunk);
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
  // offsets of this warp: selected / threshold-equal elements in lower warps of this block
  uint32_t out_pos = sh.out_base, eq_rank = sh.eq_base;
  for (int w = 0; w < warp; ++w) {
    const uint32_t e = sh.warp_eq[w];
    const uint32_t take = eq_rank >= need_eq ? 0u : min(e, need_eq - eq_rank);
    out_pos += sh.warp_gt[w] + take;
    eq_rank += e;
  }
  const uint32_t lt_mask = (1u << lane) - 1u;
  for (int i0 = c_lo; i0 < c_hi; i0 += 32) {
    const int i = i0 + lane;
    const uint32_t key = i < c_hi ? key_at(i) : 0u;
    const bool is_gt = i < c_hi && key > thr;
    const bool is_eq = i < c_hi && key == thr;
    const uint32_t eq_ballot = __ballot_sync(0xffffffffu, is_eq);
    const bool take = is_gt || (is_eq && eq_rank + __popc(eq_ballot & lt_mask) < need_eq);
    const uint32_t take_ballot = __ballot_sync(0xffffffffu, take);
    if (take) {
      const uint32_t pos = out_pos + __popc(take_ballot & lt_mask);
      if (pos < (uint32_t)kk) out[pos] = lo + i;
    }
    out_pos += __popc(take_ballot);
    eq_rank += __popc(eq_ballot);
  }
  cluster.sync();  // no block may exit while a neighbour can still read its shared memory
}

}  // namespace

TopkPlan make_topk_plan(const clsa_params& p, const DeviceInfo& dev) {
  TopkPlan plan;
  // One block per 16K visible scores, capped at the portable cluster size and rounded to a power of
  // two; when there are few rows, spread each over more blocks (down to 2K scores per block).
  int c = (p.max_seq_len + 16383) / 16384;
  if (c > kMaxCluster) c = kMaxCluster;
  int pow2 = 1;
  while (pow2 < c) pow2 <<= 1;
  const int64_t rows = (int64_t)p.num_seqs * p.q_per_seq;
  while (pow2 < kMaxCluster && rows * pow2 * 2 <= dev.sm_count && p.max_seq_len / (pow2 * 2) >= 2048) pow2 <<= 1;
  plan.cluster = pow2;
  const int per = (p.max_seq_len + plan.cluster - 1) / plan.cluster;
  const size_t want = sizeof(Shared) + (size_t)per * sizeof(uint32_t);
  if (want <= (size_t)dev.max_smem_optin) {
    plan.slice_cap = per;
    plan.smem_bytes = want;
  } else {
    plan.slice_cap = 0;  // slice too long for shared memory: keys are recomputed from global memory each pass
    plan.smem_bytes = sizeof(Shared);
  }
  return plan;
}

cudaError_t launch_topk(const clsa_params& p, const float* scores, int64_t score_stride, int32_t* idx, int32_t* count,
                        uint32_t* status, const DeviceInfo& dev, cudaStream_t stream) {
  const TopkPlan plan = make_topk_plan(p, dev);
  const int64_t rows = (int64_t)p.num_seqs * p.q_per_seq;
  auto kernel = plan.slice_cap > 0 ? topk_radix_kernel<true> : topk_radix_kernel<false>;
  cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem_bytes);
  if (err != cudaSuccess) return err;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(rows * plan.cluster), 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = plan.smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)plan.cluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, scores, score_stride, p.seq_len, (int)p.q_per_seq, (int)p.causal,
                            (int)p.top_k, (int)p.max_seq_len, idx, count, status);
}

}  // namespace clsa
