// Token-level top-k (Eq. 3, second half) as an exact MSB-first radix select.
//
// One thread-block cluster per (sequence, query) row. The row's visible scores are cut into
// contiguous slices, one per block; each block converts its slice once to order-preserving 32-bit
// keys held in shared memory, so the four 8-bit radix passes never go back to global memory.
// Per pass every warp histograms into its own 256-bin shared-memory histogram, the block folds the
// warp histograms, and the blocks of the cluster read each other's folded histogram through
// distributed shared memory; every block then finds, redundantly and identically, the digit bin
// that contains the k-th largest key. After four passes the exact threshold key and the number of
// threshold-equal elements still needed are known. The compaction is index-ordered: a block's
// output offset is the number of selected elements in lower-ranked blocks, a warp's offset the
// number selected in lower warps, so positions come out ascending and, among keys equal to the
// threshold, the lowest positions win. No atomics touch global memory and nothing spins.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace clsa {
namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kBins = 256;
constexpr int kHistStride = kBins + 1;  // odd stride: equal bins of different warps fall in different banks
constexpr int kMaxCluster = 8;

struct Shared {
  uint32_t warp_hist[kWarps * kHistStride];
  uint32_t block_hist[2][kBins];   // double-buffered: read remotely by the other blocks of the cluster
  uint32_t global_hist[kBins];
  uint32_t warp_gt[kWarps], warp_eq[kWarps];
  uint32_t block_gt_eq[2];         // read remotely
  uint32_t digit, k_rem;
  uint32_t out_base, eq_base;
};

__device__ __forceinline__ uint32_t score_key(float x) {
  uint32_t u = __float_as_uint(x);
  if (u == 0x80000000u) u = 0u;  // -0.0 ranks equal to +0.0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

template <bool CACHED>
__global__ void __launch_bounds__(kThreads, 1)
topk_radix_kernel(const float* __restrict__ scores, int64_t score_stride, const int32_t* __restrict__ seq_len,
                  int q_per_seq, int causal, int top_k, int max_seq_len, int slice_cap, int32_t* __restrict__ idx_out,
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
  __syncthreads();

  // ---- four radix passes -------------------------------------------------------------------
  uint32_t prefix = 0, prefix_mask = 0, k_rem = (uint32_t)kk;
#pragma unroll 1
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int i = tid; i < kWarps * kHistStride; i += kThreads) sh.warp_hist[i] = 0;
    __syncthreads();
    uint32_t* my_hist = sh.warp_hist + warp * kHistStride;
    for (int i = tid; i < cnt; i += kThreads) {
      const uint32_t key = key_at(i);
      if ((key & prefix_mask) == prefix) atomicAdd(&my_hist[(key >> shift) & 0xffu], 1u);
    }
    __syncthreads();
    uint32_t* bh = sh.block_hist[pass & 1];
    if (tid < kBins) {
      uint32_t s = 0;
#pragma unroll 8
      for (int w = 0; w < kWarps; ++w) s += sh.warp_hist[w * kHistStride + tid];
      bh[tid] = s;
    }
    cluster.sync();
    if (tid < kBins) {
      uint32_t s = 0;
      for (int r = 0; r < nblk; ++r) s += cluster.map_shared_rank(bh, r)[tid];
      sh.global_hist[tid] = s;
    }
    __syncthreads();
    if (warp == 0) {
      // lane l owns bins 255-8l .. 248-8l, scanned from the top bin down
      uint32_t own = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) own += sh.global_hist[255 - 8 * lane - j];
      uint32_t incl = own;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const uint32_t up = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += up;
      }
      const uint32_t excl = incl - own;
      if (excl < k_rem && k_rem <= incl) {
        uint32_t acc = excl;
        for (int j = 0; j < 8; ++j) {
          const int bin = 255 - 8 * lane - j;
          const uint32_t c = sh.global_hist[bin];
          if (acc + c >= k_rem) { sh.digit = (uint32_t)bin; sh.k_rem = k_rem - acc; break; }
          acc += c;
        }
      }
    }
    __syncthreads();
    prefix |= sh.digit << shift;
    prefix_mask |= 0xffu << shift;
    k_rem = sh.k_rem;
    // block_hist is double-buffered, so the next pass may start without a second cluster barrier:
    // buffer (pass & 1) is rewritten only in pass + 2, after the cluster.sync() of pass + 1.
  }
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
    uint32_t g = sh.warp_gt[lane], e = sh.warp_eq[lane];
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
                            (int)p.top_k, (int)p.max_seq_len, plan.slice_cap, idx, count, status);
}

}  // namespace clsa
