// Token-level top-k (Eq. 3, second half) for many long rows at once (a prefill chunk: thousands of
// (sequence, query) rows of 10^5 scores each; or a decode batch with more rows than the general kernel's
// clusters can all be resident for), where throughput matters and not the latency of one row.
//
// The general kernel (topk.cu) reads a row three times and pays a vote and a shared-memory atomic per
// score. Here a row is read ONCE at full width, and per score only a float compare is paid:
//   1. sample   4096 scores of the row (1024 16-byte loads spread evenly over it, kept in registers) -> a
//               22-bit radix select finds a pivot key near the r-th largest sample, r chosen so that the pivot
//               lies below the row's k-th largest key with a margin of a few standard deviations;
//   2. filter   one sweep over the row compares each score with the pivot (as floats: one instruction per
//               score) and sets one bit per passing score in a position bitmap in shared memory (one atomic OR
//               of a 4-bit group per 16-byte load that has any);
//   3. list     a prefix count over the bitmap turns it into the list of candidate positions, already in
//               ascending order (about 1.4 k entries); their scores are fetched again (a sparse gather, mostly
//               L2 hits) and converted to order-preserving keys;
//   4. select   if the list holds at least k entries (then it contains the k largest, with all their ties) and
//               no more than its capacity, an exact select over it gives the threshold key and the number of
//               threshold-equal keys still needed: one 4096-bin histogram over the candidates' actual spread
//               (key - pivot, shifted), then a direct ranking of the handful of keys in the threshold's bin
//               (or, when ties crowd that bin, 10-bit radix passes over the remaining bits);
//   5. emit     an ordered compaction of the list: keys above the threshold and the first needed keys equal to
//               it, in list (= position) order.
// The result is exact whenever the block finishes. A row it cannot finish -- pivot too high (fewer than k
// candidates), too many candidates (long runs of equal scores, or scores far from the sampled profile), a row
// too long for the bitmap, misaligned for 16-byte loads, or holding NaNs that the float compare lets through
// below the pivot -- is marked pending (count = -1) and is taken by the general kernel, launched right after for
// pending rows only. Nothing is approximated.
#include <cmath>

#include "common.cuh"

namespace clsa {
namespace {

constexpr int kThreads = 512;           // two blocks per SM: one row's sweep overlaps the other's select/order
constexpr int kWarps = kThreads / 32;
constexpr int kSample = 4096;
constexpr int kCandCap = 6144;
constexpr int kSmallBin = 64;           // a threshold bin this small is finished by one warp ranking its keys
constexpr uint32_t kFull = 0xffffffffu;

struct alignas(16) FShared {
  uint32_t hist[4096];
  uint32_t hist10[1024];
  uint32_t warp_tot[kWarps];
  uint32_t small_key[kSmallBin];
  uint32_t digit, k_rem, bin_count, cand_count;
  uint32_t cand_max, small_count, thr, need_eq;
  uint32_t below_pivot, pad_[3];
  uint32_t cand_pos[kCandCap];  // candidate positions, ascending
  uint32_t cand_key[kCandCap];  // their keys
};
static_assert(sizeof(FShared) % 16 == 0, "the arrays behind FShared must stay 16-byte aligned");

__device__ __forceinline__ uint32_t score_key(float x) {
  uint32_t u = __float_as_uint(x);
  if (u == 0x80000000u) u = 0u;  // -0.0 ranks equal to +0.0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_score(uint32_t key) {  // inverse of score_key
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// Exclusive prefix sum of `val` over the block in thread order.
__device__ __forceinline__ uint32_t block_excl_scan(FShared& sh, uint32_t val) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t incl = val;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t up = __shfl_up_sync(kFull, incl, d);
    if (lane >= d) incl += up;
  }
  __syncthreads();  // warp_tot may still be read by the previous scan
  if (lane == 31) sh.warp_tot[warp] = incl;
  __syncthreads();
  // every warp scans the kWarps warp totals itself with shuffles (lane l holds warp l's total)
  uint32_t tot = lane < kWarps ? sh.warp_tot[lane] : 0u;
#pragma unroll
  for (int d = 1; d < kWarps; d <<= 1) {
    const uint32_t up = __shfl_up_sync(kFull, tot, d);
    if (lane >= d) tot += up;
  }
  const uint32_t before = __shfl_sync(kFull, tot, (warp + 31) & 31);  // inclusive total of the warps below this one
  return (warp == 0 ? 0u : before) + incl - val;
}

// Scan hist[0..NB) from the top bin down to the bin in which the running count reaches k_rem; clears the
// histogram. After it (block-synchronised): sh.digit = that bin, sh.k_rem = what is still needed inside it,
// sh.bin_count = its population.
template <int NB>
__device__ __forceinline__ void scan_from_top(FShared& sh, uint32_t* hist, uint32_t k_rem) {
  constexpr int PT = NB / kThreads;
  static_assert(NB % kThreads == 0, "bins divide evenly over the threads");
  const int tid = threadIdx.x;
  uint32_t own[PT], tot = 0;
#pragma unroll
  for (int j = 0; j < PT; ++j) {
    own[j] = hist[NB - 1 - (tid * PT + j)];  // thread t owns the bins NB-1-(t*PT+j)
    tot += own[j];
  }
  const uint32_t excl = block_excl_scan(sh, tot);
  if (excl < k_rem && k_rem <= excl + tot) {
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
#pragma unroll
  for (int j = 0; j < PT; ++j) hist[NB - 1 - (tid * PT + j)] = 0u;
  __syncthreads();
}

__global__ void __launch_bounds__(kThreads, 2)
topk_prefilter_kernel(const float* __restrict__ scores, int64_t score_stride, const int32_t* __restrict__ seq_len,
                      int q_per_seq, int causal, int top_k, int max_seq_len, int bitmap_words,
                      int32_t* __restrict__ idx_out, int32_t* __restrict__ count_out, uint32_t* status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  FShared& sh = *reinterpret_cast<FShared*>(smem_raw);
  uint32_t* bitmap = reinterpret_cast<uint32_t*>(smem_raw + sizeof(FShared));  // one bit per position of the row

  const int row = blockIdx.x;
  const int b = row / q_per_seq, t = row % q_per_seq;
  const int tid = threadIdx.x, lane = tid & 31;
  // Programmatic dependent launch: the kernel behind this one may be scheduled early (it waits for this grid
  // itself), and this grid may have been scheduled before the kernel that writes the scores has finished: shared
  // memory is cleared meanwhile, and the wait comes before the first global access.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  for (int i = tid; i < 4096; i += kThreads) sh.hist[i] = 0u;
  for (int i = tid; i < 1024; i += kThreads) sh.hist10[i] = 0u;
  for (int i = tid; i < bitmap_words; i += kThreads) bitmap[i] = 0u;
  if (tid == 0) { sh.cand_count = 0u; sh.cand_max = 0u; sh.small_count = 0u; sh.below_pivot = 0u; }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int n = seq_len[b];
  int v = causal ? n - q_per_seq + t + 1 : n;
  if (n < q_per_seq || n > max_seq_len) {
    v = 0;
    if (tid == 0) flag_status(status, CLSA_DEV_BAD_SEQLEN);
  }
  const int kk = min(top_k, v);
  int32_t* out = idx_out + (int64_t)row * top_k;
  const float* src = scores + (int64_t)row * score_stride;
  if (kk == v) {  // nothing to select: every visible position is taken, in order
    if (tid == 0) count_out[row] = kk;
    for (int i = tid; i < top_k; i += kThreads) out[i] = i < kk ? i : -1;
    return;
  }
  if (v > bitmap_words * 32 || (reinterpret_cast<uintptr_t>(src) & 15u) != 0) {
    if (tid == 0) count_out[row] = -1;  // left to the general kernel
    return;
  }
  const float4* src4 = reinterpret_cast<const float4*>(src);
  const int n4 = v >> 2;

  // ---- 1. pivot from a sample ------------------------------------------------------------------------------------
  constexpr int kPer = kSample / 4 / kThreads;  // 16-byte samples per thread, kept in registers
  float4 smp[kPer];
  if (v > kCandCap) {
#pragma unroll
    for (int u = 0; u < kPer; ++u) smp[u] = src4[(int)(((int64_t)(tid + u * kThreads) * n4) / (kSample / 4))];
  }
  __syncthreads();  // the clears at the top

  uint32_t pivot = 0u;  // rows that fit the candidate list whole need none
  if (v > kCandCap) {
    uint4 key[kPer];
#pragma unroll
    for (int u = 0; u < kPer; ++u) {
      key[u] = make_uint4(score_key(smp[u].x), score_key(smp[u].y), score_key(smp[u].z), score_key(smp[u].w));
      atomicAdd(&sh.hist[key[u].x >> 20], 1u);
      atomicAdd(&sh.hist[key[u].y >> 20], 1u);
      atomicAdd(&sh.hist[key[u].z >> 20], 1u);
      atomicAdd(&sh.hist[key[u].w >> 20], 1u);
    }
    __syncthreads();
    // rank of the pivot inside the sample: the expected number of sampled keys among the row's k largest, plus
    // 10 % and 3.5 standard deviations of that count, so that the pivot falls below the k-th largest key
    const float expect = (float)kSample * (float)kk / (float)v * 1.10f;
    const uint32_t r = min((uint32_t)kSample, (uint32_t)(expect + 3.5f * sqrtf(expect) + 4.0f));
    scan_from_top<4096>(sh, sh.hist, r);
    const uint32_t d0 = sh.digit, r1 = sh.k_rem;
#pragma unroll
    for (int u = 0; u < kPer; ++u) {  // second digit: only the sampled keys inside the first digit's bin
      if ((key[u].x >> 20) == d0) atomicAdd(&sh.hist10[(key[u].x >> 10) & 1023u], 1u);
      if ((key[u].y >> 20) == d0) atomicAdd(&sh.hist10[(key[u].y >> 10) & 1023u], 1u);
      if ((key[u].z >> 20) == d0) atomicAdd(&sh.hist10[(key[u].z >> 10) & 1023u], 1u);
      if ((key[u].w >> 20) == d0) atomicAdd(&sh.hist10[(key[u].w >> 10) & 1023u], 1u);
    }
    __syncthreads();
    scan_from_top<1024>(sh, sh.hist10, r1);
    pivot = (d0 << 20) | (sh.digit << 10);
  }
  // The sweep compares scores as floats (one instruction per score) against the score whose key is the pivot;
  // float order and key order agree for everything but NaN, and "not below" lets every NaN through to the exact
  // key comparison. A pivot that is itself a NaN pattern cannot be compared against: hand the row back.
  const float pivot_f = pivot == 0u ? __int_as_float(0xff800000) : key_score(pivot);  // no pivot: -inf, all pass
  if (pivot_f != pivot_f) {
    if (tid == 0) count_out[row] = -1;
    return;
  }

  // ---- 2. one sweep: mark every score that is not below the pivot -------------------------------------------
  {
    // Rolling prefetch: a thread keeps kBatch 16-byte loads in flight; a consumed register is refilled at once
    // with the load kBatch steps ahead.
    constexpr int kBatch = 8;
    const float4 pad = make_float4(pivot_f, pivot_f, pivot_f, pivot_f);
    float4 f[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u) {
      const int i = u * kThreads + tid;
      f[u] = i < n4 ? src4[i] : pad;
    }
    for (int i0 = 0; i0 < n4; i0 += kThreads * kBatch) {
#pragma unroll
      for (int u = 0; u < kBatch; ++u) {
        const int i = i0 + u * kThreads + tid;
        const float4 cur = f[u];
        const int nxt = i + kThreads * kBatch;
        f[u] = nxt < n4 ? src4[nxt] : pad;
        const uint32_t m = (cur.x < pivot_f ? 0u : 1u) | (cur.y < pivot_f ? 0u : 2u) | (cur.z < pivot_f ? 0u : 4u) |
                           (cur.w < pivot_f ? 0u : 8u);
        if (m != 0u && i < n4) atomicOr(&bitmap[i >> 3], m << (4 * (i & 7)));  // positions 4i .. 4i+3
      }
    }
    const int i = n4 * 4 + tid;  // up to three leftover scores
    if (i < v && !(src[i] < pivot_f)) atomicOr(&bitmap[i >> 5], 1u << (i & 31));
  }
  __syncthreads();

  // ---- 3. bitmap -> ascending list of candidate positions, then their keys -------------------------------------
  const int words = (v + 31) >> 5;
  {
    const int per = (words + kThreads - 1) / kThreads;  // consecutive bitmap words per thread
    const int w_lo = min(words, tid * per), w_hi = min(words, w_lo + per);
    uint32_t mine = 0;
    for (int w = w_lo; w < w_hi; ++w) mine += __popc(bitmap[w]);
    uint32_t off = block_excl_scan(sh, mine);
    if (tid == kThreads - 1) sh.cand_count = off + mine;
    __syncthreads();
    const uint32_t total = sh.cand_count;
    if (total > (uint32_t)kCandCap || total < (uint32_t)kk) {  // too many, or the pivot came out above the k-th largest
      if (tid == 0) count_out[row] = -1;
      return;
    }
    for (int w = w_lo; w < w_hi; ++w) {
      uint32_t bits = bitmap[w];
      while (bits != 0u) {
        sh.cand_pos[off++] = (uint32_t)(w * 32 + __ffs(bits) - 1);
        bits &= bits - 1u;
      }
    }
  }
  __syncthreads();
  const uint32_t C = sh.cand_count;
  {
    uint32_t my_max = 0u, bad = 0u;
    constexpr int kPerThread = kCandCap / kThreads;  // all of a thread's gather loads are issued before the first is used
    static_assert(kCandCap % kThreads == 0, "whole candidates per thread");
    float x[kPerThread];
#pragma unroll
    for (int u = 0; u < kPerThread; ++u) {
      const uint32_t i = (uint32_t)(u * kThreads + tid);
      x[u] = i < C ? src[sh.cand_pos[i]] : 0.f;
    }
#pragma unroll
    for (int u = 0; u < kPerThread; ++u) {
      const uint32_t i = (uint32_t)(u * kThreads + tid);
      if (i < C) {
        const uint32_t key = score_key(x[u]);
        sh.cand_key[i] = key;
        my_max = max(my_max, key);
        bad |= key < pivot ? 1u : 0u;  // a NaN with the sign bit set: not below the pivot as a float, below it as a key
      }
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) my_max = max(my_max, __shfl_xor_sync(kFull, my_max, d));
    if (lane == 0) atomicMax(&sh.cand_max, my_max);
    if (bad != 0u) sh.below_pivot = 1u;
  }
  __syncthreads();
  if (sh.below_pivot != 0u) {
    if (tid == 0) count_out[row] = -1;
    return;
  }

  // ---- 4. exact select over the candidates ------------------------------------------------------------------------
  // Candidates lie in [pivot, cand_max]. d = key - pivot is order preserving; its top 12 significant bits (of the
  // actual spread, not of the float format) make a first digit that spreads the candidates thinly over 4096 bins.
  const uint32_t range = sh.cand_max - pivot;
  const int s = max(0, 32 - __clz(range) - 12);  // range >> s < 4096
  for (uint32_t i = tid; i < C; i += kThreads) atomicAdd(&sh.hist[(sh.cand_key[i] - pivot) >> s], 1u);
  __syncthreads();
  scan_from_top<4096>(sh, sh.hist, (uint32_t)kk);
  const uint32_t b1 = sh.digit, k1 = sh.k_rem, cnt1 = sh.bin_count;
  if (cnt1 <= (uint32_t)kSmallBin) {
    // the usual case: a handful of keys share the threshold's bin; one warp ranks them
    for (uint32_t i = tid; i < C; i += kThreads) {
      const uint32_t key = sh.cand_key[i];
      if (((key - pivot) >> s) == b1) sh.small_key[atomicAdd(&sh.small_count, 1u)] = key;
    }
    __syncthreads();
    if (tid < kSmallBin && tid < (int)cnt1) {
      const uint32_t mine = sh.small_key[tid];
      uint32_t greater = 0, equal = 0;
      for (uint32_t j = 0; j < cnt1; ++j) {
        const uint32_t other = sh.small_key[j];
        greater += other > mine;
        equal += other == mine;
      }
      if (greater < k1 && k1 <= greater + equal) {  // the k1-th largest of the bin (equal keys all write the same)
        sh.thr = mine;
        sh.need_eq = k1 - greater;
      }
    }
    __syncthreads();
  } else {
    // many keys in the threshold's bin (ties, quantised scores): resolve the remaining s bits of d, 10 at a time
    uint32_t prefix = b1 << s, mask = s == 0 ? 0xffffffffu : ~((1u << s) - 1u), k_rem = k1;
    int rest = s;
#pragma unroll 1
    while (rest > 0) {
      const int wbits = min(10, rest), shift = rest - wbits;
      for (uint32_t i = tid; i < C; i += kThreads) {
        const uint32_t d = sh.cand_key[i] - pivot;
        if ((d & mask) == prefix) atomicAdd(&sh.hist10[(d >> shift) & ((1u << wbits) - 1u)], 1u);
      }
      __syncthreads();
      scan_from_top<1024>(sh, sh.hist10, k_rem);
      prefix |= sh.digit << shift;
      mask |= ((1u << wbits) - 1u) << shift;
      k_rem = sh.k_rem;
      rest = shift;
    }
    if (tid == 0) { sh.thr = pivot + prefix; sh.need_eq = k_rem; }
    __syncthreads();
  }
  const uint32_t thr = sh.thr, need_eq = sh.need_eq;  // take every key > thr and the need_eq lowest positions with key == thr

  // ---- 5. ordered compaction of the list ---------------------------------------------------------------------
  {
    const uint32_t per = (C + kThreads - 1) / kThreads;  // consecutive list entries per thread
    const uint32_t c_lo = min(C, (uint32_t)tid * per), c_hi = min(C, c_lo + per);
    uint32_t n_gt = 0, n_eq = 0;
    for (uint32_t i = c_lo; i < c_hi; ++i) {
      const uint32_t key = sh.cand_key[i];
      n_gt += key > thr;
      n_eq += key == thr;
    }
    // one scan for both counts (each is below 2^16): keys above the threshold / equal to it at lower positions
    const uint32_t both = block_excl_scan(sh, (n_gt << 16) | n_eq);
    uint32_t eq_rank = both & 0xffffu;
    uint32_t off = (both >> 16) + min(eq_rank, need_eq);  // equal keys are taken in order until need_eq are in
    for (uint32_t i = c_lo; i < c_hi; ++i) {
      const uint32_t key = sh.cand_key[i];
      bool sel = key > thr;
      if (key == thr) sel = eq_rank++ < need_eq;  // the lowest positions first
      if (sel) {
        if (off < (uint32_t)kk) out[off] = (int32_t)sh.cand_pos[i];
        ++off;
      }
    }
  }
  if (tid == 0) count_out[row] = kk;
  for (int i = kk + tid; i < top_k; i += kThreads) out[i] = -1;
}

// ---------------------------------------------------------------------------------------------------------------------
// Exact TopK of a row from a candidate list that somebody else filtered (the chunk GEMM's epilogue, clsa_index_topk):
// unordered (score bits, position) pairs that contain every score not below the row's pivot. Steps 4 and 5 of the
// kernel above on that list; the positions come out ascending through a position bitmap, since the list has no order.
// A row that cannot be finished exactly from its list -- fewer than k candidates (pivot too high), more than the list
// holds, a NaN below the pivot, more threshold-equal keys than can be ranked here -- gets count = -1 and is recomputed
// by the caller.
constexpr int kEqCap = 1024;  // threshold-equal candidates that are ranked by position here

__global__ void __launch_bounds__(kThreads, 2)
topk_candidates_kernel(const uint2* __restrict__ cand, const uint32_t* __restrict__ cand_count, int cand_cap,
                       const float* __restrict__ pivot_of_row, const int32_t* __restrict__ seq_len, int q_per_seq, int causal,
                       int top_k, int max_seq_len, int bitmap_words, int32_t* __restrict__ idx_out,
                       int32_t* __restrict__ count_out, uint32_t* status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  FShared& sh = *reinterpret_cast<FShared*>(smem_raw);
  uint32_t* eq_pos = reinterpret_cast<uint32_t*>(smem_raw + sizeof(FShared));
  uint32_t* bitmap = eq_pos + kEqCap;  // one bit per position of the row

  const int row = blockIdx.x;
  const int b = row / q_per_seq, t = row % q_per_seq;
  const int tid = threadIdx.x, lane = tid & 31;
  for (int i = tid; i < 4096; i += kThreads) sh.hist[i] = 0u;
  for (int i = tid; i < 1024; i += kThreads) sh.hist10[i] = 0u;
  if (tid == 0) { sh.cand_count = 0u; sh.cand_max = 0u; sh.small_count = 0u; sh.below_pivot = 0u; }
  const int n = seq_len[b];
  int v = causal ? n - q_per_seq + t + 1 : n;
  if (n < q_per_seq || n > max_seq_len) {
    v = 0;
    if (tid == 0) flag_status(status, CLSA_DEV_BAD_SEQLEN);
  }
  const int kk = min(top_k, v);
  int32_t* out = idx_out + (int64_t)row * top_k;
  if (kk == v) {  // nothing to select: every visible position is taken, in order
    if (tid == 0) count_out[row] = kk;
    for (int i = tid; i < top_k; i += kThreads) out[i] = i < kk ? i : -1;
    return;
  }
  const int words = (v + 31) >> 5;
  for (int i = tid; i < words; i += kThreads) bitmap[i] = 0u;
  const uint32_t slots = cand_count[row];  // slots handed out, holes included
  if (slots > (uint32_t)cand_cap || words > bitmap_words) {
    if (tid == 0) count_out[row] = -1;
    return;
  }
  const uint32_t pivot = score_key(pivot_of_row[row]);
  const uint2* list = cand + (int64_t)row * cand_cap;
  __syncthreads();  // sh.cand_count is zero
  {
    // the list's entries without its holes (position = 0xffffffff: a slot that was reserved and not used), in no
    // particular order
    uint32_t my_max = 0u, bad = 0u;
    constexpr int kPerThread = kCandCap / kThreads;  // all of a thread's loads are issued before the first is used
    uint2 e[kPerThread];
#pragma unroll
    for (int u = 0; u < kPerThread; ++u) {
      const uint32_t i = (uint32_t)(u * kThreads + tid);
      e[u] = i < slots ? list[i] : make_uint2(0u, 0xffffffffu);
    }
#pragma unroll
    for (int u = 0; u < kPerThread; ++u) {
      if ((uint32_t)(u * kThreads) >= slots) break;  // uniform over the block
      const bool real = e[u].y != 0xffffffffu;
      const uint32_t ballot = __ballot_sync(kFull, real);
      uint32_t at = 0;
      if (lane == 0 && ballot != 0u) at = atomicAdd(&sh.cand_count, (uint32_t)__popc(ballot));
      at = __shfl_sync(kFull, at, 0) + __popc(ballot & ((1u << lane) - 1u));
      if (real) {
        const uint32_t key = score_key(__uint_as_float(e[u].x));
        sh.cand_key[at] = key;
        sh.cand_pos[at] = e[u].y;
        my_max = max(my_max, key);
        bad |= (key < pivot || e[u].y >= (uint32_t)v) ? 1u : 0u;  // a NaN with the sign bit set passed the float compare
      }
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) my_max = max(my_max, __shfl_xor_sync(kFull, my_max, d));
    if (lane == 0) atomicMax(&sh.cand_max, my_max);
    if (bad != 0u) sh.below_pivot = 1u;
  }
  __syncthreads();
  const uint32_t C = sh.cand_count;
  if (sh.below_pivot != 0u || C < (uint32_t)kk) {  // a NaN below the pivot, or the pivot came out above the k-th largest
    if (tid == 0) count_out[row] = -1;
    return;
  }
  // exact select over the candidates: first digit = top 12 bits of the candidates' actual spread
  const uint32_t range = sh.cand_max - pivot;
  const int s = max(0, 32 - __clz(range) - 12);  // range >> s < 4096
  for (uint32_t i = tid; i < C; i += kThreads) atomicAdd(&sh.hist[(sh.cand_key[i] - pivot) >> s], 1u);
  __syncthreads();
  scan_from_top<4096>(sh, sh.hist, (uint32_t)kk);
  const uint32_t b1 = sh.digit, k1 = sh.k_rem, cnt1 = sh.bin_count;
  if (cnt1 <= (uint32_t)kSmallBin) {
    for (uint32_t i = tid; i < C; i += kThreads) {
      const uint32_t key = sh.cand_key[i];
      if (((key - pivot) >> s) == b1) sh.small_key[atomicAdd(&sh.small_count, 1u)] = key;
    }
    __syncthreads();
    if (tid < kSmallBin && tid < (int)cnt1) {
      const uint32_t mine = sh.small_key[tid];
      uint32_t greater = 0, equal = 0;
      for (uint32_t j = 0; j < cnt1; ++j) {
        const uint32_t other = sh.small_key[j];
        greater += other > mine;
        equal += other == mine;
      }
      if (greater < k1 && k1 <= greater + equal) {
        sh.thr = mine;
        sh.need_eq = k1 - greater;
      }
    }
    __syncthreads();
  } else {
    uint32_t prefix = b1 << s, mask = s == 0 ? 0xffffffffu : ~((1u << s) - 1u), k_rem = k1;
    int rest = s;
#pragma unroll 1
    while (rest > 0) {
      const int wbits = min(10, rest), shift = rest - wbits;
      for (uint32_t i = tid; i < C; i += kThreads) {
        const uint32_t d = sh.cand_key[i] - pivot;
        if ((d & mask) == prefix) atomicAdd(&sh.hist10[(d >> shift) & ((1u << wbits) - 1u)], 1u);
      }
      __syncthreads();
      scan_from_top<1024>(sh, sh.hist10, k_rem);
      prefix |= sh.digit << shift;
      mask |= ((1u << wbits) - 1u) << shift;
      k_rem = sh.k_rem;
      rest = shift;
    }
    if (tid == 0) { sh.thr = pivot + prefix; sh.need_eq = k_rem; }
    __syncthreads();
  }
  const uint32_t thr = sh.thr, need_eq = sh.need_eq;  // every key > thr, and the need_eq lowest positions with key == thr
  // selected positions -> bitmap; threshold-equal ones are collected and, if not all are needed, ranked by position
  if (tid == 0) sh.small_count = 0u;  // reused: number of threshold-equal candidates
  __syncthreads();
  for (uint32_t i = tid; i < C; i += kThreads) {
    const uint32_t key = sh.cand_key[i], pos = sh.cand_pos[i];
    if (key > thr) atomicOr(&bitmap[pos >> 5], 1u << (pos & 31u));
    else if (key == thr) {
      const uint32_t at = atomicAdd(&sh.small_count, 1u);
      if (at < (uint32_t)kEqCap) eq_pos[at] = pos;
    }
  }
  __syncthreads();
  const uint32_t n_eq = sh.small_count;
  if (n_eq > (uint32_t)kEqCap) {  // a long run of equal scores at the threshold
    if (tid == 0) count_out[row] = -1;
    return;
  }
  for (uint32_t i = tid; i < n_eq; i += kThreads) {
    const uint32_t mine = eq_pos[i];
    uint32_t lower = 0;
    if (n_eq != need_eq)
      for (uint32_t j = 0; j < n_eq; ++j) lower += eq_pos[j] < mine;
    if (lower < need_eq) atomicOr(&bitmap[mine >> 5], 1u << (mine & 31u));
  }
  __syncthreads();
  {
    const int per = (words + kThreads - 1) / kThreads;  // consecutive bitmap words per thread
    const int w_lo = min(words, tid * per), w_hi = min(words, w_lo + per);
    uint32_t mine = 0;
    for (int w = w_lo; w < w_hi; ++w) mine += __popc(bitmap[w]);
    uint32_t off = block_excl_scan(sh, mine);
    for (int w = w_lo; w < w_hi; ++w) {
      uint32_t bits = bitmap[w];
      while (bits != 0u) {
        if (off < (uint32_t)kk) out[off] = (int32_t)(w * 32 + __ffs(bits) - 1);
        ++off;
        bits &= bits - 1u;
      }
    }
  }
  if (tid == 0) count_out[row] = kk;
  for (int i = kk + tid; i < top_k; i += kThreads) out[i] = -1;
}

}  // namespace

// Whether the one-sweep kernel can take this launch at all (the caller decides whether it should).
bool topk_prefilter_fits(const clsa_params& p, const float* scores, int64_t score_stride, const DeviceInfo& dev) {
  if (p.max_seq_len <= kCandCap) return false;               // short rows fit the general kernel's shared memory
  {
    // The candidate list must hold what the sampled pivot lets through on the longest row: the pivot sits at rank
    // r of the sample (the kernel's formula), so about n r / kSample scores pass it, give or take n sqrt(r) / kSample;
    // a launch whose rows would mostly overflow the list is better served by the general kernel from the start
    // (k = 4096 of 131072: 5960 +- 440 expected against 6144 slots).
    const double n = (double)p.max_seq_len, k = (double)(p.top_k < p.max_seq_len ? p.top_k : p.max_seq_len);
    const double expect = (double)kSample * k / n * 1.10;
    const double r = expect + 3.5 * sqrt(expect) + 4.0;
    if (n * (r + 2.5 * sqrt(r)) / (double)kSample > (double)kCandCap) return false;
  }
  if (score_stride % 4 != 0 || reinterpret_cast<uintptr_t>(scores) % 16 != 0) return false;
  const int bitmap_words = ((p.max_seq_len + 31) / 32 + 3) & ~3;
  const size_t smem = sizeof(FShared) + (size_t)bitmap_words * sizeof(uint32_t);
  const size_t half_sm = ((size_t)dev.max_smem_optin + 1024) / 2 - 1024;  // two blocks per SM
  return smem <= half_sm;                                    // longer rows do not fit the bitmaps
}

// Launches the one-sweep kernel (the shape must fit, see above). The caller follows up with the general kernel
// restricted to rows whose count is -1.
cudaError_t launch_topk_prefilter(const clsa_params& p, const float* scores, int64_t score_stride, int32_t* idx,
                                  int32_t* count, uint32_t* status, const DeviceInfo& dev, cudaStream_t stream) {
  (void)dev;
  const int64_t rows = (int64_t)p.num_seqs * p.q_per_seq;
  const int bitmap_words = ((p.max_seq_len + 31) / 32 + 3) & ~3;
  const size_t smem = sizeof(FShared) + (size_t)bitmap_words * sizeof(uint32_t);
  cudaError_t err = cudaFuncSetAttribute(topk_prefilter_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (err != cudaSuccess) return err;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)rows, 1, 1);
  cfg.blockDim = dim3(kThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, topk_prefilter_kernel, scores, score_stride, p.seq_len, (int)p.q_per_seq, (int)p.causal,
                            (int)p.top_k, (int)p.max_seq_len, bitmap_words, idx, count, status);
}

}  // namespace clsa

namespace clsa {

int topk_candidates_capacity() { return kCandCap; }

// Shared memory of topk_candidates_kernel for rows of up to max_seq_len positions (0 if it does not fit two blocks
// per SM).
size_t topk_candidates_smem(int max_seq_len, const DeviceInfo& dev) {
  const int bitmap_words = ((max_seq_len + 31) / 32 + 3) & ~3;
  const size_t smem = sizeof(FShared) + (size_t)kEqCap * sizeof(uint32_t) + (size_t)bitmap_words * sizeof(uint32_t);
  const size_t half_sm = ((size_t)dev.max_smem_optin + 1024) / 2 - 1024;
  return smem <= half_sm ? smem : 0;
}

cudaError_t launch_topk_candidates(const clsa_params& p, const uint2* cand, const uint32_t* cand_count, const float* pivot,
                                   int32_t* idx, int32_t* count, uint32_t* status, const DeviceInfo& dev, cudaStream_t stream) {
  const size_t smem = topk_candidates_smem(p.max_seq_len, dev);
  if (smem == 0) return cudaErrorInvalidValue;
  const int bitmap_words = ((p.max_seq_len + 31) / 32 + 3) & ~3;
  cudaError_t err = cudaFuncSetAttribute(topk_candidates_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (err != cudaSuccess) return err;
  const int64_t rows = (int64_t)p.num_seqs * p.q_per_seq;
  topk_candidates_kernel<<<(unsigned)rows, kThreads, smem, stream>>>(cand, cand_count, kCandCap, pivot, p.seq_len, p.q_per_seq,
                                                                     p.causal, p.top_k, p.max_seq_len, bitmap_words, idx, count,
                                                                     status);
  return cudaGetLastError();
}

}  // namespace clsa
