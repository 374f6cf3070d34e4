// Scores and TopK of a prefill chunk in one go (Eq. 3, both halves, T > 1 queries per sequence), with the T x n score
// matrix never written to memory.
//
// Materialised, the scores of a 4096-query chunk over a 128K-token cache are 2.2 GB that one kernel writes and the
// next reads back, where the operands (34 MB of keys) and the result (33 MB of indices) are sixty times smaller. Here
// the contraction runs twice on the tensor cores instead -- once over a sample of the keys, once over all of them --
// and only candidates leave the SMs:
//   1. sample   the chunk GEMM over 16-position groups spread evenly over the cache (about 4096 positions per
//               sequence) writes a small sample of every row's scores;
//   2. pivot    one warp per row finds, by bisection over the key bits, the sample's r-th largest score, r chosen so
//               that the pivot lies below the row's k-th largest score with a margin of several standard deviations;
//   3. filter   the chunk GEMM over all keys, its epilogue comparing every score in registers with the row's pivot
//               and appending the few that are not below it, as (score, position) pairs, to the row's list;
//   4. select   exact TopK of every row from its list (topk_candidates_kernel), positions ascending, ties to the
//               lower position: the same result as a selection over the full row, because the list holds every score
//               that can matter;
//   5. rest     rows whose list cannot give the exact answer (pivot too high, list overflowed by long runs of equal
//               scores, NaNs) are numbered, their scores are recomputed by the same tensor-core kernel into a small
//               scratch matrix, and the general top-k kernel finishes them: bit for bit what clsa_index_scores +
//               clsa_topk give. If more rows need this than the scratch holds, the surplus rows get count 0 and
//               CLSA_DEV_ROUTING_OVERFLOW is raised.
#include <math.h>

#include "common.cuh"

namespace clsa {
namespace {

constexpr int kSampleTarget = 4096;   // sampled positions per sequence (16 x the number of groups)
constexpr int kSamplePerLane = kSampleTarget / 32;
constexpr int kHandBackRows = 64;     // rows of scratch for step 5

__device__ __forceinline__ uint32_t score_key(float x) {
  uint32_t u = __float_as_uint(x);
  if (u == 0x80000000u) u = 0u;  // -0.0 ranks equal to +0.0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_score(uint32_t key) {  // inverse of score_key
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// Step 2. One warp per (sequence, query) row. Column j of the sample stands for position (j / 16) * gs + j % 16.
__global__ void __launch_bounds__(128)
chunk_pivot_kernel(const float* __restrict__ sample, int64_t sample_stride, int sample_gs, const int32_t* __restrict__ seq_len,
                   int q_per_seq, int causal, int top_k, int max_seq_len, int whole_row_cap, int64_t rows,
                   float* __restrict__ pivot) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows) return;
  const int b = (int)(row / q_per_seq), t = (int)(row % q_per_seq);
  const int n = seq_len[b];
  const float kInf = __int_as_float(0x7f800000);
  if (n < q_per_seq || n > max_seq_len) {  // the select flags the sequence
    if (lane == 0) pivot[row] = kInf;
    return;
  }
  const int v = causal ? n - q_per_seq + t + 1 : n;
  const int kk = min(top_k, v);
  if (kk == v) {            // every visible position is selected: no candidates needed
    if (lane == 0) pivot[row] = kInf;
    return;
  }
  if (v <= whole_row_cap) {  // the whole row fits the candidate list, holes included
    if (lane == 0) pivot[row] = -kInf;
    return;
  }
  const int cols = (n / sample_gs) * 16;  // sampled columns of this sequence (whole groups only)
  const float* src = sample + row * sample_stride;
  uint32_t key[kSamplePerLane];
  int m_v = 0;  // visible samples held by this lane
#pragma unroll
  for (int i = 0; i < kSamplePerLane; ++i) {
    const int j = lane + 32 * i;
    const int pos = (j >> 4) * sample_gs + (j & 15);
    const bool vis = j < cols && pos < v;
    key[i] = vis ? score_key(src[j]) : 0u;  // 0 ranks below every score, and is never counted for a candidate >= 2^16
    m_v += vis ? 1 : 0;
  }
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) m_v += __shfl_xor_sync(0xffffffffu, m_v, d);
  // rank of the pivot inside the sample: the expected number of sampled scores among the row's k largest, plus 10 %
  // and 3.5 standard deviations of that count
  const float expect = (float)m_v * (float)kk / (float)v * 1.10f;
  const int r = (int)(expect + 3.5f * sqrtf(expect) + 4.0f);
  if (r >= m_v) {  // the sample cannot place the pivot: everything is a candidate (and the row is handed back if that overflows)
    if (lane == 0) pivot[row] = -kInf;
    return;
  }
  // the largest 16-bit prefix P (sign, exponent, 7 mantissa bits: a pivot at most 0.8 % below the sample's r-th
  // largest score) with at least r sampled keys >= P
  uint32_t P = 0u;
#pragma unroll 1
  for (int bit = 31; bit >= 16; --bit) {
    const uint32_t c = P | (1u << bit);
    int cnt = 0;
#pragma unroll
    for (int i = 0; i < kSamplePerLane; ++i) cnt += key[i] >= c ? 1 : 0;
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, d);
    if (cnt >= r) P = c;
  }
  float pv = key_score(P);
  if (pv != pv) pv = -kInf;  // a NaN pattern cannot be compared against
  if (lane == 0) pivot[row] = pv;
}

// Step 5a. Rows that the select could not finish get a scratch row each (as long as there are any).
__global__ void chunk_hand_back_kernel(int64_t rows, int q_per_seq, int m_blocks, int top_k, int max_slots,
                                       int32_t* __restrict__ count, int32_t* __restrict__ idx, int32_t* __restrict__ slot_of_row,
                                       int32_t* __restrict__ row_of_slot, uint32_t* __restrict__ nslots,
                                       uint32_t* __restrict__ qblock_flag, uint32_t* status) {
  const int64_t row = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= rows || count[row] != -1) return;
  const uint32_t slot = atomicAdd(nslots, 1u);
  if (slot < (uint32_t)max_slots) {
    slot_of_row[row] = (int32_t)slot;
    row_of_slot[slot] = (int32_t)row;
    const int b = (int)(row / q_per_seq), t = (int)(row % q_per_seq);
    qblock_flag[b * m_blocks + t / 128] = 1u;
  } else {
    count[row] = 0;
    for (int i = 0; i < top_k; ++i) idx[row * top_k + i] = -1;
    flag_status(status, CLSA_DEV_ROUTING_OVERFLOW);
  }
}

// Caps the slot counter at the scratch's size (the kernels behind read it as "rows handed back").
__global__ void chunk_cap_slots_kernel(uint32_t* nslots, int max_slots) {
  if (*nslots > (uint32_t)max_slots) *nslots = (uint32_t)max_slots;
}

struct Layout {
  int sample_gs;
  int64_t sample_stride;
  int cand_cap;
  size_t pivot, cand_count, slot_of_row, row_of_slot, nslots, qflags, sample, cand, fb_scores, total;
  size_t zero_begin, zero_end;  // counters that start at zero
};

Layout make_layout(const clsa_params& p) {
  Layout l;
  auto align = [](size_t x) { return (x + 255) / 256 * 256; };
  const size_t rows = (size_t)p.num_seqs * p.q_per_seq;
  const int m_blocks = (p.q_per_seq + 127) / 128;
  l.sample_gs = 16 * ((p.max_seq_len + kSampleTarget - 1) / kSampleTarget);
  const int cols = (p.max_seq_len / l.sample_gs) * 16;
  l.sample_stride = ((int64_t)(cols > 0 ? cols : 16) + 63) / 64 * 64;
  l.cand_cap = topk_candidates_capacity();
  size_t at = 0;
  l.pivot = at; at = align(at + rows * 4);
  l.slot_of_row = at; at = align(at + rows * 4);
  l.zero_begin = at;
  l.cand_count = at; at = align(at + rows * 4);
  l.row_of_slot = at; at = align(at + (size_t)kHandBackRows * 4);
  l.nslots = at; at = align(at + 4);
  l.qflags = at; at = align(at + (size_t)p.num_seqs * m_blocks * 4);
  l.zero_end = at;
  l.sample = at; at = align(at + rows * (size_t)l.sample_stride * 4);
  l.cand = at; at = align(at + rows * (size_t)l.cand_cap * 8);
  const size_t score_stride = ((size_t)p.max_seq_len + 63) / 64 * 64;
  l.fb_scores = at; at = align(at + (size_t)kHandBackRows * score_stride * 4);
  l.total = at;
  return l;
}

}  // namespace

size_t index_topk_scratch_bytes(const clsa_params& p) { return make_layout(p).total; }

bool index_topk_fits(const clsa_params& p, const DeviceInfo& dev) {
  if (p.q_per_seq < 2) return false;
  if (topk_candidates_smem(p.max_seq_len, dev) == 0) return false;  // rows too long for the select's position bitmap
  // The candidate list must hold what the pivot is expected to let through on the longest row, give or take 2.5
  // standard deviations (the pivot sits at rank r of about kSampleTarget samples: about n r / samples scores pass).
  const double n = (double)p.max_seq_len, k = (double)(p.top_k < p.max_seq_len ? p.top_k : p.max_seq_len);
  // what the filter may leave of a list as holes comes off its capacity
  const double cap = (double)topk_candidates_capacity() - (double)index_gemm_filter_hole_slack(p, dev);
  if (n <= cap) return true;
  const double samples = n < kSampleTarget ? n : (double)kSampleTarget;
  const double expect = samples * k / n * 1.10;
  const double r = expect + 3.5 * sqrt(expect) + 4.0;
  return n * (r + 2.5 * sqrt(r)) / samples <= cap;
}

cudaError_t launch_index_topk(const clsa_params& p, const void* q_idx, int32_t* idx, int32_t* count, unsigned char* scratch,
                              uint32_t* status, const DeviceInfo& dev, cudaStream_t stream) {
  const Layout l = make_layout(p);
  const int64_t rows = (int64_t)p.num_seqs * p.q_per_seq;
  const int m_blocks = (p.q_per_seq + 127) / 128;
  auto pivot = reinterpret_cast<float*>(scratch + l.pivot);
  auto cand_count = reinterpret_cast<uint32_t*>(scratch + l.cand_count);
  auto slot_of_row = reinterpret_cast<int32_t*>(scratch + l.slot_of_row);
  auto row_of_slot = reinterpret_cast<int32_t*>(scratch + l.row_of_slot);
  auto nslots = reinterpret_cast<uint32_t*>(scratch + l.nslots);
  auto qflags = reinterpret_cast<uint32_t*>(scratch + l.qflags);
  auto sample = reinterpret_cast<float*>(scratch + l.sample);
  auto cand = reinterpret_cast<uint2*>(scratch + l.cand);
  auto fb_scores = reinterpret_cast<float*>(scratch + l.fb_scores);
  const int64_t score_stride = ((int64_t)p.max_seq_len + 63) / 64 * 64;

  cudaError_t err = cudaMemsetAsync(scratch + l.zero_begin, 0, l.zero_end - l.zero_begin, stream);
  if (err != cudaSuccess) return err;
  err = cudaMemsetAsync(slot_of_row, 0xff, (size_t)rows * 4, stream);  // -1: no slot
  if (err != cudaSuccess) return err;
  // 1. sample, 2. pivot
  err = launch_index_gemm_sample(p, q_idx, sample, l.sample_stride, l.sample_gs, status, dev, stream);
  if (err != cudaSuccess) return err;
  chunk_pivot_kernel<<<(unsigned)((rows + 3) / 4), 128, 0, stream>>>(sample, l.sample_stride, l.sample_gs, p.seq_len, p.q_per_seq,
                                                                     p.causal, p.top_k, p.max_seq_len,
                                                                     l.cand_cap - index_gemm_filter_hole_slack(p, dev), rows, pivot);
  if ((err = cudaGetLastError()) != cudaSuccess) return err;
  // 3. filter, 4. select
  GemmFused fx = {pivot, cand, cand_count, l.cand_cap, slot_of_row, qflags, nslots};
  err = launch_index_gemm_filter(p, q_idx, fx, status, dev, stream);
  if (err != cudaSuccess) return err;
  err = launch_topk_candidates(p, cand, cand_count, pivot, idx, count, status, dev, stream);
  if (err != cudaSuccess) return err;
  // 5. the rows the select handed back
  chunk_hand_back_kernel<<<(unsigned)((rows + 255) / 256), 256, 0, stream>>>(rows, p.q_per_seq, m_blocks, p.top_k, kHandBackRows,
                                                                             count, idx, slot_of_row, row_of_slot, nslots, qflags,
                                                                             status);
  if ((err = cudaGetLastError()) != cudaSuccess) return err;
  chunk_cap_slots_kernel<<<1, 1, 0, stream>>>(nslots, kHandBackRows);
  if ((err = cudaGetLastError()) != cudaSuccess) return err;
  err = launch_index_gemm_handed_back(p, q_idx, fb_scores, score_stride, fx, status, dev, stream);
  if (err != cudaSuccess) return err;
  return launch_topk_slots(p, fb_scores, score_stride, row_of_slot, nslots, kHandBackRows, idx, count, status, dev, stream);
}

}  // namespace clsa
