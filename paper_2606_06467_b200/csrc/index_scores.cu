// Index scores for decoding (Eq. 3, first half): one fp32 dot product per cached token, streamed
// once over the bf16 indexer-key cache. The kernel is bound by HBM bandwidth (1 flop per byte).
//
// Work split: the (sequence, 128-or-256-row tile) space goes to a persistent grid of 4 blocks per
// SM: the first three quarters of the tiles round-robin, the rest on demand from a ticket counter
// (blocks do not all run at the same pace -- with a fixed deal the last blocks finish well after
// the median one, time during which the memory system runs below capacity and the kernel behind
// this one waits). Inside a tile each warp owns a contiguous run of rows; a key row (d_idx bf16)
// is covered by d_idx/8 lanes holding 16 bytes each, and every thread keeps 8 independent 16-byte
// loads in flight (128 KiB per SM at 1024 resident threads), which is what it takes to cover the
// DRAM latency at full bandwidth. The per-row sum uses one fixed order (8 sequential FMAs per lane,
// then a butterfly over the lanes of the row) that does not depend on where the row sits, so rows
// with identical contents always get bit-identical scores -- the tie-break of the top-k relies on it.
#include "common.cuh"

namespace clsa {
namespace {

constexpr int kThreads = 256;
constexpr int kLoads = 8;  // independent 16-byte loads per thread per tile

template <int DIDX>
__global__ void __launch_bounds__(kThreads, 4)
index_scores_decode_kernel(const uint16_t* __restrict__ kidx, int64_t tok_stride, const uint16_t* __restrict__ q_idx,
                           const int64_t* __restrict__ seq_start, const int32_t* __restrict__ seq_len,
                           float* __restrict__ scores, int64_t score_stride, int num_seqs, int tiles_per_seq,
                           int max_seq_len, const int32_t* __restrict__ block_table, int block_shift, int max_blocks,
                           int64_t static_tiles, uint32_t* status, uint32_t* sched) {
  constexpr int LPR = DIDX / 8;               // lanes per key row
  constexpr int RPI = 32 / LPR;               // rows covered by one warp-wide load
  constexpr int ROWS_PER_WARP = RPI * kLoads;
  constexpr int TILE = ROWS_PER_WARP * (kThreads / 32);

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int sub = lane / LPR;                 // which of the RPI rows of a load this lane reads
  const int col = (lane % LPR) * 8;           // first element of this lane's 16 bytes
  const int64_t total_tiles = (int64_t)num_seqs * tiles_per_seq;

  // let a dependent launch (the top-k) be scheduled onto SMs as this grid's blocks retire
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  int cur_b = -1;
  float q[8];
  auto process = [&](const int64_t tile) {
    const int b = (int)(tile / tiles_per_seq);
    const int row0 = (int)(tile % tiles_per_seq) * TILE + warp * ROWS_PER_WARP;
    const int n = seq_len[b];
    if (n < 1 || n > max_seq_len) {
      if (threadIdx.x == 0 && row0 == 0) flag_status(status, CLSA_DEV_BAD_SEQLEN);
      return;
    }
    if (row0 >= n) return;
    if (b != cur_b) {
      const uint4 qw = *reinterpret_cast<const uint4*>(q_idx + (int64_t)b * DIDX + col);
      q[0] = bf16_lo(qw.x); q[1] = bf16_hi(qw.x); q[2] = bf16_lo(qw.y); q[3] = bf16_hi(qw.y);
      q[4] = bf16_lo(qw.z); q[5] = bf16_hi(qw.z); q[6] = bf16_lo(qw.w); q[7] = bf16_hi(qw.w);
      cur_b = b;
    }
    uint4 kw[kLoads];
    if (block_table == nullptr) {
      const uint16_t* base = kidx + (seq_start[b] + row0 + sub) * tok_stride + col;
#pragma unroll
      for (int u = 0; u < kLoads; ++u) {
        const int r = row0 + u * RPI + sub;
        kw[u] = r < n ? __ldcs(reinterpret_cast<const uint4*>(base + (int64_t)u * RPI * tok_stride)) : make_uint4(0, 0, 0, 0);
      }
    } else if ((1 << block_shift) >= ROWS_PER_WARP) {
      // paged cache whose blocks hold at least a warp's run of rows (which starts on a multiple of its length): the
      // run lies in one block, so one lookup gives a base pointer and the loads are the strided ones of the contiguous
      // layout (a lookup and a 64-bit product per load cost registers, and with them loads in flight)
      const int32_t* table = block_table + (int64_t)b * max_blocks;
      const int64_t blk = __ldg(table + (row0 >> block_shift));  // row0 < n: this block exists
      const uint16_t* base = kidx + ((blk << block_shift) + ((row0 + sub) & ((1 << block_shift) - 1))) * tok_stride + col;
#pragma unroll
      for (int u = 0; u < kLoads; ++u) {
        const int r = row0 + u * RPI + sub;
        kw[u] = r < n ? __ldcs(reinterpret_cast<const uint4*>(base + (int64_t)u * RPI * tok_stride)) : make_uint4(0, 0, 0, 0);
      }
    } else {
      // paged cache: position r lives in block table[b][r >> shift] at offset r & (block_size - 1)
      const int32_t* table = block_table + (int64_t)b * max_blocks;
      int64_t prow[kLoads];
#pragma unroll
      for (int u = 0; u < kLoads; ++u) {
        const int r = row0 + u * RPI + sub;
        prow[u] = r < n ? ((int64_t)__ldg(table + (r >> block_shift)) << block_shift) + (r & ((1 << block_shift) - 1)) : 0;
      }
#pragma unroll
      for (int u = 0; u < kLoads; ++u) {
        const int r = row0 + u * RPI + sub;
        kw[u] = r < n ? __ldcs(reinterpret_cast<const uint4*>(kidx + prow[u] * tok_stride + col)) : make_uint4(0, 0, 0, 0);
      }
    }
    float v[kLoads];
#pragma unroll
    for (int u = 0; u < kLoads; ++u) {
      float a = bf16_lo(kw[u].x) * q[0];
      a = fmaf(bf16_hi(kw[u].x), q[1], a);
      a = fmaf(bf16_lo(kw[u].y), q[2], a);
      a = fmaf(bf16_hi(kw[u].y), q[3], a);
      a = fmaf(bf16_lo(kw[u].z), q[4], a);
      a = fmaf(bf16_hi(kw[u].z), q[5], a);
      a = fmaf(bf16_lo(kw[u].w), q[6], a);
      a = fmaf(bf16_hi(kw[u].w), q[7], a);
      v[u] = a;
    }
    // Transposing butterfly over the LPR lanes of a row: each step halves the number of values a
    // lane carries while summing lane pairs, so 8 rows cost 8 shuffles (LPR = 16) instead of 32.
    // Which lane pair is summed at each level is the same for every row: the order is fixed.
    int nv = kLoads, u_of_lane = 0;
    bool writer = true;
#pragma unroll
    for (int m = LPR / 2; m >= 1; m >>= 1) {
      const bool hi = (lane & m) != 0;
      if (nv > 1) {
        const int half = nv / 2;
#pragma unroll
        for (int i = 0; i < half; ++i) {
          const float send = hi ? v[i] : v[i + half];
          const float keep = hi ? v[i + half] : v[i];
          v[i] = keep + __shfl_xor_sync(0xffffffffu, send, m);
        }
        u_of_lane += hi ? half : 0;
        nv = half;
      } else {
        v[0] += __shfl_xor_sync(0xffffffffu, v[0], m);
        writer = writer && !hi;
      }
    }
    const int r = row0 + u_of_lane * RPI + sub;
    if (writer && r < n) scores[(int64_t)b * score_stride + r] = v[0];
  };

  // Tiles below static_tiles (a multiple of the grid size) are dealt round-robin; no block waits for another.
  for (int64_t tile = blockIdx.x; tile < static_tiles; tile += gridDim.x) process(tile);
  if (static_tiles >= total_tiles) return;

  // The rest on demand. sched[0] hands out tickets, sched[1] counts the blocks that have drawn their last one;
  // both are zero between launches (the block that finishes last puts them back). Thread 0 draws the ticket for the
  // tile after the current one before the current one is processed, so the draw's latency hides behind the tile.
  __shared__ int64_t next_tile[2];
  // Every block draws exactly one ticket past the end, so a ticket beyond total + grid means that the counters were
  // not zero when the launch began (a workspace header that was never cleared): tiles have been skipped.
  auto draw = [&]() -> int64_t {
    const int64_t t = static_tiles + (int64_t)atomicAdd(&sched[0], 1u);
    if (t >= total_tiles + (int64_t)gridDim.x) flag_status(status, CLSA_DEV_BAD_WORKSPACE);
    return t;
  };
  if (threadIdx.x == 0) next_tile[0] = draw();
  __syncthreads();
  int buf = 0;
  while (true) {
    const int64_t tile = next_tile[buf];
    if (tile >= total_tiles) break;  // the same for every thread of the block
    int64_t drawn = 0;
    if (threadIdx.x == 0) drawn = draw();
    process(tile);
    if (threadIdx.x == 0) next_tile[buf ^ 1] = drawn;
    __syncthreads();  // the next ticket is visible, and nobody still reads the current one
    buf ^= 1;
  }
  if (threadIdx.x == 0) {
    // This block draws no more tickets. Once every block has said so the counters can go back to zero for the
    // next launch on this workspace (launches that share a workspace do not overlap).
    __threadfence();
    if (atomicAdd(&sched[1], 1u) == gridDim.x - 1) {
      sched[0] = 0u;
      sched[1] = 0u;
    }
  }
}

}  // namespace

cudaError_t launch_index_scores_decode(const clsa_params& p, const void* q_idx, float* scores, int64_t score_stride,
                                       uint32_t* status, uint32_t* sched, const DeviceInfo& dev, cudaStream_t stream) {
  const int lpr = p.idx_dim / 8;
  const int tile = (32 / lpr) * kLoads * (kThreads / 32);
  const int tiles_per_seq = (p.max_seq_len + tile - 1) / tile;
  const int64_t total = (int64_t)p.num_seqs * tiles_per_seq;
  int64_t grid = (int64_t)dev.sm_count * 4;
  if (grid > total) grid = total;
  // three quarters of the tiles by a fixed deal (whole rounds of the grid), the rest on demand: a larger on-demand
  // share balances the end of the launch better, but tiles past the end of a short sequence cost nothing in the fixed
  // deal and a draw from the one counter on demand, which a ragged batch notices. Launches with only a few tiles per
  // block are dealt whole.
  int64_t static_tiles = total;
  if (total >= 8 * grid) static_tiles = (total * 3 / 4) / grid * grid;
  auto kidx = static_cast<const uint16_t*>(p.idx_k_cache);
  auto q = static_cast<const uint16_t*>(q_idx);
  int block_shift = 0;
  while (p.block_table != nullptr && (1 << block_shift) < p.block_size) ++block_shift;
  if (p.idx_dim == 128) {
    index_scores_decode_kernel<128><<<(unsigned)grid, kThreads, 0, stream>>>(
        kidx, p.idx_token_stride, q, p.seq_start, p.seq_len, scores, score_stride, p.num_seqs, tiles_per_seq,
        p.max_seq_len, p.block_table, block_shift, p.max_blocks_per_seq, static_tiles, status, sched);
  } else {
    index_scores_decode_kernel<64><<<(unsigned)grid, kThreads, 0, stream>>>(
        kidx, p.idx_token_stride, q, p.seq_start, p.seq_len, scores, score_stride, p.num_seqs, tiles_per_seq,
        p.max_seq_len, p.block_table, block_shift, p.max_blocks_per_seq, static_tiles, status, sched);
  }
  return cudaGetLastError();
}

}  // namespace clsa
