// Index scores for a prefill chunk (Eq. 3, first half, T > 1 queries per sequence): a dense
// bf16 x bf16 -> fp32 contraction  scores[t][s] = sum_j Q_idx[t][j] * K_idx[s][j]  on the
// 5th-generation tensor cores.
//
// Shape of the problem: M = T queries (4096), N = cached tokens (135168), K = d_idx (64 or 128).
// K is tiny, so the kernel is bound by writing the fp32 scores, not by the MMAs; the design keeps
// the tensor pipe and the store path busy at the same time rather than chasing MMA peak.
//
// One persistent block per SM walks output tiles of 128 queries x 256 keys (query block fastest,
// so neighbouring SMs share a key tile in L2). Warp roles:
//   warp 0           : TMA producer. Per tile, 2 + 2 tiled bulk copies (128-byte swizzle) bring the
//                      128 x d_idx query tile and the 256 x d_idx key tile into a 2-stage ring. With a
//                      paged key cache the key tile is assembled from one box per cache block (blocks of
//                      16..128 rows; every box starts on a 1024-byte swizzle atom, so the assembled tile
//                      has the layout of a single 256-row box).
//   warp 1, one lane : MMA issuer. d_idx/16 tcgen05.mma (M128 N256 K16, kind::f16, bf16 inputs, fp32
//                      accumulate) per tile into one of two 256-column TMEM accumulators;
//                      tcgen05.commit frees the smem stage and publishes the accumulator.
//   warp 2           : allocates / frees the 512 TMEM columns.
//   warps 4..11      : epilogue. Two warps per 32 TMEM lanes (= 32 query rows), 128 columns each: tcgen05.ld 32
//                      columns at a time (double-buffered) into a swizzled shared-memory tile; chunks that
//                      every query of the warp may see leave as one tiled bulk store, the others (causal
//                      diagonal, end of a sequence) as masked 32-byte stores, four lanes per row. The
//                      epilogue of tile i overlaps the MMAs of tile i+1. The filtering mode of clsa_index_topk
//                      runs warps 4..19 instead: four per 32 TMEM lanes, 64 columns each, 16 at a time.
// Tiles that lie entirely above the causal diagonal are skipped by every role alike.
// Every mbarrier wait is bounded: on expiry the block raises CLSA_DEV_TIMEOUT in the status word,
// all roles leave their loops, in-flight copies are given time to land, TMEM is freed, and the
// kernel returns.
#include <cuda.h>

#include "common.cuh"

namespace clsa {
namespace {

constexpr int kBM = 128, kBN = 256, kBK = 64;  // tile; kBK bf16 = one 128-byte swizzle row
constexpr int kStages = 2, kAccBufs = 2;
// Epilogue warps: two per TMEM lane quadrant with 128 columns each where the scores are stored; four per quadrant with
// 64 columns each in the filtering mode, whose epilogue is a chain of dependent instructions per warp (twice the warps
// hide twice the latency; its 16-column register buffers keep 640 threads within the register file).
__host__ __device__ constexpr int epi_warps(int mode) { return mode == 1 ? 16 : 8; }
__host__ __device__ constexpr int gemm_threads(int mode) { return (4 + epi_warps(mode)) * 32; }
constexpr int kABytes = kBM * kBK * 2;          // one k-block of the query tile (16 KiB)
constexpr int kBBytes = kBN * kBK * 2;          // one k-block of the key tile (32 KiB)
constexpr int kStageBytes = 2 * kABytes + 2 * kBBytes;  // up to two k-blocks each (96 KiB)
constexpr int kBarrierBytes = 128;
constexpr int kEpiTileBytes = 8 * 4096;          // a 32 x 32 fp32 tile per storing warp (128-byte rows, 128-byte swizzle) or a 32 x 16 one per filtering warp
constexpr size_t kSmemBytes = (size_t)kStages * kStageBytes + kBarrierBytes + kEpiTileBytes + 1024;  // + alignment slack
constexpr uint32_t kSpinLimit = 1u << 22;       // polls with back-off: a few seconds at most
constexpr uint32_t kFilterRun = 8;              // slots of a candidate list that a lane reserves at a time

struct GemmArgs {
  const int64_t* seq_start;
  const int32_t* seq_len;
  float* scores;
  int64_t score_stride;
  uint32_t* status;
  int num_seqs, q_per_seq, causal, max_seq_len, idx_dim;
  int m_blocks, n_tiles;
  int vec_ok;  // rows of `scores` are 32-byte aligned: 256-bit stores and tiled bulk stores allowed
  // paged key cache: a 256-key tile is fetched as key_boxes boxes of box_rows rows, one per cache block
  // (block_size < 256), or as one box inside a block (block_size >= 256). Contiguous: one box, no table.
  const int32_t* block_table;
  int block_size, max_blocks_per_seq, box_rows, key_boxes;
  // Sampling (sample_gs > 0): the "keys" of this launch are groups of 16 consecutive positions spaced sample_gs
  // positions apart (a multiple of 16), column j of the output standing for position (j / 16) * sample_gs + j % 16;
  // only groups that lie wholly inside a sequence count, and every query sees all of them (the caller applies the
  // causal rule when it reads the sample). A key tile is then sixteen 16-row boxes, like a paged tile.
  int sample_gs;
  // Tile order. 0: query block fastest, tiles dealt round-robin (neighbouring SMs share a key tile in L2).
  // 1: key tile fastest and every block takes one contiguous run of tiles, so that a block stays on the same 128
  // queries for a long time (the filtering epilogue keeps per-query state between tiles).
  int row_major;
  // MODE 1 (filter): per query row, the score below which a key cannot be among the k largest; keys at or above it
  // are appended as (score bits, position) pairs to the row's candidate list.
  const float* pivot;
  uint2* cand;
  uint32_t* cand_count;
  int cand_cap;
  // MODE 2 (rows handed back): only query blocks with a set flag are computed, and only rows with a slot are stored,
  // row `slot` of `scores`.
  const int32_t* slot_of_row;
  const uint32_t* qblock_flag;
  const uint32_t* nslots;
};

// ---- PTX wrappers ----------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait. Returns false if the limit ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 63u) {
      if (*abort_flag != 0u) return false;
      __nanosleep(64);
    }
  }
  *abort_flag = 1u;
  return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// 16 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, K-major operand, 128-byte swizzle: 8-row groups are 1024 bytes
// apart (stride byte offset), the leading byte offset is unused inside one swizzle row.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3ffffu) >> 4);        // start address, 16-byte units
  d |= (uint64_t)(1024u >> 4) << 32;               // stride byte offset
  d |= (uint64_t)1 << 46;                          // descriptor version (sm_100)
  d |= (uint64_t)2 << 61;                          // layout: 128-byte swizzle
  return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, N and M encoded as N/8 and M/16.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int m, int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

struct TileCoord {
  int b, mb, nt, n, valid;
};
// The same enumeration for every role: tile id -> (sequence, query block, key tile); valid == 0 for
// tiles of a sequence with a bad length and for tiles wholly above the causal diagonal.
template <int MODE>
__device__ __forceinline__ TileCoord tile_coord(const GemmArgs& a, int64_t id) {
  TileCoord c;
  const int per_seq = a.m_blocks * a.n_tiles;
  c.b = (int)(id / per_seq);
  const int rem = (int)(id - (int64_t)c.b * per_seq);
  if (a.row_major) {
    c.mb = rem / a.n_tiles;
    c.nt = rem - c.mb * a.n_tiles;
  } else {
    c.nt = rem / a.m_blocks;
    c.mb = rem - c.nt * a.m_blocks;
  }
  c.n = a.seq_len[c.b];
  const bool n_ok = c.n >= a.q_per_seq && c.n <= a.max_seq_len;
  if (a.sample_gs > 0) c.n = n_ok ? (c.n / a.sample_gs) * 16 : 0;  // sampled columns: whole groups inside the sequence
  const int t_last = min(a.q_per_seq, (c.mb + 1) * kBM) - 1;
  const int v_max = (a.causal && a.sample_gs == 0) ? c.n - a.q_per_seq + t_last + 1 : c.n;
  c.valid = (n_ok && c.nt * kBN < v_max) ? 1 : 0;
  if (MODE == 2 && c.valid) c.valid = a.qblock_flag[c.b * a.m_blocks + c.mb] != 0u ? 1 : 0;
  return c;
}

// MODE 0: the scores are stored (clsa_index_scores; also the sampling pass of clsa_index_topk).
// MODE 1: the scores are compared with a per-row pivot in registers and only candidates leave the SM (clsa_index_topk).
// MODE 2: MODE 0 for the few rows that clsa_index_topk hands back, into a small scratch matrix.
template <int MODE>
__global__ void __launch_bounds__(gemm_threads(MODE), 1)
index_scores_gemm_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                         const __grid_constant__ CUtensorMap map_s, const GemmArgs a) {
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t raw = smem_u32(smem_dyn);
  const uint32_t base = (raw + 1023u) & ~1023u;  // 128-byte swizzle wants 1024-byte aligned tiles
  unsigned char* base_ptr = smem_dyn + (base - raw);
  const uint32_t bars = base + kStages * kStageBytes + kEpiTileBytes;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 16u + 8u * s; };
  auto tfull_bar = [&](int i) { return bars + 32u + 8u * i; };
  auto tempty_bar = [&](int i) { return bars + 48u + 8u * i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + kStages * kStageBytes + kEpiTileBytes + 64);
  volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(base_ptr + kStages * kStageBytes + kEpiTileBytes + 68);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr int kEpi = epi_warps(MODE);
  constexpr int kColsPerWarp = kBN / (kEpi / 4);  // columns of a tile that one epilogue warp drains
  const int kblocks = a.idx_dim / kBK;  // 1 or 2
  const bool causal = a.causal != 0 && a.sample_gs == 0;
  const int64_t total_tiles = (int64_t)a.num_seqs * a.m_blocks * a.n_tiles;
  // this block's tiles: first, first + step, ... below last
  const int64_t per_block = (total_tiles + gridDim.x - 1) / gridDim.x;
  const int64_t tile_first = a.row_major ? (int64_t)blockIdx.x * per_block : (int64_t)blockIdx.x;
  const int64_t tile_step = a.row_major ? 1 : (int64_t)gridDim.x;
  const int64_t tile_last = a.row_major ? min(total_tiles, tile_first + per_block) : total_tiles;
  if (MODE == 2 && *a.nslots == 0u) return;  // nothing was handed back (the usual case): before any barrier or TMEM use

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int i = 0; i < kAccBufs; ++i) { mbar_init(tfull_bar(i), 1); mbar_init(tempty_bar(i), kEpi); }
    *abort_flag = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(bars + 64u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    // Lane 0 owns the barriers and the query tile; key boxes are spread over the lanes (lane i fetches box i),
    // so that a tile made of sixteen 16-row cache blocks does not queue 32 copies behind one thread.
    uint32_t it = 0;
    for (int64_t id = tile_first; id < tile_last; id += tile_step) {
      const TileCoord c = tile_coord<MODE>(a, id);
      if (!c.valid) continue;
      const int s = it % kStages;
      const uint32_t ph = (it / kStages) & 1u;
      // first cache row of this lane's key box (looked up before the wait, used after it)
      int krow = 0, boxes = 1;
      if (a.sample_gs > 0) {
        // sixteen 16-row groups, sample_gs positions apart; groups past the sequence's last whole one are not fetched
        const int group = c.nt * 16 + lane;
        boxes = min(16, c.n / 16 - c.nt * 16);
        if (lane < boxes) {
          const int pos = group * a.sample_gs;
          if (a.block_table == nullptr) krow = (int)(a.seq_start[c.b] + pos);
          else krow = a.block_table[(int64_t)c.b * a.max_blocks_per_seq + pos / a.block_size] * a.block_size + pos % a.block_size;
        }
      } else if (a.block_table == nullptr) {
        krow = (int)(a.seq_start[c.b] + (int64_t)c.nt * kBN);
      } else {
        const int32_t* tab = a.block_table + (int64_t)c.b * a.max_blocks_per_seq;
        const int pos0 = c.nt * kBN;
        if (a.block_size >= kBN) {
          krow = tab[pos0 / a.block_size] * a.block_size + pos0 % a.block_size;
        } else {
          // only blocks that hold positions of the sequence: entries past them need not be valid
          boxes = min(a.key_boxes, (c.n - pos0 + a.block_size - 1) / a.block_size);
          if (lane < boxes) krow = tab[pos0 / a.block_size + lane] * a.block_size;
        }
      }
      int ok = 1;
      if (lane == 0) ok = mbar_wait(empty_bar(s), ph ^ 1u, abort_flag) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      const uint32_t st = base + s * kStageBytes;
      const uint32_t box_bytes = (uint32_t)a.box_rows * kBK * 2;
      if (lane == 0) {
        mbar_expect_tx(full_bar(s), (uint32_t)kblocks * (kABytes + (uint32_t)boxes * box_bytes));
        const int qrow = c.b * a.q_per_seq + c.mb * kBM;
        for (int kb = 0; kb < kblocks; ++kb) tma_load_2d(st + kb * kABytes, &map_q, kb * kBK, qrow, full_bar(s));
      }
      __syncwarp();  // the expected byte count is posted before any key box can complete
      if (lane < boxes)  // rows of boxes that are not fetched keep stale bits: their columns are never stored
        for (int kb = 0; kb < kblocks; ++kb)
          tma_load_2d(st + 2 * kABytes + kb * kBBytes + lane * box_bytes, &map_k, kb * kBK, krow, full_bar(s));
      ++it;
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc_bf16(kBM, kBN);
      uint32_t it = 0;
      for (int64_t id = tile_first; id < tile_last; id += tile_step) {
        const TileCoord c = tile_coord<MODE>(a, id);
        if (!c.valid) continue;
        const int s = it % kStages, acc = it % kAccBufs;
        const uint32_t ph = (it / kStages) & 1u, aph = (it / kAccBufs) & 1u;
        if (!mbar_wait(tempty_bar(acc), aph ^ 1u, abort_flag)) break;
        if (!mbar_wait(full_bar(s), ph, abort_flag)) break;
        tc_fence_after();
        const uint32_t st = base + s * kStageBytes;
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kBN);
        for (int kb = 0; kb < kblocks; ++kb) {
          const uint64_t adesc = smem_desc_sw128(st + kb * kABytes);
          const uint64_t bdesc = smem_desc_sw128(st + 2 * kABytes + kb * kBBytes);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) {
            // 16 bf16 = 32 bytes further along K inside the swizzle row: +2 in 16-byte address units
            tc_mma_bf16(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, (kb | k) != 0 ? 1u : 0u);
          }
        }
        tc_commit(empty_bar(s));     // the stage may be refilled once these MMAs have read it
        tc_commit(tfull_bar(acc));   // the accumulator is complete
        ++it;
      }
    }
  } else if (warp >= 4) {
    // ---------------- epilogue: TMEM -> registers -> global ----------------
    const int quad = warp & 3;          // TMEM lanes 32*quad .. 32*quad+31 (a warp may only touch its own quadrant)
    const int part = (warp - 4) >> 2;   // which kColsPerWarp of the tile's 256 columns
    // MODE 1: a lane appends its row's candidates straight to the row's list in global memory, into runs of kRun slots
    // that it reserves with one atomic add each. A warp's scoreboard tracks a register for all lanes at once, so an
    // atomic whose result any lane still waits for would stall every lane that touches the same register: the runs
    // are therefore requested only at tile starts, by one convergent instruction into `f_pending`, which nothing reads
    // before the next tile start (a whole tile later: the result has long arrived); there it becomes the lane's spare
    // run, and a lane that fills its current run in the middle of a tile switches to the spare without touching an
    // outstanding request. Only a lane that uses up both inside one tile reserves on the spot. When the block moves on
    // to other queries, what is left of the runs is filled with holes (position = kHole), which the select skips.
    // Entries past the list's capacity are dropped; the count keeps growing, which is how the select learns that the
    // row overflowed.
    constexpr uint32_t kRun = kFilterRun, kHole = 0xffffffffu;
    int64_t f_row = -1;
    float f_pivot = 0.f;
    uint32_t f_base = 0, f_used = kRun, f_spare = 0, f_pending = 0;
    bool f_has_spare = false, f_has_pending = false;
    uint2* f_list = nullptr;
    auto reserve_run = [&]() -> uint32_t { return atomicAdd(a.cand_count + f_row, kRun); };
    auto put = [&](uint32_t slot, uint2 e) {
      if (slot < (uint32_t)a.cand_cap) f_list[slot] = e;
    };
    auto close_runs = [&]() {  // the row is done for this lane: the unused slots become holes
      if (MODE != 1 || f_list == nullptr) return;
      for (uint32_t e = f_used; e < kRun; ++e) put(f_base + e, make_uint2(0u, kHole));
      if (f_has_spare)
        for (uint32_t e = 0; e < kRun; ++e) put(f_spare + e, make_uint2(0u, kHole));
      if (f_has_pending)
        for (uint32_t e = 0; e < kRun; ++e) put(f_pending + e, make_uint2(0u, kHole));
      f_list = nullptr;
      f_used = kRun;
      f_has_spare = f_has_pending = false;
    };
    uint32_t it = 0;
    for (int64_t id = tile_first; id < tile_last; id += tile_step) {
      const TileCoord c = tile_coord<MODE>(a, id);
      if (!c.valid) continue;
      const int acc = it % kAccBufs;
      const uint32_t aph = (it / kAccBufs) & 1u;
      if (!mbar_wait(tfull_bar(acc), aph, abort_flag)) break;
      tc_fence_after();
      const int t = c.mb * kBM + quad * 32 + lane;       // query of this thread's row
      const bool row_ok = t < a.q_per_seq;
      const int v = row_ok ? (causal ? c.n - a.q_per_seq + t + 1 : c.n) : 0;  // visible keys of this query
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * kBN);
      // columns this warp has to drain: up to the last one any of its 32 queries can see (a multiple of 32)
      const int v_warp = __reduce_max_sync(0xffffffffu, v) - c.nt * kBN;
      const int c_begin = part * kColsPerWarp;
      const int c_end = min(c_begin + kColsPerWarp, (max(v_warp, 0) + 31) & ~31);
      if (MODE == 1) {
        // ---- filter: compare with the row's pivot in registers; only candidates leave the SM ----
        const int64_t row = (int64_t)c.b * a.q_per_seq + t;
        if (row != f_row) {           // the block moved on to other queries
          close_runs();
          f_row = row;
          f_pivot = __int_as_float(0x7f800000);
          if (row_ok) {
            f_pivot = a.pivot[row];
            // a row with +inf needs no candidates at all
            if (f_pivot < __int_as_float(0x7f800000)) f_list = a.cand + row * a.cand_cap;
          }
        }
        if (f_list != nullptr) {      // tile start: last tile's request becomes the spare run, and a new one goes out
          if (f_has_pending && !f_has_spare) { f_spare = f_pending; f_has_spare = true; f_has_pending = false; }
          // ... unless this is the block's last tile on these queries: a run requested now would only become holes
          bool more = false;
          if (id + tile_step < tile_last) {
            const TileCoord nx = tile_coord<MODE>(a, id + tile_step);
            more = nx.valid && nx.b == c.b && nx.mb == c.mb;
          }
          // ... nor while the current run is less than half used and a spare is at hand
          const bool soon = f_used * 2 >= kRun || !f_has_spare;
          if (!f_has_pending && more && soon) { f_pending = reserve_run(); f_has_pending = true; }
        }
        uint32_t ra[16], rb[16];
        // The warp's staging tile (32 rows x 64 bytes, 16-byte chunk c of row r at r * 64 + ((c ^ ((r >> 1) & 3)) << 4),
        // free of bank conflicts for a row per lane) holds the chunk so that a lane can fetch the few columns that pass
        // by index: a lane's pass mask costs one compare per column, and only its own set bits cost anything more.
        unsigned char* tile = base_ptr + kStages * kStageBytes + (warp - 4) * 2048;
        const int swz = (lane >> 1) & 3;
        auto filter16 = [&](const uint32_t (&r)[16], int s0) {
          // Two instructions per column: the sign of (score - pivot) is shifted into a mask by a funnel shift. Four
          // chains of 4 columns, highest column first, so that column i ends up at bit i. The difference of a NaN is the
          // canonical (positive) NaN: it passes, like everything that is not below the pivot.
          uint32_t sg[4] = {0u, 0u, 0u, 0u};
#pragma unroll
          for (int j = 3; j >= 0; --j) {
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4)
              sg[q4] = __funnelshift_l(__float_as_uint(__uint_as_float(r[q4 * 4 + j]) - f_pivot), sg[q4], 1);
          }
          uint32_t mask = ~((sg[0] & 0xfu) | ((sg[1] & 0xfu) << 4) | ((sg[2] & 0xfu) << 8) | ((sg[3] & 0xfu) << 12)) & 0xffffu;
          if (s0 + 16 > v) mask &= s0 >= v ? 0u : (0xffffu >> (16 - (v - s0)));
          if (f_list == nullptr) mask = 0u;
          if (__any_sync(0xffffffffu, mask != 0u) == 0) return;
          __syncwarp();  // the previous chunk's reads of the tile are done
#pragma unroll
          for (int ch = 0; ch < 4; ++ch)
            *reinterpret_cast<uint4*>(tile + lane * 64 + ((ch ^ swz) << 4)) =
                make_uint4(r[4 * ch], r[4 * ch + 1], r[4 * ch + 2], r[4 * ch + 3]);
          // a lane reads back only what it wrote: no barrier needed in between
          while (mask != 0u) {
            const int i = __ffs(mask) - 1;
            mask &= mask - 1u;
            const uint32_t bits = *reinterpret_cast<const uint32_t*>(tile + lane * 64 + (((i >> 2) ^ swz) << 4) + (i & 3) * 4);
            if (f_used == kRun) {  // the current run is full: take the spare, or (rarely) reserve on the spot
              if (f_has_spare) { f_base = f_spare; f_has_spare = false; }
              else f_base = reserve_run();
              f_used = 0;
            }
            put(f_base + f_used, make_uint2(bits, (uint32_t)(s0 + i)));
            ++f_used;
          }
        };
        if (c_end > c_begin) tc_ld16(taddr + (uint32_t)c_begin, ra);
#pragma unroll 1
        for (int c0 = c_begin; c0 < c_end; c0 += 32) {
          tc_ld_wait();
          tc_ld16(taddr + (uint32_t)(c0 + 16), rb);   // c_end - c_begin is a multiple of 32
          filter16(ra, c.nt * kBN + c0);
          tc_ld_wait();
          if (c0 + 32 < c_end) tc_ld16(taddr + (uint32_t)(c0 + 32), ra);
          filter16(rb, c.nt * kBN + c0 + 16);
        }
      } else if (MODE == 2) {
        // ---- rows handed back: a lane stores its own row (if it has a slot) as it comes from TMEM ----
        const int64_t row = (int64_t)c.b * a.q_per_seq + t;
        const int slot = row_ok ? a.slot_of_row[row] : -1;
        float* dst_row = a.scores + (int64_t)max(slot, 0) * a.score_stride;
        uint32_t ra[32];
#pragma unroll 1
        for (int c0 = c_begin; c0 < c_end; c0 += 32) {
          tc_ld32(taddr + (uint32_t)c0, ra);
          tc_ld_wait();
          const int s0 = c.nt * kBN + c0;
          if (slot >= 0) {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (s0 + i < v) dst_row[s0 + i] = __uint_as_float(ra[i]);
          }
        }
      } else {
      // 32 columns at a time through two register buffers (the TMEM load of the next 32 columns is in flight
      // while the current 32 are stored). A TMEM load leaves a lane with 32 columns of ONE row; stored as they
      // come, a warp instruction would scatter 32-byte pieces over 32 rows. They go through a padded
      // shared-memory tile instead and come back with four lanes per row, so that every store instruction writes
      // eight complete 128-byte lines.
      // The staging tile holds 32 rows x 128 bytes in the 128-byte-swizzle layout of the tensor maps: the 16-byte
      // chunk c of row r sits at r * 128 + ((c ^ (r & 7)) << 4). Written a row per lane and read back four lanes per
      // row, both without bank conflicts; a chunk that is visible to all 32 queries leaves as ONE tiled bulk store
      // (the copy engine writes whole lines and the warp does not wait for them), the others -- on the causal
      // diagonal, at the end of a sequence -- as masked 32-byte stores.
      unsigned char* tile = base_ptr + kStages * kStageBytes + (warp - 4) * 4096;
      const uint32_t tile_u32 = smem_u32(tile);
      const int t0 = c.mb * kBM + quad * 32;  // first query row of this warp
      // every key below v_all is visible to all 32 rows (under the causal rule the first row sees the fewest)
      const int v_all = (t0 + 31 < a.q_per_seq) ? (causal ? c.n - a.q_per_seq + t0 + 1 : c.n) : 0;
      auto store32 = [&](const uint32_t (&r)[32], int s0) {
        // the copy engine must have finished reading the tile's previous contents; so must the other lanes
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncwarp();
#pragma unroll
        for (int ch = 0; ch < 8; ++ch)
          *reinterpret_cast<uint4*>(tile + lane * 128 + ((ch ^ (lane & 7)) << 4)) =
              make_uint4(r[4 * ch], r[4 * ch + 1], r[4 * ch + 2], r[4 * ch + 3]);
        if (a.vec_ok && s0 + 32 <= v_all) {
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the copy engine
          __syncwarp();
          if (lane == 0) {
            asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                         ::"l"(&map_s), "r"(s0), "r"(c.b * a.q_per_seq + t0), "r"(tile_u32) : "memory");
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          }
          return;
        }
        __syncwarp();
        const int s = s0 + (lane & 3) * 8;  // this lane's 8 columns
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int row = k * 8 + (lane >> 2);
          const int tq = t0 + row;
          const int vr = tq < a.q_per_seq ? (causal ? c.n - a.q_per_seq + tq + 1 : c.n) : 0;
          if (s >= vr) continue;
          const int ch = (lane & 3) * 2;
          const float4 w0 = *reinterpret_cast<const float4*>(tile + row * 128 + ((ch ^ (row & 7)) << 4));
          const float4 w1 = *reinterpret_cast<const float4*>(tile + row * 128 + (((ch + 1) ^ (row & 7)) << 4));
          const float w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
          float* dst = a.scores + ((int64_t)c.b * a.q_per_seq + tq) * a.score_stride + s;
          if (a.vec_ok && s + 8 <= vr) {
            asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(dst), "f"(w[0]), "f"(w[1]), "f"(w[2]),
                         "f"(w[3]), "f"(w[4]), "f"(w[5]), "f"(w[6]), "f"(w[7])
                         : "memory");
          } else {
#pragma unroll
            for (int e = 0; e < 8; ++e)
              if (s + e < vr) dst[e] = w[e];
          }
        }
      };
      uint32_t ra[32], rb[32];
      if (c_end > c_begin) tc_ld32(taddr + (uint32_t)c_begin, ra);
#pragma unroll 1
      for (int c0 = c_begin; c0 < c_end; c0 += 64) {
        tc_ld_wait();
        if (c0 + 32 < c_end) tc_ld32(taddr + (uint32_t)(c0 + 32), rb);
        store32(ra, c.nt * kBN + c0);
        if (c0 + 32 < c_end) {
          tc_ld_wait();
          if (c0 + 64 < c_end) tc_ld32(taddr + (uint32_t)(c0 + 64), ra);
          store32(rb, c.nt * kBN + c0 + 32);
        }
      }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));        // one arrival per epilogue warp frees the accumulator
      ++it;
    }
    close_runs();
    if (MODE == 0 && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // this warp's bulk stores have landed
  }

  tc_fence_before();
  __syncthreads();
  if (*abort_flag != 0u) {
    // A wait ran out: report it, and give copies that may still be in flight time to land before
    // the block (and its shared memory) goes away.
    if (threadIdx.x == 0) flag_status(a.status, CLSA_DEV_TIMEOUT);
    const long long t0 = clock64();
    while (clock64() - t0 < 4000000LL) {}
    __syncthreads();
  }
  if (warp == 2) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
      return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 [rows][cols] with `row_stride` elements between rows; box = 64 columns x box_rows rows.
bool make_map(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint64_t row_stride, uint32_t box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {row_stride * 2};
  const cuuint32_t box[2] = {(cuuint32_t)kBK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// fp32 [rows][row_stride] (all row_stride columns addressable), box = 32 columns x 32 rows, 128-byte swizzle.
bool make_map_f32(CUtensorMap* map, void* ptr, uint64_t rows, uint64_t row_stride) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (fn == nullptr) return false;
  const cuuint64_t dims[2] = {row_stride, rows};
  const cuuint64_t strides[1] = {row_stride * 4};
  const cuuint32_t box[2] = {32, 32};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, ptr, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

namespace {

// One launch of the chunk GEMM. mode 0: scores are stored into `scores` (sample_gs > 0: the sampled columns only);
// mode 1: filtered against fx.pivot into fx.cand; mode 2: rows with a slot are stored into row `slot` of `scores`.
cudaError_t launch_gemm(int mode, const clsa_params& p, const void* q_idx, float* scores, int64_t score_stride,
                        int sample_gs, const GemmFused* fx, uint32_t* status, const DeviceInfo& dev, cudaStream_t stream) {
  CUtensorMap map_q, map_k;
  const uint64_t q_rows = (uint64_t)p.num_seqs * p.q_per_seq;
  if (!make_map(&map_q, q_idx, q_rows, (uint64_t)p.idx_dim, (uint64_t)p.idx_dim, kBM)) return cudaErrorInvalidValue;
  const bool paged = p.block_table != nullptr;
  const int box_rows = sample_gs > 0 ? 16 : (paged && p.block_size < kBN ? p.block_size : kBN);
  if (!make_map(&map_k, p.idx_k_cache, (uint64_t)p.num_cache_rows, (uint64_t)p.idx_dim, (uint64_t)p.idx_token_stride,
                (uint32_t)box_rows))
    return cudaErrorInvalidValue;
  // fp32 scores [rows][score_stride], box = 32 columns x 32 rows, for the storing epilogue's tiled bulk stores (only
  // when the rows are 32-byte aligned; otherwise the map is a valid dummy over the key cache and is never used)
  const bool vec_ok = mode == 0 && score_stride % 8 == 0 && reinterpret_cast<uintptr_t>(scores) % 32 == 0;
  CUtensorMap map_s = map_k;
  if (vec_ok && !make_map_f32(&map_s, scores, q_rows, (uint64_t)score_stride)) return cudaErrorInvalidValue;
  GemmArgs a = {};
  a.block_table = p.block_table;
  a.block_size = paged ? p.block_size : 0;
  a.max_blocks_per_seq = p.max_blocks_per_seq;
  a.box_rows = box_rows;
  a.key_boxes = kBN / box_rows;
  a.seq_start = p.seq_start;
  a.seq_len = p.seq_len;
  a.scores = scores;
  a.score_stride = score_stride;
  a.status = status;
  a.num_seqs = p.num_seqs;
  a.q_per_seq = p.q_per_seq;
  a.causal = p.causal;
  a.max_seq_len = p.max_seq_len;
  a.idx_dim = p.idx_dim;
  a.m_blocks = (p.q_per_seq + kBM - 1) / kBM;
  const int columns = sample_gs > 0 ? (p.max_seq_len / sample_gs) * 16 : p.max_seq_len;
  a.n_tiles = (columns + kBN - 1) / kBN;
  a.vec_ok = vec_ok ? 1 : 0;
  a.sample_gs = sample_gs;
  a.row_major = mode == 0 ? 0 : 1;
  if (fx != nullptr) {
    a.pivot = fx->pivot;
    a.cand = fx->cand;
    a.cand_count = fx->cand_count;
    a.cand_cap = fx->cand_cap;
    a.slot_of_row = fx->slot_of_row;
    a.qblock_flag = fx->qblock_flag;
    a.nslots = fx->nslots;
  }
  const int64_t tiles = (int64_t)p.num_seqs * a.m_blocks * a.n_tiles;
  if (tiles < 1) return cudaSuccess;
  const int grid = (int)(tiles < dev.sm_count ? tiles : dev.sm_count);
  auto kernel = mode == 0 ? index_scores_gemm_kernel<0> : mode == 1 ? index_scores_gemm_kernel<1> : index_scores_gemm_kernel<2>;
  cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  if (err != cudaSuccess) return err;
  kernel<<<grid, gemm_threads(mode), kSmemBytes, stream>>>(map_q, map_k, map_s, a);
  return cudaGetLastError();
}

}  // namespace

// Slots of a row's candidate list that the filtering launch may leave as holes, at most: every lane that appends to
// the row (four per block: one per 64-column part of a tile) can end its stay on the row with a part-filled run and an
// unused spare, and the row's key tiles are spread over the blocks that the tile order gives it.
int index_gemm_filter_hole_slack(const clsa_params& p, const DeviceInfo& dev) {
  const int64_t m_blocks = (p.q_per_seq + kBM - 1) / kBM, n_tiles = (p.max_seq_len + kBN - 1) / kBN;
  const int64_t tiles = (int64_t)p.num_seqs * m_blocks * n_tiles;
  const int64_t grid = tiles < dev.sm_count ? tiles : dev.sm_count;
  const int64_t per_block = grid > 0 ? (tiles + grid - 1) / grid : 1;
  int64_t blocks_per_row = n_tiles / per_block + 2;
  if (blocks_per_row > n_tiles) blocks_per_row = n_tiles;
  return (int)((epi_warps(1) / 4) * blocks_per_row * 2 * kFilterRun);
}

cudaError_t launch_index_scores_gemm(const clsa_params& p, const void* q_idx, float* scores, int64_t score_stride,
                                     uint32_t* status, const DeviceInfo& dev, cudaStream_t stream) {
  return launch_gemm(0, p, q_idx, scores, score_stride, 0, nullptr, status, dev, stream);
}

cudaError_t launch_index_gemm_sample(const clsa_params& p, const void* q_idx, float* sample, int64_t sample_stride,
                                     int sample_gs, uint32_t* status, const DeviceInfo& dev, cudaStream_t stream) {
  return launch_gemm(0, p, q_idx, sample, sample_stride, sample_gs, nullptr, status, dev, stream);
}

cudaError_t launch_index_gemm_filter(const clsa_params& p, const void* q_idx, const GemmFused& fx, uint32_t* status,
                                     const DeviceInfo& dev, cudaStream_t stream) {
  return launch_gemm(1, p, q_idx, nullptr, 0, 0, &fx, status, dev, stream);
}

cudaError_t launch_index_gemm_handed_back(const clsa_params& p, const void* q_idx, float* scratch, int64_t score_stride,
                                          const GemmFused& fx, uint32_t* status, const DeviceInfo& dev, cudaStream_t stream) {
  return launch_gemm(2, p, q_idx, scratch, score_stride, 0, &fx, status, dev, stream);
}

}  // namespace clsa
