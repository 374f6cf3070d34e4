// GQA sparse attention over the selected rows only (Eq. 4), one launch per cross-decoder layer: the kernel for
// launches that share the GPU with their neighbours on the stream (the chained layers of a decode step) and for
// launches with many query rows (prefill chunks). A decode launch that has the GPU to itself uses the token-granular
// kernel in sparse_attn_sk.cu, which shares this file's staging ring and arithmetic.
//
// The kernel is bound by the gather of K/V rows from HBM (4 flops per byte per KV head), so its
// shape is chosen for memory behaviour; the small matrix products ride on warp-level bf16 MMAs
// (m16n8k16, fp32 accumulate) formed transposed -- tokens along M, the query heads of one KV head
// packed into the 8 columns of one tile -- far below tensor-pipe capacity.
//
// Decomposition. One thread-block cluster of C blocks serves one query row (sequence, query
// token); its selected tokens are cut into C * S contiguous ranges. A block has 12 autonomous
// warps (8 for query-head groups above 8): warp w serves KV head w % HC of token range w / HC (HC
// heads per block, S = warps / HC ranges per block). A warp streams
// its range in 16-token stages through a private 2-deep cp.async ring (16-byte chunks,
// XOR-swizzled for conflict-free ldmatrix), runs S = Q K^T, an online softmax in the exp2 domain
// and O += P V per stage; there is no block-level barrier in the main loop. Split-K merge: every
// warp leaves its unnormalised partial (O, running max, running sum) in its own shared memory,
// the cluster synchronises once, and the (KV head, query head) outputs are dealt round-robin to
// the warps of the cluster, each reading the C * S partials it needs through distributed shared
// memory and combining them by log-sum-exp. Nothing goes through global memory, nothing spins.
// Two launch shapes. A launch on its own (its output feeds the next kernel) gets the whole GPU: HC shrinks
// (down to one KV head per block, its warps splitting the tokens) until rows * Hkv / HC fits the SM
// count, then C grows while all clusters stay resident at once. Decoding a batch of 16 with 8 KV heads
// runs 128 single-block clusters whose merge never leaves the block; a launch with far more rows than SMs
// (a prefill chunk) puts several rows in a block, up to one warp per (row, KV head) with nothing to merge. The layers of one decode step, which do not wait for one another,
// are launched side by side instead: about 32 large blocks per layer (as many KV heads per block as that
// allows), so that four or five layers are in flight at once: every SM stays busy and the per-block
// fixed costs are paid 32 instead of 128 times per layer. And where a warp has a head tile to spare (groups of up to
// 8 query heads), such layers go two per launch: every layer of a step gathers the same rows, so the second tile
// takes the next layer's query heads over the same staged rows (about 16 blocks per launch of two layers).
// `reverse` flips the order in which a warp walks its range (a locality hint for callers that issue
// dependent layers one by one; the chained layers of a step all walk the same way).
#include <cooperative_groups.h>
#include <mutex>

#include "attn_common.cuh"

namespace cg = cooperative_groups;

namespace clsa {
namespace {

constexpr int kMergeBatch = 8;

struct AttnArgs {
  const uint16_t* q;
  const uint16_t* q2;   // PAIR: the second layer's queries
  const uint16_t* kc;
  const uint16_t* vc;
  int64_t tok_stride, head_stride;
  const int64_t* seq_start;
  const int32_t* seq_len;
  const int32_t* idx;
  const int32_t* count;
  const int32_t* block_table;  // paged caches: [B][max_blocks] physical block numbers, or nullptr
  int block_shift, max_blocks;
  uint16_t* out;
  uint16_t* out2;       // PAIR: the second layer's outputs
  float* lse;
  uint32_t* status;
  int q_per_seq, num_q_heads, num_kv_heads, group, top_k;
  int heads_per_block, subs, rows_per_block, reverse;
  int64_t num_rows;
  int wait_prior;  // 1: inputs may come from the kernel launched just before this one (wait for it first)
  int early;       // 1 (with wait_prior): only q is pending; index, counts and caches may be read before the wait
  int off32;          // every row offset of the caches fits 32 bits when counted in 16-byte units
  int64_t rows_max;   // extent of the cache row space (off32 only): rows at or beyond it are refused like bad indices
  int keep;           // 1: the rows are fetched with the L2 evict_last priority (launches behind this one read them again)
  int pin;            // -1: one L2 priority for every row (evict_last if keep). 0..8: of every 8 consecutive stages of a row's
                      // selected set the first `pin` are fetched evict_last and the others evict_first
  int max_seq_len;    // sequences longer than this (or shorter than q_per_seq) are skipped and flagged
  float scale_log2;
};

// NT = number of 8-head tiles that hold the query heads of one KV head (1 for groups up to 8, 2 up to 16).
// WARPS = warps per block: 12 for NT = 1 (about 165 registers per thread), 8 for NT = 2.
// MULTI: a block serves several query rows (rows_per_block > 1); the single-row instances keep the row uniform
// over the block.
// PAIR = two layers in one launch (NT == 2, groups of up to 8 query heads): head tile 0 holds the first layer's query
// heads, tile 1 the second layer's, both over the same staged K/V rows -- the rows of a step are the same for every
// layer, so a pair of layers whose queries are both at hand copies them from L2 once instead of twice. Per layer the
// arithmetic is that of a single-layer launch of the same block shape, bit for bit.
template <int NT, bool PAGED, int WARPS, bool MULTI, bool PAIR = false>
__global__ void __launch_bounds__(WARPS * 32, 1) sparse_attn_kernel(const AttnArgs a) {
  static_assert(!PAIR || NT == 2, "a pair of layers takes the two head tiles");
  extern __shared__ __align__(128) unsigned char smem[];
  cg::cluster_group cluster = cg::this_cluster();
  const int C = (int)cluster.num_blocks();
  const int crank = (int)cluster.block_rank();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned bx = blockIdx.x, by = blockIdx.y;
  const int HC = a.heads_per_block, S = a.subs, G = a.group;
  const int g_local = warp % HC;
  const int RB = MULTI ? a.rows_per_block : 1;
  const int row_local = MULTI ? (warp / HC) / S : 0;  // which of the block's rows
  const int sub = (warp / HC) - row_local * S;       // which of that row's token ranges
  const int64_t r_true = (int64_t)(bx / C) * RB + row_local;
  const int g = by * HC + g_local;                  // KV head of this warp
  const bool active = sub < S && row_local < RB && r_true < a.num_rows && g < a.num_kv_heads;
  const int64_t r = (!MULTI || r_true < a.num_rows) ? r_true : a.num_rows - 1;  // query row (clamped past the last row)
  const int nsplit = C * S;                         // token ranges of the row

  unsigned char* ring = smem + warp * kWarpRingBytes;
  const uint32_t ring_u32 = smem_u32(ring);
  uint32_t* stage_mask = reinterpret_cast<uint32_t*>(smem + WARPS * kWarpRingBytes) + warp * kAttnStages;

  // Fragment coordinates. The products are formed transposed, tokens along M:
  //   S^T[16 tokens x 8 heads] = K[16 x 128] Q^T,   O^T[128 x 8 heads] += V^T[128 x 16 tokens] P^T
  // so a lane's accumulator columns are always the same two query heads (hcol, hcol+1 of each 8-head
  // tile), and its rows are tokens (for S^T: rowq and rowq+8) or output dimensions (for O^T).
  const int rowq = lane >> 2;
  const int hcol = (lane & 3) * 2;
  const int h0 = g * G;                // first query head of this KV head

  // Programmatic dependent launch. Unless the caller vouches that every input predates the previous
  // kernel, wait for that kernel's results before the first global read; only then let the next
  // kernel of the stream be scheduled (as SMs free up). The order matters: a kernel launched behind
  // this one may skip its own wait on the grounds that everything it reads was complete before this
  // grid started reading -- which holds only if this grid has waited before it releases anybody.
  // A launch whose only pending input is q (a.early) waits later: behind the first stage of row copies, in front of
  // the first read of q and of every global write.
  bool waited = !(a.wait_prior && a.early);
  if (a.wait_prior && !a.early) asm volatile("griddepcontrol.wait;" ::: "memory");
  if (waited) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  auto wait_now = [&]() {
    if (!waited) {
      asm volatile("griddepcontrol.wait;" ::: "memory");
      asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
      waited = true;
    }
  };

  // The row's k slots are cut into nsplit ranges of `per` slots (a multiple of the stage size); the
  // split does not depend on the row's count, so the first positions can be fetched together with it.
  const int per = (((a.top_k + nsplit - 1) / nsplit) + kAttnStageTokens - 1) / kAttnStageTokens * kAttnStageTokens;
  const int range = crank * S + sub;
  const int slot_lo = min(a.top_k, range * per), slot_hi = min(a.top_k, slot_lo + per);
  const int32_t* row_idx = a.idx + r * a.top_k;
  int cnt = a.count[r];
  const int b = (int)(r / a.q_per_seq);
  constexpr bool paged = PAGED;
  const int64_t s0 = paged ? 0 : a.seq_start[b];  // paged: positions are translated to cache rows when they are fetched
  const int32_t* table = paged ? a.block_table + (int64_t)b * a.max_blocks : nullptr;
  // A sequence whose length lies outside its declared bounds is never read: with n = 0 no position passes the range
  // check, every stage is masked, and the row comes out as zeros with lse = -inf. (A select, not a branch: the length
  // is first needed when the first copies are issued, and the flag is raised behind the main loop.)
  const int n_raw = a.seq_len[b];
  const bool n_ok = n_raw >= a.q_per_seq && n_raw <= a.max_seq_len;
  const int n = n_ok ? n_raw : 0;
  // Positions are fetched two pipeline steps before they are used and (paged caches) their block numbers one
  // step before, so that no load is consumed in the step that issued it. The first three steps' positions are
  // fetched here, speculatively for a range that lies entirely below the row's count (entries past the count
  // are never used).
  const int nst_full = (slot_hi - slot_lo + kAttnStageTokens - 1) / kAttnStageTokens;
  int spec_raw[3] = {-1, -1, -1};
  if (active && lane < kAttnStageTokens) {
#pragma unroll
    for (int i = 0; i < 3; ++i) {
      const int tt = slot_lo + (a.reverse ? nst_full - 1 - i : i) * kAttnStageTokens + lane;
      if (i < nst_full && tt < slot_hi) spec_raw[i] = row_idx[tt];
    }
  }
  if (cnt < 0 || cnt > a.top_k) {
    if (lane == 0 && sub == 0 && g_local == 0 && crank == 0 && by == 0 && active) flag_status(a.status, CLSA_DEV_BAD_COUNT);
    cnt = cnt < 0 ? 0 : a.top_k;
  }
  const int t_lo = min(cnt, slot_lo), t_hi = active ? min(cnt, slot_hi) : t_lo;

  float o[NT][8][4];                   // O^T: [head tile][16-wide slice of D][c0..c3]
  float mA[NT], mB[NT], lA[NT], lB[NT];  // running max / sum of heads hcol and hcol+1 (log2 domain)
  float lacc[NT][4];                   // the sums as an MMA accumulator: ones[16 x 16] . P^T puts a head's sum over the stage's
                                       // 16 tokens in every row of its column (c0: head hcol, c1: head hcol + 1)
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    mA[nt] = -INFINITY; mB[nt] = -INFINITY; lA[nt] = 0.f; lB[nt] = 0.f;
    lacc[nt][0] = 0.f; lacc[nt][1] = 0.f; lacc[nt][2] = 0.f; lacc[nt][3] = 0.f;
#pragma unroll
    for (int j = 0; j < 8; ++j) { o[nt][j][0] = 0.f; o[nt][j][1] = 0.f; o[nt][j][2] = 0.f; o[nt][j][3] = 0.f; }
  }

  if (t_lo < t_hi) {
    // Q^T fragments (B operand, 128 x 8 per head tile): head = rowq, two consecutive d per register.
    uint32_t qb[NT][8][2];
    auto load_q = [&]() {
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const uint16_t* qbase = ((PAIR && nt == 1) ? a.q2 : a.q) + (r * a.num_q_heads + h0) * 128;
        const int head = PAIR ? rowq : nt * 8 + rowq;
        const bool hv = head < G;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const int d = ks * 16 + hcol;
          qb[nt][ks][0] = hv ? *reinterpret_cast<const uint32_t*>(qbase + head * 128 + d) : 0u;
          qb[nt][ks][1] = hv ? *reinterpret_cast<const uint32_t*>(qbase + head * 128 + d + 8) : 0u;
        }
      }
    };
    if (waited) load_q();

    const int nstages = (t_hi - t_lo + kAttnStageTokens - 1) / kAttnStageTokens;
    const uint16_t* kbase = a.kc + g * a.head_stride + (lane & 15) * 8;
    const uint16_t* vbase = a.vc + g * a.head_stride + (lane & 15) * 8;

    // token offset of pipeline step i
    auto stage_t0 = [&](int i) { return t_lo + (a.reverse ? nstages - 1 - i : i) * kAttnStageTokens; };
    // lanes 0..15 fetch the 16 positions of step i (-1 past the end); the value is not touched here
    auto load_raw = [&](int i) -> int {
      if (i >= nstages || lane >= kAttnStageTokens) return -1;
      const int tt = stage_t0(i) + lane;
      return tt < t_hi ? row_idx[tt] : -1;
    };
    // paged caches: block number of a position fetched at least one step ago (not touched here either)
    auto load_blk = [&](int raw) -> int {
      if (!paged || raw < 0 || raw >= n) return 0;
      return __ldg(table + (raw >> a.block_shift));
    };
    // L2 residency across layers: the layers of a step walk the same rows in the same direction a few microseconds
    // apart, so what one layer fetches the next ones find in L2. Such launches fetch with the evict_last priority
    // (other traffic through L2 does not push the rows out in between); a launch on its own leaves the replacement
    // policy alone.
    const uint64_t pol_keep = a.keep ? l2_policy_evict_last() : l2_policy_evict_normal();
    const uint64_t pol_last = l2_policy_evict_last(), pol_first = l2_policy_evict_first();
    // Per-lane constants of the copies: where in a stage buffer this lane's 16-byte chunk of token j = 2*it + lane/16
    // goes (XOR swizzle), and the lane's byte offset inside a row.
    uint32_t sw[8];
#pragma unroll
    for (int it = 0; it < 8; ++it) {
      const int j = it * 2 + (lane >> 4);
      sw[it] = (uint32_t)(j * 256 + (((lane & 15) ^ (j & 7)) << 4));
    }
    const char* kbytes = reinterpret_cast<const char*>(kbase);
    const char* vbytes = reinterpret_cast<const char*>(vbase);
    const uint32_t stride16 = (uint32_t)(a.tok_stride >> 3);  // row stride in 16-byte units (the stride is a multiple of 8)
    auto issue = [&](int i, int raw, int blk) {
      if (i < nstages) {
        const int buf = i % kAttnStages;
        const uint32_t kdst = ring_u32 + buf * kStageBytes, vdst = kdst + kStageBytes / 2;
        const uint64_t pol = a.pin < 0 ? pol_keep : (pin_rank((stage_t0(i) >> 4) & 7) < a.pin ? pol_last : pol_first);
        // cache row relative to s0: the position itself, or its place inside its block
        const int my_idx = paged ? (blk << a.block_shift) + (raw & ((1 << a.block_shift) - 1)) : raw;
        const bool in_range = raw >= 0 && raw < n && (!a.off32 || (uint64_t)(s0 + my_idx) < (uint64_t)a.rows_max);
        const uint32_t okmask = __ballot_sync(0xffffffffu, in_range) & 0xffffu;
        const bool bad = lane < kAttnStageTokens && !in_range && n_ok && (stage_t0(i) + lane) < t_hi;
        if (bad) flag_status(a.status, CLSA_DEV_BAD_INDEX);
        if (lane == 0) stage_mask[buf] = okmask;
        if (a.off32) {
          // the whole cache spans fewer than 2^32 16-byte units: a row's offset is one 32-bit number, computed once
          // by the lane that holds the position and widened with the base pointer in one multiply-add per copy
          const uint32_t my_off16 = in_range ? ((uint32_t)s0 + (uint32_t)my_idx) * stride16 : 0u;
          if (okmask == 0xffffu) {  // the usual stage: all 16 positions valid, plain copies
#pragma unroll
            for (int it = 0; it < 8; ++it) {
              const uint32_t off16 = __shfl_sync(0xffffffffu, my_off16, it * 2 + (lane >> 4));
              cp_async16_full(kdst + sw[it], kbytes + (uint64_t)off16 * 16u, pol);
              cp_async16_full(vdst + sw[it], vbytes + (uint64_t)off16 * 16u, pol);
            }
          } else {
#pragma unroll
            for (int it = 0; it < 8; ++it) {
              const int j = it * 2 + (lane >> 4);  // token of the stage this lane helps fetch
              const uint32_t off16 = __shfl_sync(0xffffffffu, my_off16, j);
              const bool ok = (okmask >> j) & 1u;
              cp_async16(kdst + sw[it], kbytes + (uint64_t)off16 * 16u, ok, pol);
              cp_async16(vdst + sw[it], vbytes + (uint64_t)off16 * 16u, ok, pol);
            }
          }
        } else {
#pragma unroll
          for (int it = 0; it < 8; ++it) {
            const int j = it * 2 + (lane >> 4);
            const int tok = __shfl_sync(0xffffffffu, my_idx, j);
            const bool ok = (okmask >> j) & 1u;
            const int64_t off = (s0 + (ok ? tok : 0)) * a.tok_stride;
            cp_async16(kdst + sw[it], kbase + off, ok, pol);
            cp_async16(vdst + sw[it], vbase + off, ok, pol);
          }
        }
      }
      cp_async_commit();
    };

    // prologue: stage 0 in flight; positions of steps 1 and 2 (and step 1's block numbers) in registers
    int r0 = spec_raw[0], rawA = spec_raw[1], rawB = spec_raw[2];
    if (t_hi != slot_hi) {  // the count cuts this range short: fetch the real first positions
      r0 = load_raw(0); rawA = load_raw(1); rawB = load_raw(2);
    }
    int blkA;
    {
      const int b0 = load_blk(r0);
      blkA = load_blk(rawA);
      issue(0, r0, b0);
    }
    if (!waited) {  // only q was pending: the first stage of copies is in flight, now wait for q's producer
      wait_now();
      load_q();
    }
#pragma unroll 1
    for (int i = 0; i < nstages; ++i) {
      {  // refill the buffer freed by step i-1, then advance the position pipeline
        const int raw_new = load_raw(i + kAttnStages + 1);
        const int blk_new = load_blk(rawB);
        issue(i + kAttnStages - 1, rawA, blkA);
        rawA = rawB;
        blkA = blk_new;
        rawB = raw_new;
      }
      cp_async_wait<kAttnStages - 1>();
      __syncwarp();
      const int buf = i % kAttnStages;
      const uint32_t kbuf = ring_u32 + buf * kStageBytes, vbuf = kbuf + kStageBytes / 2;
      const uint32_t okmask = stage_mask[buf];

      // S^T = K Q^T for 16 tokens: A = K rows (tokens) from shared memory, B = Q^T from registers. Two accumulators
      // (even and odd 16-wide slices of D) halve the chain of dependent MMAs.
      float s[NT][4], s_odd[NT][4];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        s[nt][0] = 0.f; s[nt][1] = 0.f; s[nt][2] = 0.f; s[nt][3] = 0.f;
        s_odd[nt][0] = 0.f; s_odd[nt][1] = 0.f; s_odd[nt][2] = 0.f; s_odd[nt][3] = 0.f;
      }
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const int tok = (lane & 7) + 8 * ((lane >> 3) & 1), chunk = 2 * ks + (lane >> 4);
        uint32_t kf[4];
        ldmatrix_x4(kf, kbuf + tok * 256 + ((chunk ^ (tok & 7)) << 4));
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) mma_bf16((ks & 1) ? s_odd[nt] : s[nt], kf, qb[nt][ks][0], qb[nt][ks][1]);
      }
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        s[nt][0] += s_odd[nt][0]; s[nt][1] += s_odd[nt][1]; s[nt][2] += s_odd[nt][2]; s[nt][3] += s_odd[nt][3];
      }
      // online softmax over tokens (rows), per head (columns), exp2 domain; masked tokens get -inf. The maxima are
      // taken over the raw dot products (the scale is positive) and the scale rides in the multiply-add of the exponent.
      const bool full = okmask == 0xffffu;  // the usual stage: nothing to mask
      const bool ok_lo = (okmask >> rowq) & 1u, ok_hi = (okmask >> (rowq + 8)) & 1u;
      uint32_t pb0[NT], pb1[NT];
      bool rescale = false;
      float alphaA[NT], alphaB[NT];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        float r0 = s[nt][0], r1 = s[nt][1], r2 = s[nt][2], r3 = s[nt][3];  // tokens rowq (r0, r1) and rowq + 8; heads hcol, hcol + 1
        if (!full) {
          r0 = ok_lo ? r0 : -INFINITY; r1 = ok_lo ? r1 : -INFINITY;
          r2 = ok_hi ? r2 : -INFINITY; r3 = ok_hi ? r3 : -INFINITY;
        }
        float mxA = fmaxf(r0, r2), mxB = fmaxf(r1, r3);
#pragma unroll
        for (int d = 4; d <= 16; d <<= 1) {
          mxA = fmaxf(mxA, __shfl_xor_sync(0xffffffffu, mxA, d));
          mxB = fmaxf(mxB, __shfl_xor_sync(0xffffffffu, mxB, d));
        }
        const float mnA = fmaxf(mA[nt], mxA * a.scale_log2), mnB = fmaxf(mB[nt], mxB * a.scale_log2);
        const float muA = mnA == -INFINITY ? 0.f : mnA, muB = mnB == -INFINITY ? 0.f : mnB;
        alphaA[nt] = fast_exp2(mA[nt] - muA);
        alphaB[nt] = fast_exp2(mB[nt] - muB);
        rescale = rescale || mnA != mA[nt] || mnB != mB[nt];
        mA[nt] = mnA;
        mB[nt] = mnB;
        const uint32_t p_lo = pack_bf16x2(fast_exp2(fmaf(r0, a.scale_log2, -muA)), fast_exp2(fmaf(r1, a.scale_log2, -muB)));
        const uint32_t p_hi = pack_bf16x2(fast_exp2(fmaf(r2, a.scale_log2, -muA)), fast_exp2(fmaf(r3, a.scale_log2, -muB)));
        // P is held [token][head]; the PV product wants P^T as its B operand: transpose the two 8x8 halves
        pb0[nt] = movmatrix_trans(p_lo);
        pb1[nt] = movmatrix_trans(p_hi);
      }
      if (__any_sync(0xffffffffu, rescale)) {  // the running max moved for some head: rescale the accumulators
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            o[nt][j][0] *= alphaA[nt]; o[nt][j][1] *= alphaB[nt]; o[nt][j][2] *= alphaA[nt]; o[nt][j][3] *= alphaB[nt];
          }
          lacc[nt][0] *= alphaA[nt]; lacc[nt][1] *= alphaB[nt]; lacc[nt][2] *= alphaA[nt]; lacc[nt][3] *= alphaB[nt];
        }
      }
      // the denominators: the same bf16-rounded weights as the numerators, summed over the stage's tokens by one MMA
      {
        const uint32_t ones[4] = {0x3f803f80u, 0x3f803f80u, 0x3f803f80u, 0x3f803f80u};
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) mma_bf16(lacc[nt], ones, pb0[nt], pb1[nt]);
      }
      // O^T += V^T P^T: A = V^T (transposing ldmatrix of the [token][d] tile), 8 slices of 16 output dimensions
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int tok = (lane & 7) + 8 * (lane >> 4), chunk = 2 * j + ((lane >> 3) & 1);
        uint32_t vf[4];
        ldmatrix_x4_trans(vf, vbuf + tok * 256 + ((chunk ^ (tok & 7)) << 4));
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) mma_bf16(o[nt][j], vf, pb0[nt], pb1[nt]);
      }
      __syncwarp();  // everyone is done with this buffer before the next step refills it
    }
    cp_async_wait<0>();

#pragma unroll
    for (int nt = 0; nt < NT; ++nt) { lA[nt] = lacc[nt][0]; lB[nt] = lacc[nt][1]; }
  }

  wait_now();  // a warp without tokens has not waited yet; what follows writes global memory
  if (!n_ok && lane == 0 && sub == 0 && g_local == 0 && crank == 0 && by == 0 && active) flag_status(a.status, CLSA_DEV_BAD_SEQLEN);

  // ---- split-K merge through (distributed) shared memory --------------------------------------------
  // Each warp parks its partial in its own (now idle) staging ring: [G][kPartialStride] floats, row = head.
  float* mypart = reinterpret_cast<float*>(ring);
  if (active) {
    __syncwarp();
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      // slot of a head in the warp's partial: the head itself, or (PAIR) layer * G + head of the layer
      const int headA = PAIR ? nt * G + hcol : nt * 8 + hcol, headB = headA + 1;
      const bool okA = PAIR ? hcol < G : headA < G, okB = PAIR ? hcol + 1 < G : headB < G;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int d = 16 * j + rowq;
        if (okA) { mypart[headA * kPartialStride + d] = o[nt][j][0]; mypart[headA * kPartialStride + d + 8] = o[nt][j][2]; }
        if (okB) { mypart[headB * kPartialStride + d] = o[nt][j][1]; mypart[headB * kPartialStride + d + 8] = o[nt][j][3]; }
      }
      if (rowq == 0) {
        if (okA) *reinterpret_cast<float2*>(mypart + headA * kPartialStride + 128) = make_float2(mA[nt], lA[nt]);
        if (okB) *reinterpret_cast<float2*>(mypart + headB * kPartialStride + 128) = make_float2(mB[nt], lB[nt]);
      }
    }
  }
  if (C == 1) __syncthreads(); else cluster.sync();

  // Output jobs (KV head of this block's group, query head of the group) dealt over the cluster's warps.
  const int heads_here = min(HC, a.num_kv_heads - (int)by * HC);
  const int jobs_per_layer = heads_here * G;
  const int jobs_per_row = jobs_per_layer * (PAIR ? 2 : 1);
  const int njobs = RB * jobs_per_row;
  const uint32_t smem_base = smem_u32(smem);
  for (int job = crank + C * warp; job < njobs; job += C * WARPS) {
    const int rl = MULTI ? job / jobs_per_row : 0;  // which of the block's rows
    const int64_t r_job = (int64_t)(bx / C) * RB + rl;
    if (MULTI && r_job >= a.num_rows) continue;
    const int jrow_all = job - rl * jobs_per_row;
    const int lyr = PAIR ? jrow_all / jobs_per_layer : 0;   // which layer of the pair
    const int jrow = jrow_all - lyr * jobs_per_layer;
    const int jg = jrow / G, hh = jrow - jg * G;   // local KV head, query head within the group
    const int hslot = PAIR ? lyr * G + hh : hh;    // the head's slot in a warp's partial
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float L = 0.f, M = -INFINITY;
    // Partial p = (block p / S, range p % S) of row rl was left by warp (rl * S + p % S) * HC + jg of block p / S. Lane p of each
    // 32-partial chunk resolves that partial's shared::cluster address once; everyone then reads through it.
    for (int p0 = 0; p0 < nsplit; p0 += 32) {
      const int p = p0 + lane;
      uint32_t src = 0;
      float2 ml = make_float2(-INFINITY, 0.f);
      if (p < nsplit) {
        const int c2 = p / S, sub2 = p - c2 * S;
        const uint32_t local = smem_base + (uint32_t)(((rl * S + sub2) * HC + jg) * kWarpRingBytes + hslot * kPartialStride * 4);
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(src) : "r"(local), "r"(c2));
        asm volatile("ld.shared::cluster.v2.f32 {%0, %1}, [%2];" : "=f"(ml.x), "=f"(ml.y) : "r"(src + 512u) : "memory");
      }
      // running max over this chunk and what came before; rescale what came before
      float mc = ml.x;
#pragma unroll
      for (int d = 16; d >= 1; d >>= 1) mc = fmaxf(mc, __shfl_xor_sync(0xffffffffu, mc, d));
      const float Mn = fmaxf(M, mc);
      const float mu = Mn == -INFINITY ? 0.f : Mn;
      const float rescale = fast_exp2(M - mu);
      acc.x *= rescale; acc.y *= rescale; acc.z *= rescale; acc.w *= rescale;
      L *= rescale;
      M = Mn;
      const float wl = fast_exp2(ml.x - mu);   // 0 for lanes past the end
      float lsum = wl * ml.y;
#pragma unroll
      for (int d = 16; d >= 1; d >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, d);
      L += lsum;
      const int chunk_n = min(32, nsplit - p0);
      for (int q0 = 0; q0 < chunk_n; q0 += kMergeBatch) {
        float4 v[kMergeBatch];
#pragma unroll
        for (int qq = 0; qq < kMergeBatch; ++qq) {
          const uint32_t sq = __shfl_sync(0xffffffffu, src, (q0 + qq) & 31);
          v[qq] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (q0 + qq < chunk_n)
            asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                         : "=f"(v[qq].x), "=f"(v[qq].y), "=f"(v[qq].z), "=f"(v[qq].w) : "r"(sq + (uint32_t)lane * 16u) : "memory");
        }
#pragma unroll
        for (int qq = 0; qq < kMergeBatch; ++qq) {
          const float w = __shfl_sync(0xffffffffu, wl, (q0 + qq) & 31);
          const float wq = q0 + qq < chunk_n ? w : 0.f;
          acc.x = fmaf(wq, v[qq].x, acc.x); acc.y = fmaf(wq, v[qq].y, acc.y);
          acc.z = fmaf(wq, v[qq].z, acc.z); acc.w = fmaf(wq, v[qq].w, acc.w);
        }
      }
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
    const int64_t item = r_job * a.num_q_heads + (int64_t)(by * HC + jg) * G + hh;
    uint2 packed;
    packed.x = pack_bf16x2(acc.x * inv, acc.y * inv);
    packed.y = pack_bf16x2(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2*>(((PAIR && lyr == 1) ? a.out2 : a.out) + item * 128 + lane * 4) = packed;
    if (a.lse != nullptr && lane == 0) a.lse[item] = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
  }
  if (C > 1) cluster.sync();  // no block may exit while a neighbour can still read its shared memory
}

// Blocks of `cluster` that can be resident at once on the current device (cached per device and cluster size;
// 0 if the query fails).
static int max_resident_blocks(int cluster, size_t smem_bytes, int warps) {
  static std::mutex mu;
  static int cache[64][9][2] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return 0; }
  const int which = warps == kAttnWarpsNarrow ? 0 : 1;
  std::lock_guard<std::mutex> lock(mu);
  if (cache[dev][cluster][which] != 0) return cache[dev][cluster][which];
  auto kernel = which == 0 ? sparse_attn_kernel<1, false, kAttnWarpsNarrow, false> : sparse_attn_kernel<2, false, kAttnWarpsWide, false>;
  cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)cluster * 64, 1, 1);
  cfg.blockDim = dim3((unsigned)warps * 32, 1, 1);
  cfg.dynamicSmemBytes = smem_bytes;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)cluster;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
  cache[dev][cluster][which] = n * cluster;
  return cache[dev][cluster][which];
}

}  // namespace

// Block model of the two-layer decode launches (measured on a B200 at the headline: a block of 8 KV heads x 2048 tokens
// x 2 layers takes about 125 us).
constexpr double kPairBytesPerUs = 64.0e3;   // bytes of K/V rows a block copies per microsecond
constexpr double kPairBlockFixedUs = 9.5;    // launch gap + pipeline ramp + merge of one block

AttnPlan make_attn_plan(const clsa_params& p, const DeviceInfo& dev, int throughput) {
  AttnPlan plan;
  // 12 warps per block where the registers allow it (query-head groups up to 8: one 8-column tile per warp); the
  // main loop is a dependent chain per warp, so warps per SM, not bytes in flight, set the pace once the rows come
  // from L2.
  plan.warps = p.num_q_heads / p.num_kv_heads <= 8 ? kAttnWarpsNarrow : kAttnWarpsWide;
  const bool pair_shape = throughput == 3 || throughput == 4;
  if (pair_shape) plan.warps = kAttnWarpsWide;  // two layers per launch: two head tiles per warp, as for wide groups
  const int64_t rows_ = (int64_t)p.num_seqs * p.q_per_seq;
  // Side by side, 32 to 63 rows of 8 or more KV heads: 8 warps can take all 8 heads of a row (32 to 63 blocks per
  // launch, the shape that works best), which 12 warps cannot (4 heads per block, twice the blocks).
  if (throughput && p.num_kv_heads >= 8 && rows_ * ((p.num_kv_heads + 7) / 8) >= 32 && rows_ * ((p.num_kv_heads + 7) / 8) < 64)
    plan.warps = kAttnWarpsWide;
  plan.smem_bytes = (size_t)plan.warps * kWarpRingBytes + plan.warps * kAttnStages * sizeof(uint32_t);
  const int hkv = p.num_kv_heads;
  const int64_t rows = (int64_t)p.num_seqs * p.q_per_seq;
  // heads per block: a power of two that divides the warps (1, 2, 4 of 12; 1, 2, 4, 8 of 8) and does not exceed Hkv
  int hc_max = 1;
  while (hc_max * 2 <= hkv && plan.warps % (hc_max * 2) == 0) hc_max *= 2;
  int hc, c = 1;
  bool pair_fine_grain = false;
  if (throughput) {
    // The launch shares the GPU with the launches next to it on the stream (the layers of one step: each reads
    // only the index, the caches and its own queries, so none waits for its predecessor). What counts then is the
    // work per block, not how many SMs one launch covers: as many KV heads per block as leave about 32 blocks
    // per launch, no clusters. Four or five layers are then in flight at once and keep every SM busy
    // (measured: 32 blocks per layer beat 16, 64 and 128 at every batch size tried).
    hc = hc_max;
    while (hc > 1 && rows * ((hkv + hc - 1) / hc) < (pair_shape ? 16 : 32)) hc /= 2;
    // ... as long as the step has at most about two and a half rounds of blocks; beyond that the finer blocks lose more
    // (split rows, rows of a step no longer walked together by its launches) than the fuller last round returns.
    pair_fine_grain = pair_shape && p.q_per_seq == 1 &&
                      (p.num_layers >= 2 ? p.num_layers / 2 : 1) * rows * ((hkv + hc - 1) / hc) * 2 <= 5 * (int64_t)dev.sm_count;
    if (pair_fine_grain) {
      // Two layers per launch, decoding: blocks run twice as long, and about 16 per launch do best while all launches
      // of the step are resident at once (16 rows of 8 KV heads: a block takes a whole row, one KV head per warp,
      // nothing split and nothing merged; 8 launches x 16 blocks on 148 SMs). One row more and the step's blocks no
      // longer fit one round: then fewer heads per block fill the last round at a finer grain. The same block model as
      // for the finer tail of one-layer chains: a fixed part plus the block's bytes at the rate a block of this kernel
      // copies them; the step's blocks are placed in rounds of one per SM.
      const double k_eff = (double)(p.top_k < p.max_seq_len ? p.top_k : p.max_seq_len);
      const double us_per_head = k_eff * 512.0 / kPairBytesPerUs;
      const int64_t launches = p.num_layers >= 2 ? p.num_layers / 2 : 1;
      double best = 0.0;
      int best_hc = hc;
      for (int cand = hc; cand >= 1; cand /= 2) {
        const int64_t blocks = launches * rows * ((hkv + cand - 1) / cand);
        const int64_t rounds = (blocks + dev.sm_count - 1) / dev.sm_count;
        const double cost = (double)rounds * (kPairBlockFixedUs + cand * us_per_head);
        if (cand == hc || cost < 0.97 * best) { best = cost; best_hc = cand; }
      }
      hc = best_hc;
    }
    if (throughput == 4 && hc > 1 && pair_fine_grain) hc /= 2;
    if (throughput == 2 && hc > 1) hc /= 2;
  } else {
    // Heads per block: as few as it takes for all blocks to be resident at once (more blocks, and the
    // split over tokens then stays inside a block); as many as possible once there are more rows than SMs.
    hc = 1;
    while (hc < hc_max && rows * ((hkv + hc - 1) / hc) > dev.sm_count) hc *= 2;
  }
  // A prefill chunk: the queries of a sequence all gather from the same cache, and blocks run head group by head
  // group (rows fastest), so the rows of the head group in flight are what L2 has to hold: as few heads per
  // block as it takes for them to fit in about 60 % of it (a 128K-token cache: one head, 66 MB).
  if (p.q_per_seq > 1 && rows > dev.sm_count)
    while (hc > 1 && (double)hc * p.max_seq_len * 512.0 > 0.6 * (double)dev.l2_bytes) hc /= 2;
  // every token range should hold at least one 16-token stage
  while (hc < hc_max && (int64_t)(plan.warps / hc) * kAttnStageTokens > p.top_k) hc *= 2;
  plan.heads_per_block = hc;
  plan.head_groups = (hkv + hc - 1) / hc;
  // Rows per block. With many more (row, head group) pairs than the launch needs blocks, a block takes several
  // rows: every warp then walks a longer range (up to a whole row of one KV head: no split, nothing to merge), and
  // the ramp of its pipeline and the merge are paid less often. Kept: at least 2 blocks per SM for a launch on its
  // own, about 32 blocks for one that runs side by side with its neighbours.
  plan.rows_per_block = 1;
  {
    const int per_block = plan.warps / hc;  // (row, range) slots of a block
    const int64_t want_blocks = throughput ? (throughput == 2 ? 64 : 32) : 2 * (int64_t)dev.sm_count;
    // (not for the two-layer decode launches: their heads per block were chosen for the number of blocks they give)
    for (int rb = per_block; rb > 1 && !pair_fine_grain; --rb) {
      if (per_block % rb != 0) continue;
      if ((rows + rb - 1) / rb * plan.head_groups >= want_blocks) { plan.rows_per_block = rb; break; }
    }
  }
  plan.subs = plan.warps / hc / plan.rows_per_block;
  if (throughput) {
    // a handful of (row, KV head) pairs (batch of one): split each over a small cluster until there are 16 blocks
    while (plan.rows_per_block == 1 && c < 8 && rows * plan.head_groups * c < 16 &&
           (int64_t)(c * 2) * plan.subs * kAttnStageTokens <= p.top_k)
      c *= 2;
  } else {
    // Cluster: the largest power of two that still keeps every block resident at once.
    const int64_t blocks = rows * plan.head_groups;
    while (plan.rows_per_block == 1 && c < 8 && blocks * (c * 2) <= max_resident_blocks(c * 2, plan.smem_bytes, plan.warps) &&
           (int64_t)(c * 2) * plan.subs * kAttnStageTokens <= p.top_k)
      c *= 2;
  }
  plan.cluster = c;
  return plan;
}

// The layers of a chain are launched back to back and none waits for its predecessor, so their blocks fill the
// SMs like a list schedule: a block starts when an SM frees up, and a layer's blocks are placed only once the layer
// before it has started all of its own. With equal blocks the last round is usually part empty (16 layers of 32
// blocks on 148 SMs: 3.46 rounds, the fourth with 68 blocks). Blocks of half the size at the end of the chain --
// the last query rows of one layer and every layer behind it -- fill that round at a finer grain. Where the finer
// shape begins: the schedule is simulated for a short list of choices (up to kTailMaxLayers whole layers, and eighths
// of the rows of the layer before them) with a block's duration modelled as a fixed part (launch gap, ramp, merge)
// plus its bytes at the per-SM gather rate, and the best choice is taken if it gains at least 2 %.
//
// Host cost. Blocks of one launch are equal, so the SMs' free times take few distinct values: the schedule is kept
// as a short sorted list of (time, number of SMs) groups and a launch of nb blocks is placed group by group, not
// block by block; the coarse layers that every candidate shares are placed once. A shape that has not been seen
// costs a few microseconds; results are memoised (LRU, keyed on every input of the model), and the lock guards only
// the memo, not the simulation.
namespace {

constexpr int kTailMaxLayers = 3;       // whole layers the finer shape may take (the last round is at most that deep)
constexpr double kBlockFixedUs = 9.5;   // launch gap + pipeline ramp + merge of one block, measured on a B200
constexpr double kPortBytesPerClock = 64.0 * 0.94;  // L2 -> SM port, and the share of it the gather reaches

// SM free times as sorted groups (ascending time).
struct SmGroups {
  static constexpr int kMax = 24;
  double t[kMax];
  int c[kMax];
  int n;
  void init(int sms) { n = 1; t[0] = 0.0; c[0] = sms; }
  // Places nb blocks of duration d, none before `gate`; returns the start time of the last one placed.
  double place(int64_t nb, double d, double gate, double& end) {
    double last_start = gate;
    while (nb > 0) {
      const double start = t[0] > gate ? t[0] : gate;
      const int take = (int64_t)c[0] <= nb ? c[0] : (int)nb;
      nb -= take;
      last_start = start;
      const double fin = start + d;
      if (fin > end) end = fin;
      // remove `take` SMs from the first group, add them at time fin
      if (take == c[0]) { for (int i = 1; i < n; ++i) { t[i - 1] = t[i]; c[i - 1] = c[i]; } --n; }
      else c[0] -= take;
      int pos = n;
      while (pos > 0 && t[pos - 1] > fin) --pos;
      if (pos > 0 && t[pos - 1] == fin) { c[pos - 1] += take; continue; }
      if (n == kMax) {  // cannot happen with two block sizes; merge into the last group rather than overflow
        c[n - 1] += take;
        if (fin > t[n - 1]) t[n - 1] = fin;
        continue;
      }
      for (int i = n; i > pos; --i) { t[i] = t[i - 1]; c[i] = c[i - 1]; }
      t[pos] = fin; c[pos] = take; ++n;
    }
    return last_start;
  }
};

struct TailKey {
  int L, sms, clock_khz, k_eff, hb, hf, hkv;  // L: launches of the chain
  int64_t rows;
  int pair;                                   // launches of two layers each (their own block model)
  bool operator==(const TailKey& o) const {
    return L == o.L && sms == o.sms && clock_khz == o.clock_khz && k_eff == o.k_eff && hb == o.hb && hf == o.hf &&
           hkv == o.hkv && rows == o.rows && pair == o.pair;
  }
};

ChainTail simulate_fine_tail(const TailKey& key, int64_t nb_base, int64_t nb_fine, int hg_base, int hg_fine) {
  const ChainTail none = {0, 0};
  // bytes per microsecond that a block copies: the L2-to-SM port for one-layer blocks, what the two-layer kernel reaches
  const double rate = key.pair ? kPairBytesPerUs : kPortBytesPerClock * (double)key.clock_khz * 1e3 / 1e6;
  const double fixed = key.pair ? kPairBlockFixedUs : kBlockFixedUs;
  auto duration = [&](int heads_per_block) { return fixed + (double)heads_per_block * key.k_eff * 512.0 / rate; };
  const double d_base = duration(key.hb), d_fine = duration(key.hf);
  const int L = key.L;
  const int max_tail = L - 1 < kTailMaxLayers ? L - 1 : kTailMaxLayers;
  // state after the coarse layers that every candidate shares: layers [0, L - max_tail - 1)
  SmGroups g;
  g.init(key.sms);
  double end = 0.0, gate = 0.0;
  const int shared = L - max_tail - 1;
  // snapshots[i]: state after `shared + i` coarse layers
  SmGroups snap[kTailMaxLayers + 2];
  double snap_gate[kTailMaxLayers + 2], snap_end[kTailMaxLayers + 2];
  for (int l = 0; l < shared; ++l) gate = g.place(nb_base, d_base, gate, end);
  for (int i = 0; i <= max_tail + 1; ++i) {
    snap[i] = g; snap_gate[i] = gate; snap_end[i] = end;
    if (i <= max_tail) gate = g.place(nb_base, d_base, gate, end);
  }
  const double plain = snap_end[max_tail + 1];  // all L layers coarse
  double best = plain;
  ChainTail best_tail = none;
  const int64_t rows = key.rows;
  // Whole layers only: the chains that still take this route (groups of 9 to 16 query heads; narrower groups go two
  // layers per launch) have no launch of two block sizes.
  const int64_t step = rows;
  for (int tail = 0; tail <= max_tail; ++tail)
    for (int64_t part = 0; part < rows; part += step) {
      if (tail == 0 && part == 0) continue;
      // layers [0, L - tail - 1) coarse; layer L - tail - 1 coarse except its last `part` rows; the last `tail` fine
      const int coarse_layers = L - tail - 1;
      SmGroups h = snap[coarse_layers - shared];
      double gt = snap_gate[coarse_layers - shared], en = snap_end[coarse_layers - shared];
      if (part > 0) {
        const double g0 = gt;
        const double s1 = h.place((rows - part) * hg_base, d_base, g0, en);
        const double s2 = h.place(part * hg_fine, d_fine, g0, en);
        gt = s1 > s2 ? s1 : s2;
      } else {
        gt = h.place(nb_base, d_base, gt, en);
      }
      for (int l = 0; l < tail; ++l) gt = h.place(nb_fine, d_fine, gt, en);
      if (en < best - 1e-9) { best = en; best_tail = ChainTail{tail, 0}; }
    }
  if (best > 0.98 * plain) best_tail = none;
  return best_tail;
}

}  // namespace

ChainTail chain_fine_tail(const clsa_params& p, const DeviceInfo& dev) {
  const int L = p.num_layers;
  if (L < 2) return ChainTail{0, 0};
  // Chains of query-head groups up to 8: the layers go two per launch (an odd last layer on its own); the last of
  // those launches may take the finer shape too.
  const bool pair = p.num_q_heads / p.num_kv_heads <= 8;
  const ChainTail plain = {0, pair ? (L & ~1) : 0};
  if (!pair && p.block_table != nullptr) return plain;  // paged caches: the finer blocks cost more than the fuller last round returns
  // The block models were measured on a B200 (148 SMs); on anything else the chain keeps one block size.
  if (dev.sm_count != 148 || dev.clock_khz <= 0) return plain;
  if (pair && p.q_per_seq != 1) return plain;
  const AttnPlan base = make_attn_plan(p, dev, pair ? 3 : 1), fine = make_attn_plan(p, dev, pair ? 4 : 2);
  if (base.cluster != 1 || fine.cluster != 1 || fine.heads_per_block == base.heads_per_block ||
      base.rows_per_block != 1 || fine.rows_per_block != 1)
    return plain;
  const int64_t rows = (int64_t)p.num_seqs * p.q_per_seq;
  const int64_t nb_base = rows * base.head_groups, nb_fine = rows * fine.head_groups;
  if (nb_base > 4096 || nb_fine > 8192) return plain;  // far more blocks than SMs: the last round is a small part of the whole
  const int launches = pair ? L / 2 : L;
  if (launches < 2) return plain;
  const TailKey key = {launches, dev.sm_count, dev.clock_khz, p.top_k < p.max_seq_len ? p.top_k : p.max_seq_len,
                       base.heads_per_block, fine.heads_per_block, p.num_kv_heads, rows, pair ? 1 : 0};
  struct Entry { TailKey key; ChainTail tail; uint64_t used; };
  constexpr int kMemo = 64;
  static std::mutex mu;
  static Entry memo[kMemo];
  static int filled = 0;
  static uint64_t tick = 0;
  {
    std::lock_guard<std::mutex> lock(mu);
    for (int i = 0; i < filled; ++i)
      if (memo[i].key == key) { memo[i].used = ++tick; return memo[i].tail; }
  }
  ChainTail tail = simulate_fine_tail(key, nb_base, nb_fine, base.head_groups, fine.head_groups);  // outside the lock
  if (pair) tail = ChainTail{2 * tail.layers, L & ~1};  // the model counts launches; the plan counts layers
  {
    std::lock_guard<std::mutex> lock(mu);
    int slot = 0;
    if (filled < kMemo) slot = filled++;
    else for (int i = 1; i < kMemo; ++i) if (memo[i].used < memo[slot].used) slot = i;  // least recently used
    memo[slot] = Entry{key, tail, ++tick};
  }
  return tail;
}

double attn_alone_occupancy(const clsa_params& p, const DeviceInfo& dev) {
  const AttnPlan plan = make_attn_plan(p, dev, 0);
  const int64_t rows = (int64_t)p.num_seqs * p.q_per_seq;
  const int64_t blocks = (rows + plan.rows_per_block - 1) / plan.rows_per_block * plan.cluster * plan.head_groups;
  const int64_t rounds = (blocks + dev.sm_count - 1) / dev.sm_count;
  return (double)blocks / (double)(rounds * dev.sm_count);
}

cudaError_t launch_sparse_attn(const clsa_params& p, const void* q, const int32_t* idx, const int32_t* count, void* out,
                               float* lse, uint32_t* status, int reverse, int wait_prior, int only_q_pending,
                               int keep_for_next, int throughput_plan, const void* q2, void* out2,
                               const DeviceInfo& dev, cudaStream_t stream) {
  const AttnPlan plan = make_attn_plan(p, dev, throughput_plan);
  const bool pair = q2 != nullptr && out2 != nullptr;
  AttnArgs a;
  a.q = static_cast<const uint16_t*>(q);
  a.q2 = static_cast<const uint16_t*>(q2);
  a.out2 = static_cast<uint16_t*>(out2);
  a.kc = static_cast<const uint16_t*>(p.k_cache);
  a.vc = static_cast<const uint16_t*>(p.v_cache);
  a.tok_stride = p.kv_token_stride;
  a.head_stride = p.kv_head_stride;
  a.seq_start = p.seq_start;
  a.seq_len = p.seq_len;
  a.idx = idx;
  a.count = count;
  a.block_table = p.block_table;
  a.block_shift = 0;
  while (p.block_table != nullptr && (1 << a.block_shift) < p.block_size) ++a.block_shift;
  a.max_blocks = p.max_blocks_per_seq;
  a.out = static_cast<uint16_t*>(out);
  a.lse = lse;
  a.status = status;
  a.q_per_seq = p.q_per_seq;
  a.num_q_heads = p.num_q_heads;
  a.num_kv_heads = p.num_kv_heads;
  a.group = p.num_q_heads / p.num_kv_heads;
  a.top_k = p.top_k;
  a.heads_per_block = plan.heads_per_block;
  a.subs = plan.subs;
  a.rows_per_block = plan.rows_per_block;
  a.num_rows = (int64_t)p.num_seqs * p.q_per_seq;
  a.reverse = reverse;
  a.wait_prior = wait_prior;
  a.early = (wait_prior && only_q_pending) ? 1 : 0;
  // L2 priority of the gathered rows. A launch with a successor that will read the same rows (the chained layers)
  // fetches all of them with evict_last, so that scores, indices and outputs passing through L2 do not push them
  // out before the layers behind it arrive; a launch on its own leaves the replacement policy alone.
  a.keep = keep_for_next ? 1 : 0;
  // A launch with the GPU to itself whose rows the next launch reads again keeps the share of them in L2 that fits
  // there (pinned_stages_of_eight); chained launches trail one another over the same rows and fetch everything
  // evict_last.
  a.pin = (keep_for_next && throughput_plan == 0) ? pinned_stages_of_eight(p, dev) : -1;
  a.max_seq_len = p.max_seq_len;
  a.scale_log2 = p.sm_scale * kLog2e;
  // With the extent of the row space known (num_cache_rows) and below 2^32 16-byte units, row offsets are 32-bit.
  a.rows_max = p.num_cache_rows;
  a.off32 = (a.rows_max > 0 && (double)a.rows_max * (double)(p.kv_token_stride >> 3) < 4294967296.0) ? 1 : 0;
  void (*kernel)(const AttnArgs);
  const bool multi = plan.rows_per_block > 1, pg = p.block_table != nullptr;
#define CLSA_ATTN_PICK(NT_, W_)                                                                      \
  (multi ? (pg ? sparse_attn_kernel<NT_, true, W_, true> : sparse_attn_kernel<NT_, false, W_, true>) \
         : (pg ? sparse_attn_kernel<NT_, true, W_, false> : sparse_attn_kernel<NT_, false, W_, false>))
  if (a.group > 8) kernel = CLSA_ATTN_PICK(2, kAttnWarpsWide);
  else if (plan.warps == kAttnWarpsNarrow) kernel = CLSA_ATTN_PICK(1, kAttnWarpsNarrow);
  else kernel = CLSA_ATTN_PICK(1, kAttnWarpsWide);
#undef CLSA_ATTN_PICK
  if (pair) kernel = multi ? (pg ? sparse_attn_kernel<2, true, kAttnWarpsWide, true, true>
                                 : sparse_attn_kernel<2, false, kAttnWarpsWide, true, true>)
                           : (pg ? sparse_attn_kernel<2, true, kAttnWarpsWide, false, true>
                                 : sparse_attn_kernel<2, false, kAttnWarpsWide, false, true>);
  cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem_bytes);
  if (err != cudaSuccess) return err;
  const int64_t rows = (int64_t)p.num_seqs * p.q_per_seq;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((rows + plan.rows_per_block - 1) / plan.rows_per_block * plan.cluster), (unsigned)plan.head_groups, 1);
  cfg.blockDim = dim3((unsigned)plan.warps * 32, 1, 1);
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
  return cudaLaunchKernelEx(&cfg, kernel, a);
}

}  // namespace clsa
