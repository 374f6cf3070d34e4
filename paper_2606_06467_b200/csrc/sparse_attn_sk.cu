// GQA sparse attention over the selected rows only (Eq. 4) for decoding (one query per sequence), one launch per
// cross-decoder layer, with the work cut at token granularity so that every SM gets the same share whatever the
// batch size.
//
// The kernel in sparse_attn.cu hands whole (query row, KV head) units to blocks: 16 rows x 8 KV heads are 128
// blocks on 148 SMs, 20 rows are 160 blocks in two rounds. Here the launch is a flat list of 16-token stages,
//   stage id = ((row * Hkv + kv head) * NS + stage of the row's k slots),   NS = ceil(k / 16),
// and worker w of W (a warp; block b holds workers b * wpb .. b * wpb + wpb - 1, one block per SM) takes a contiguous
// span of the TS stages: the first TS % W workers TS / W + 1 of them, the others TS / W. A span may end inside one (row, KV head) unit
// and continue in the next; each piece ("segment") is streamed through the warp's private cp.async ring exactly as
// in the other kernel (16-byte copies with an L2 priority, tokens along M of a warp-level bf16 MMA with the GQA
// group in its 8 columns, online softmax in the exp2 domain).
//
// Split-K merge across warps AND blocks, without spinning. A segment that covers its whole unit is normalised and
// written out by its warp alone. Otherwise the warp parks the segment's unnormalised partial (per query head: 128
// outputs, running max, running sum): the last segment of its span in its own, now idle, staging ring, an earlier
// one in a global slot of its own. After one block barrier the (unit, query head) pairs that the block touched are
// dealt over its warps; a job combines the block's partials of its pair by log-sum-exp in worker order. If the block
// holds all of the unit the job writes the output; if the unit straddles blocks it leaves a block-level partial in a
// global slot, fences, and adds one to the pair's arrival counter -- the job whose add completes the pair (the number
// of blocks a unit straddles follows from the static split) reads the blocks' partials back in block order, so the
// result does not depend on who arrived last, writes the output and puts the counter back to zero for the next
// launch. The scratch is a few MB and stays in L2 between the write and the read.
//
// Launches whose only pending input is the query tensor (hint only_q_pending: the index and the caches were
// complete before the kernel in front of this one started, as for every layer of a decoder after the first) issue
// their first two stages of row copies before they wait for that kernel, so the ramp of the pipeline overlaps the
// predecessor's tail.
//
// The same kernel with its arithmetic compiled out is the gather probe (clsa_gather_probe): the access pattern
// alone, for measuring what the memory system delivers to it.
#include "attn_common.cuh"

namespace clsa {
namespace {

constexpr int kMergeBatch = 8;
// Release/acquire fence at GPU scope (what the message-passing pattern of the merge needs; __threadfence() is the
// sequentially consistent fence, several times as expensive with every block of the grid issuing it at once).
__device__ __forceinline__ void fence_acq_rel_gpu() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }
constexpr int kMinStagesPerWorker = 4;  // spans shorter than this cost more in partials than they return in parallelism

struct SkArgs {
  const uint16_t* q;
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
  float* lse;
  uint32_t* status;
  int q_per_seq, num_q_heads, num_kv_heads, group, top_k, max_seq_len;
  int reverse;     // 1: the whole stage list is walked from its end (the rows the previous launch read last come first)
  int wait_prior;  // 1: inputs may come from the kernel launched just before this one
  int early;       // 1 (with wait_prior): only q is pending; index, counts and caches may be read before the wait
  int keep;        // 1: launches behind this one read the same rows again
  int pin;         // -1: every row is fetched with one L2 priority (evict_last if keep, else the default). 0..8: of every
                   // 8 consecutive stages of a unit the first `pin` are fetched evict_last and the others evict_first
  int off32;       // every row offset of the caches fits 32 bits when counted in 16-byte units
  int64_t rows_max;
  int unit_stages;       // NS
  int total_stages;      // TS = rows * Hkv * NS (< 2^31)
  int aligned, span_q, span_rem;  // the split of the stages over the workers (struct Split)
  int workers;           // W <= gridDim.x * wpb, W <= TS
  int wpb;               // workers per block (<= warps per block; the warps beyond them only help with the merge)
  float* part;           // partial slots of [group][kPartialStride] floats: W "early" slots (slot w: a partial that worker
                         // w had to park before the end of its span), then gridDim.x + units block-level slots (slot of
                         // (block b, unit u) = b + u)
  uint32_t* arrive;      // [units][group] arrival counters, zero between launches
  float scale_log2;
};

// The split of the stage list over the workers, in 32-bit arithmetic. Two forms:
//   aligned (W >= units and the units' worker counts differ little): unit u gets n = W / units workers, the first
//     W % units units one more, and a unit's NS stages are cut evenly over its own workers -- no span crosses a unit
//     boundary, so no worker has to restart its pipeline inside its span;
//   flat: the first TS % W workers own TS / W + 1 consecutive stages, the others TS / W (spans cross unit boundaries).
struct Split {
  int aligned;
  int q, rem;  // aligned: W / units, W % units. flat: TS / W, TS % W.
  int NS;
};
__device__ __forceinline__ int span_begin(int w, const Split& sp) {
  if (!sp.aligned) return w * sp.q + min(w, sp.rem);
  const int big = sp.rem * (sp.q + 1);  // workers of the units that have q + 1 of them
  int u, j, n;
  if (w < big) { n = sp.q + 1; u = w / n; j = w - u * n; }
  else { n = sp.q; const int w2 = w - big; const int u2 = w2 / n; u = sp.rem + u2; j = w2 - u2 * n; }
  return u * sp.NS + (j * sp.NS) / n;
}
// first and last worker of unit u (the workers whose spans reach into it)
__device__ __forceinline__ void unit_workers(int u, const Split& sp, int& first, int& last) {
  if (sp.aligned) {
    first = u * sp.q + min(u, sp.rem);
    last = first + sp.q + (u < sp.rem ? 1 : 0) - 1;
  } else {
    const int big = sp.rem * (sp.q + 1);
    auto owner = [&](int s) { return s < big ? s / (sp.q + 1) : sp.rem + (s - big) / sp.q; };
    first = owner(u * sp.NS);
    last = owner(u * sp.NS + sp.NS - 1);
  }
}

template <int NT, bool PAGED, int WARPS, bool PROBE>
__global__ void __launch_bounds__(WARPS * 32, 1) sparse_attn_sk_kernel(const SkArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int G = a.group;
  const int NS = a.unit_stages;
  const int W = a.workers;
  const Split split = {a.aligned, a.span_q, a.span_rem, NS};
  const int w = (int)blockIdx.x * a.wpb + warp;  // block b holds workers b * wpb ..
  const bool has_work = warp < a.wpb && w < W;
  const int s_begin = has_work ? span_begin(w, split) : 0;
  const int s_end = has_work ? (w + 1 < W ? span_begin(w + 1, split) : a.total_stages) : 0;

  unsigned long long probe_t0 = 0;
  if (PROBE) asm volatile("mov.u64 %0, %globaltimer;" : "=l"(probe_t0));
  unsigned char* ring = smem + warp * kWarpRingBytes;
  const uint32_t ring_u32 = smem_u32(ring);
  uint32_t* stage_mask = reinterpret_cast<uint32_t*>(smem + WARPS * kWarpRingBytes) + warp * kAttnStages;
  int2* span_tab = reinterpret_cast<int2*>(smem + WARPS * kWarpRingBytes + WARPS * kAttnStages * sizeof(uint32_t));
  if (lane == 0) span_tab[warp] = make_int2(s_begin, s_end);  // read by the block's merge, behind its barrier

  // Fragment coordinates (products are formed transposed, tokens along M):
  //   S^T[16 tokens x 8 heads] = K[16 x 128] Q^T,   O^T[128 x 8 heads] += V^T[128 x 16 tokens] P^T
  const int rowq = lane >> 2;
  const int hcol = (lane & 3) * 2;

  // Programmatic dependent launch. A kernel that has something to wait for lets its own dependents go only after
  // its wait: a kernel behind it may skip its wait on the grounds that everything it reads was complete before THIS
  // grid started reading, which holds only if this grid has waited before it releases anybody.
  bool waited = !a.wait_prior;
  if (a.wait_prior && !a.early) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    waited = true;
  }
  if (waited) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  auto wait_now = [&]() {  // before the first read of q and before any global write
    if (!waited) {
      asm volatile("griddepcontrol.wait;" ::: "memory");
      asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
      waited = true;
    }
  };

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
  const uint32_t stride16 = (uint32_t)(a.tok_stride >> 3);  // row stride in 16-byte units
  uint32_t probe_sum = 0;

  int cur = a.reverse ? s_end : s_begin;
  while (a.reverse ? cur > s_begin : cur < s_end) {
    // ---- the next segment of this worker's span: stages [seg_lo, seg_hi) of unit u --------------------------------
    const int u = (a.reverse ? cur - 1 : cur) / NS;
    const int seg_lo = max(s_begin, u * NS), seg_hi = min(s_end, (u + 1) * NS);
    cur = a.reverse ? seg_lo : seg_hi;
    const int r = u / a.num_kv_heads;               // query row
    const int g = u - r * a.num_kv_heads;           // KV head
    const int h0 = g * G;                           // first query head of this KV head
    const int slot_lo = (seg_lo - u * NS) * kAttnStageTokens;
    const int slot_hi = min(a.top_k, (seg_hi - u * NS) * kAttnStageTokens);
    const int32_t* row_idx = a.idx + (int64_t)r * a.top_k;
    const int b = r / a.q_per_seq;
    constexpr bool paged = PAGED;
    // Positions are fetched two pipeline steps before they are used and (paged caches) their block numbers one step
    // before. The first three steps' positions are fetched together with the count, speculatively for a range that
    // lies entirely below it (entries past the count are never used).
    const int nst_full = (slot_hi - slot_lo + kAttnStageTokens - 1) / kAttnStageTokens;
    int spec_raw[3] = {-1, -1, -1};
    if (lane < kAttnStageTokens) {
#pragma unroll
      for (int i = 0; i < 3; ++i) {
        const int tt = slot_lo + (a.reverse ? nst_full - 1 - i : i) * kAttnStageTokens + lane;
        if (i < nst_full && tt < slot_hi) spec_raw[i] = row_idx[tt];
      }
    }
    int cnt = a.count[r];
    // A sequence whose length lies outside its declared bounds is never read: with n = 0 no position passes the range
    // check, every stage is masked, and the row comes out as zeros with lse = -inf (a select, not a branch: the length
    // is first needed when the first copies are issued; the flag is raised behind the segment's loop).
    const int n_raw = a.seq_len[b];
    const bool n_ok = n_raw >= a.q_per_seq && n_raw <= a.max_seq_len;
    const int n = n_ok ? n_raw : 0;
    const int64_t s0 = paged ? 0 : a.seq_start[b];
    const int32_t* table = paged ? a.block_table + (int64_t)b * a.max_blocks : nullptr;
    const bool first_of_row = slot_lo == 0 && g == 0;  // one segment per row reports the row's problems
    if (cnt < 0 || cnt > a.top_k) {
      if (lane == 0 && first_of_row) flag_status(a.status, CLSA_DEV_BAD_COUNT);
      cnt = cnt < 0 ? 0 : a.top_k;
    }
    const int t_lo = min(cnt, slot_lo), t_hi = min(cnt, slot_hi);

    float o[NT][8][4];                     // O^T: [head tile][16-wide slice of D][c0..c3]
    float mA[NT], mB[NT], lA[NT], lB[NT];  // running max / sum of heads hcol and hcol+1 (log2 domain)
    float lacc[NT][4];                     // the sums as an MMA accumulator (ones[16 x 16] . P^T)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      mA[nt] = -INFINITY; mB[nt] = -INFINITY; lA[nt] = 0.f; lB[nt] = 0.f;
      lacc[nt][0] = 0.f; lacc[nt][1] = 0.f; lacc[nt][2] = 0.f; lacc[nt][3] = 0.f;
#pragma unroll
      for (int j = 0; j < 8; ++j) { o[nt][j][0] = 0.f; o[nt][j][1] = 0.f; o[nt][j][2] = 0.f; o[nt][j][3] = 0.f; }
    }

    if (t_lo < t_hi) {
      const int nstages = (t_hi - t_lo + kAttnStageTokens - 1) / kAttnStageTokens;
      const char* kbytes = reinterpret_cast<const char*>(a.kc + g * a.head_stride + (lane & 15) * 8);
      const char* vbytes = reinterpret_cast<const char*>(a.vc + g * a.head_stride + (lane & 15) * 8);
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
              const int64_t off = (s0 + (ok ? tok : 0)) * a.tok_stride * 2;  // bytes
              cp_async16(kdst + sw[it], kbytes + off, ok, pol);
              cp_async16(vdst + sw[it], vbytes + off, ok, pol);
            }
          }
        }
        cp_async_commit();
      };

      // Prologue: stages 0 and 1 in flight (both buffers of the ring are free); the positions of stage 2 and its
      // block numbers, and the positions of stage 3, in registers.
      int r0 = spec_raw[0], r1 = spec_raw[1], rawX = spec_raw[2];
      if (t_hi != slot_hi) {  // the count cuts this range short: fetch the real first positions
        r0 = load_raw(0); r1 = load_raw(1); rawX = load_raw(2);
      }
      int rawY = load_raw(3);
      {
        const int b0 = load_blk(r0), b1 = load_blk(r1);
        issue(0, r0, b0);
        issue(1, r1, b1);
      }
      int blkX = load_blk(rawX);
      // Nothing read so far can still be in the making when only q is pending: the wait comes here, behind two
      // stages of copies, and q is read behind it.
      wait_now();
      uint32_t qb[NT][8][2];
      if (!PROBE) {
        // Q^T fragments (B operand, 128 x 8 per head tile): head = rowq, two consecutive d per register
        const uint16_t* qbase = a.q + ((int64_t)r * a.num_q_heads + h0) * 128;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const int head = nt * 8 + rowq;
          const bool hv = head < G;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            const int d = ks * 16 + hcol;
            qb[nt][ks][0] = hv ? *reinterpret_cast<const uint32_t*>(qbase + head * 128 + d) : 0u;
            qb[nt][ks][1] = hv ? *reinterpret_cast<const uint32_t*>(qbase + head * 128 + d + 8) : 0u;
          }
        }
      }
#pragma unroll 1
      for (int i = 0; i < nstages; ++i) {
        // advance the position pipeline: positions of stage i + 4, block numbers of stage i + 3
        const int raw_new = load_raw(i + 4);
        const int blk_new = load_blk(rawY);
        cp_async_wait<kAttnStages - 1>();  // stage i has landed (stage i + 1 may still be in flight)
        __syncwarp();
        const int buf = i % kAttnStages;
        const uint32_t kbuf = ring_u32 + buf * kStageBytes, vbuf = kbuf + kStageBytes / 2;
        const uint32_t okmask = stage_mask[buf];
        if (PROBE) {
          // the access pattern alone: touch the stage so that the copies cannot be dropped
          uint4 t4;
          asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                       : "=r"(t4.x), "=r"(t4.y), "=r"(t4.z), "=r"(t4.w) : "r"(kbuf + (uint32_t)lane * 16u));
          probe_sum ^= t4.x ^ t4.y ^ t4.z ^ t4.w ^ okmask;
          asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];"
                       : "=r"(t4.x), "=r"(t4.y), "=r"(t4.z), "=r"(t4.w) : "r"(vbuf + (uint32_t)lane * 16u));
          probe_sum ^= t4.x ^ t4.y ^ t4.z ^ t4.w;
        } else {
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
          // taken over the raw dot products (the scale is positive) and the scale rides in the exponent's multiply-add.
          const bool full = okmask == 0xffffu;  // the usual stage: nothing to mask
          const bool ok_lo = (okmask >> rowq) & 1u, ok_hi = (okmask >> (rowq + 8)) & 1u;
          uint32_t pb0[NT], pb1[NT];
          bool rescale = false;
          float alphaA[NT], alphaB[NT];
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            float x0 = s[nt][0], x1 = s[nt][1], x2 = s[nt][2], x3 = s[nt][3];  // tokens rowq (x0, x1) and rowq + 8; heads hcol, hcol + 1
            if (!full) {
              x0 = ok_lo ? x0 : -INFINITY; x1 = ok_lo ? x1 : -INFINITY;
              x2 = ok_hi ? x2 : -INFINITY; x3 = ok_hi ? x3 : -INFINITY;
            }
            float mxA = fmaxf(x0, x2), mxB = fmaxf(x1, x3);
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
            const uint32_t p_lo = pack_bf16x2(fast_exp2(fmaf(x0, a.scale_log2, -muA)), fast_exp2(fmaf(x1, a.scale_log2, -muB)));
            const uint32_t p_hi = pack_bf16x2(fast_exp2(fmaf(x2, a.scale_log2, -muA)), fast_exp2(fmaf(x3, a.scale_log2, -muB)));
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
        }
        __syncwarp();  // everyone is done with this buffer before it is refilled
        issue(i + kAttnStages, rawX, blkX);
        rawX = rawY;
        blkX = blk_new;
        rawY = raw_new;
      }
      cp_async_wait<0>();
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) { lA[nt] = lacc[nt][0]; lB[nt] = lacc[nt][1]; }
    }
    wait_now();  // a segment without tokens has read nothing yet; what follows writes global memory
    if (!n_ok && lane == 0 && first_of_row) flag_status(a.status, CLSA_DEV_BAD_SEQLEN);
    if (PROBE) continue;

    // ---- what becomes of this segment's result ---------------------------------------------------------------------
    // Staged through the warp's ring (idle between segments: every copy has landed) so that global stores are 16
    // bytes per lane and contiguous.
    float* mypart = reinterpret_cast<float*>(ring);
    const bool whole = seg_lo == u * NS && seg_hi == (u + 1) * NS;  // nobody else works on this unit
    __syncwarp();
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int headA = nt * 8 + hcol, headB = headA + 1;
      // a whole unit is normalised here; a partial keeps its unnormalised sums next to (max, sum)
      const float iA = whole ? (lA[nt] > 0.f ? 1.f / lA[nt] : 0.f) : 1.f, iB = whole ? (lB[nt] > 0.f ? 1.f / lB[nt] : 0.f) : 1.f;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int d = 16 * j + rowq;
        if (headA < G) { mypart[headA * kPartialStride + d] = o[nt][j][0] * iA; mypart[headA * kPartialStride + d + 8] = o[nt][j][2] * iA; }
        if (headB < G) { mypart[headB * kPartialStride + d] = o[nt][j][1] * iB; mypart[headB * kPartialStride + d + 8] = o[nt][j][3] * iB; }
      }
      if (rowq == 0) {
        if (headA < G) *reinterpret_cast<float2*>(mypart + headA * kPartialStride + 128) = make_float2(mA[nt], lA[nt]);
        if (headB < G) *reinterpret_cast<float2*>(mypart + headB * kPartialStride + 128) = make_float2(mB[nt], lB[nt]);
      }
    }
    __syncwarp();
    if (whole) {
      for (int hh = 0; hh < G; ++hh) {
        const float4 v = *reinterpret_cast<const float4*>(mypart + hh * kPartialStride + lane * 4);
        const float2 ml = *reinterpret_cast<const float2*>(mypart + hh * kPartialStride + 128);
        const int64_t item = (int64_t)r * a.num_q_heads + h0 + hh;
        uint2 packed;
        packed.x = pack_bf16x2(v.x, v.y);
        packed.y = pack_bf16x2(v.z, v.w);
        *reinterpret_cast<uint2*>(a.out + item * 128 + lane * 4) = packed;
        if (a.lse != nullptr && lane == 0) a.lse[item] = ml.y > 0.f ? (ml.x + log2f(ml.y)) * kLn2 : -INFINITY;
      }
      __syncwarp();  // the ring is reused by the next segment
    } else if (a.reverse ? cur > s_begin : cur < s_end) {
      // more segments follow and will reuse the ring: this partial waits in the worker's global slot
      const int rec4 = G * (kPartialStride / 4);
      float4* dst = reinterpret_cast<float4*>(a.part) + (int64_t)w * rec4;
      const float4* srcp = reinterpret_cast<const float4*>(mypart);
      for (int i = lane; i < rec4; i += 32) __stcg(dst + i, srcp[i]);
      __syncwarp();
    }
    // else: the last segment of the span; its partial stays in the ring for the block's merge
  }
  wait_now();  // a warp without work still takes part in the launch's dependency protocol
  if (PROBE) {
    if (has_work) reinterpret_cast<uint32_t*>(a.part)[(int64_t)w * 32 + lane] = probe_sum;
    // The launch's own duration, for the caller to read: the earliest start (as its complement, so that both words
    // accumulate by maximum from a cleared header) and the latest end over all warps, in globaltimer nanoseconds.
    if (lane == 0 && a.status != nullptr) {
      unsigned long long t1;
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t1));
      unsigned long long* clockwords = reinterpret_cast<unsigned long long*>(a.status);
      atomicMax(clockwords + 1, ~probe_t0);
      atomicMax(clockwords + 2, t1);
    }
    return;
  }
  __syncthreads();  // every partial of this block is parked (shared-memory and global writes of the block are visible)

  // ---- block-level merge: (unit, query head) jobs dealt over the warps -----------------------------------------------
  const int w_blk0 = (int)blockIdx.x * a.wpb;
  if (w_blk0 >= W) return;
  const int nw = min(W - w_blk0, a.wpb);                                        // workers of this block
  const int b_lo = span_tab[0].x, b_hi = span_tab[nw - 1].y;                     // the block's stages
  const int u_first = b_lo / NS, u_last = (b_hi - 1) / NS;
  const int rec4 = G * (kPartialStride / 4);                                    // float4 per partial record
  const float4* early = reinterpret_cast<const float4*>(a.part);
  float4* bpart = reinterpret_cast<float4*>(a.part) + (int64_t)W * rec4;
  const int njobs = (u_last - u_first + 1) * G;
  for (int job = warp; job < njobs; job += WARPS) {
    const int u = u_first + job / G;
    const int hh = job % G;
    const int us = u * NS, ue = us + NS;                                        // the unit's stages
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float L = 0.f, M = -INFINITY;
    // fold partial (m, l, v) into the running (M, L, acc); the order of the folds is fixed by the caller's loop
    auto fold = [&](float2 ml, float4 v) {
      const float Mn = fmaxf(M, ml.x);
      const float mu = Mn == -INFINITY ? 0.f : Mn;
      const float so = fast_exp2(M - mu), sn = fast_exp2(ml.x - mu);
      acc.x = fmaf(sn, v.x, acc.x * so); acc.y = fmaf(sn, v.y, acc.y * so);
      acc.z = fmaf(sn, v.z, acc.z * so); acc.w = fmaf(sn, v.w, acc.w * so);
      L = fmaf(sn, ml.y, L * so);
      M = Mn;
    };
    bool done = false;  // one worker had the unit whole: it has written the output already
    for (int lw = 0; lw < nw; ++lw) {  // the block's workers in order; those whose span reaches into the unit contribute
      const int2 sp = span_tab[lw];
      if (sp.x >= ue || sp.y <= us) continue;
      if (sp.x <= us && sp.y >= ue) { done = true; break; }
      // the worker's partial of this unit: in its ring if the unit was the last of its walk, else in its global slot
      const int last_stage = a.reverse ? sp.x : sp.y - 1;
      float2 ml;
      float4 v;
      if (last_stage >= us && last_stage < ue) {
        const float* pr = reinterpret_cast<const float*>(smem + lw * kWarpRingBytes) + hh * kPartialStride;
        ml = *reinterpret_cast<const float2*>(pr + 128);
        v = *reinterpret_cast<const float4*>(pr + lane * 4);
      } else {
        const float4* pr = early + (int64_t)(w_blk0 + lw) * rec4 + hh * (kPartialStride / 4);
        ml = __ldcg(reinterpret_cast<const float2*>(pr + 32));
        v = __ldcg(pr + lane);
      }
      fold(ml, v);
    }
    if (done) continue;
    const int r = u / a.num_kv_heads;
    const int64_t item = (int64_t)r * a.num_q_heads + (u - r * a.num_kv_heads) * G + hh;
    if (!(b_lo <= us && b_hi >= ue)) {
      // the unit straddles blocks: leave this block's partial, arrive, and finish the pair if this completes it
      float4* slot = bpart + (int64_t)(blockIdx.x + u) * rec4 + hh * (kPartialStride / 4);
      __stcg(slot + lane, acc);
      if (lane == 0) __stcg(reinterpret_cast<float2*>(slot + 32), make_float2(M, L));
      fence_acq_rel_gpu();  // release: this block's partial before its arrival
      __syncwarp();
      int wf, wl;
      unit_workers(u, split, wf, wl);
      const int blk_first = wf / a.wpb, blk_last = wl / a.wpb;
      unsigned prev = 0;
      if (lane == 0) prev = atomicAdd(a.arrive + u * G + hh, 1u);
      prev = __shfl_sync(0xffffffffu, prev, 0);
      if (prev + 1u != (unsigned)(blk_last - blk_first + 1)) continue;
      fence_acq_rel_gpu();  // acquire: the other blocks' partials are visible behind their arrivals
      if (lane == 0) a.arrive[u * G + hh] = 0u;  // ready for the next launch on this scratch
      acc = make_float4(0.f, 0.f, 0.f, 0.f);
      L = 0.f;
      M = -INFINITY;
      for (int b2 = blk_first; b2 <= blk_last; b2 += kMergeBatch) {  // in block order, a batch of loads in flight
        float2 ml[kMergeBatch];
        float4 v[kMergeBatch];
#pragma unroll
        for (int i = 0; i < kMergeBatch; ++i) {
          if (b2 + i <= blk_last) {
            const float4* pr = bpart + (int64_t)(b2 + i + u) * rec4 + hh * (kPartialStride / 4);
            ml[i] = __ldcg(reinterpret_cast<const float2*>(pr + 32));
            v[i] = __ldcg(pr + lane);
          }
        }
#pragma unroll
        for (int i = 0; i < kMergeBatch; ++i)
          if (b2 + i <= blk_last) fold(ml[i], v[i]);
      }
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
    uint2 packed;
    packed.x = pack_bf16x2(acc.x * inv, acc.y * inv);
    packed.y = pack_bf16x2(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2*>(a.out + item * 128 + lane * 4) = packed;
    if (a.lse != nullptr && lane == 0) a.lse[item] = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
  }
}

}  // namespace

// ---------------------------------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------------------------------
SkPlan make_sk_plan(const clsa_params& p, const DeviceInfo& dev) {
  SkPlan plan;
  plan.warps = p.num_q_heads / p.num_kv_heads <= 8 ? kAttnWarpsNarrow : kAttnWarpsWide;
  plan.smem_bytes = (size_t)plan.warps * kWarpRingBytes + plan.warps * (kAttnStages * sizeof(uint32_t) + sizeof(int2));
  const int64_t rows = (int64_t)p.num_seqs * p.q_per_seq;
  plan.units = rows * p.num_kv_heads;
  plan.unit_stages = (p.top_k + kAttnStageTokens - 1) / kAttnStageTokens;
  plan.total_stages = plan.units * plan.unit_stages;
  int64_t blocks = dev.sm_count;
  int64_t workers = plan.total_stages / kMinStagesPerWorker;
  if (workers < 1) workers = 1;
  if (workers > blocks * plan.warps) workers = blocks * plan.warps;
  if (blocks > workers) blocks = workers;
  plan.wpb = (int)((workers + blocks - 1) / blocks);  // a small launch is spread thinly over the SMs
  plan.blocks = (int)((workers + plan.wpb - 1) / plan.wpb);
  plan.workers = (int)workers;
  // Unit-aligned split when every unit can have workers of its own and the longest span that results (a unit with
  // the fewest workers) stays within 15 % of the even share.
  plan.aligned = 0;
  if (workers >= plan.units) {
    const int64_t n_lo = workers / plan.units;
    const int64_t longest = (plan.unit_stages + n_lo - 1) / n_lo;
    if (longest * workers * 100 <= plan.total_stages * 115) plan.aligned = 1;
  }
  return plan;
}

// Scratch of one launch: an arrival counter per (unit, query head of the group), and the partial slots -- one per
// worker (a partial parked before the end of a span) and one per (block, unit) pair that can occur (at most
// blocks + units of them).
size_t sk_counter_bytes(const clsa_params& p, const SkPlan& plan) {
  const size_t group = (size_t)(p.num_q_heads / p.num_kv_heads);
  return ((size_t)plan.units * group * sizeof(uint32_t) + 255) / 256 * 256;
}
size_t sk_partial_bytes(const clsa_params& p, const SkPlan& plan) {
  const size_t group = (size_t)(p.num_q_heads / p.num_kv_heads);
  const size_t slots = (size_t)plan.workers + (size_t)plan.blocks + (size_t)plan.units;
  return (slots * group * kPartialStride * sizeof(float) + 255) / 256 * 256;
}

namespace {

template <bool PROBE>
cudaError_t launch_sk(const clsa_params& p, const SkPlan& plan, const void* q, const int32_t* idx, const int32_t* count,
                      void* out, float* lse, uint32_t* status, uint32_t* arrive, float* part, int reverse, int wait_prior,
                      int only_q_pending, int keep_rows, const DeviceInfo& dev, cudaStream_t stream) {
  SkArgs a;
  a.q = static_cast<const uint16_t*>(q);
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
  a.max_seq_len = p.max_seq_len;
  a.reverse = reverse ? 1 : 0;
  a.wait_prior = wait_prior ? 1 : 0;
  a.early = (wait_prior && only_q_pending) ? 1 : 0;
  a.keep = keep_rows ? 1 : 0;
  // L2 policy of a launch whose rows the next launch reads again: see kPinOfEight.
  a.pin = keep_rows ? pinned_stages_of_eight(p, dev) : -1;
  // With the extent of the row space known (num_cache_rows) and below 2^32 16-byte units, row offsets are 32-bit.
  a.rows_max = p.num_cache_rows;
  a.off32 = (a.rows_max > 0 && (double)a.rows_max * (double)(p.kv_token_stride >> 3) < 4294967296.0) ? 1 : 0;
  a.unit_stages = plan.unit_stages;
  if (plan.total_stages >= ((int64_t)1 << 31)) return cudaErrorInvalidValue;  // refused by the entry points before this
  a.total_stages = (int)plan.total_stages;
  a.aligned = plan.aligned;
  a.span_q = plan.aligned ? (int)(plan.workers / plan.units) : (int)(plan.total_stages / plan.workers);
  a.span_rem = plan.aligned ? (int)(plan.workers % plan.units) : (int)(plan.total_stages % plan.workers);
  a.workers = plan.workers;
  a.wpb = plan.wpb;
  a.arrive = arrive;
  a.part = part;
  a.scale_log2 = p.sm_scale * kLog2e;
  void (*kernel)(const SkArgs);
  const bool pg = p.block_table != nullptr;
  if (a.group > 8) kernel = pg ? sparse_attn_sk_kernel<2, true, kAttnWarpsWide, PROBE> : sparse_attn_sk_kernel<2, false, kAttnWarpsWide, PROBE>;
  else kernel = pg ? sparse_attn_sk_kernel<1, true, kAttnWarpsNarrow, PROBE> : sparse_attn_sk_kernel<1, false, kAttnWarpsNarrow, PROBE>;
  cudaError_t err = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem_bytes);
  if (err != cudaSuccess) return err;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)plan.blocks, 1, 1);
  cfg.blockDim = dim3((unsigned)plan.warps * 32, 1, 1);
  cfg.dynamicSmemBytes = plan.smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, a);
}

}  // namespace

cudaError_t launch_sparse_attn_sk(const clsa_params& p, const SkPlan& plan, const void* q, const int32_t* idx,
                                  const int32_t* count, void* out, float* lse, uint32_t* status, uint32_t* arrive,
                                  float* part, int reverse, int wait_prior, int only_q_pending, int keep_rows,
                                  const DeviceInfo& dev, cudaStream_t stream) {
  return launch_sk<false>(p, plan, q, idx, count, out, lse, status, arrive, part, reverse, wait_prior, only_q_pending,
                          keep_rows, dev, stream);
}

cudaError_t launch_gather_probe(const clsa_params& p, const SkPlan& plan, const int32_t* idx, const int32_t* count,
                                uint32_t* status, float* part, int reverse, int keep_rows, const DeviceInfo& dev,
                                cudaStream_t stream) {
  return launch_sk<true>(p, plan, nullptr, idx, count, nullptr, nullptr, status, nullptr, part, reverse, 1, 0, keep_rows,
                         dev, stream);
}

}  // namespace clsa
