// GQA sparse attention over the selected rows only (Eq. 4), one launch per cross-decoder layer.
//
// The kernel is bound by the gather of K/V rows from HBM (4 flops per byte per KV head), so its
// shape is chosen for memory behaviour; the small matrix products ride on warp-level bf16 MMAs
// (m16n8k16, fp32 accumulate) with the query heads of one KV head packed into the 16 rows of one
// tile, far below tensor-pipe capacity.
//
// Decomposition. All (query row, selected slot) pairs form one flat slot space of R * k slots
// (R = B * T query rows). It is cut into J equal spans. A persistent grid of one 8-warp block per
// SM runs 8 * blocks autonomous warps; warp v serves KV head v % Hkv of span v / Hkv, so the warps
// of one block walk the same tokens for different KV heads and together fetch each token's whole
// contiguous [Hkv][D] K row and V row. A warp streams its span in 16-token stages through a
// private 3-deep cp.async ring (16-byte chunks, XOR-swizzled for conflict-free ldmatrix), runs
// S = Q K^T, an online softmax in the exp2 domain, and O += P V per stage; there is no block-level
// barrier anywhere. When spans are shorter than k (decoding) a row is split over several spans:
// each writes an unnormalised partial (O, max, sum) and a small merge kernel combines them by
// log-sum-exp. When spans hold whole rows (prefill) outputs are written directly.
// `reverse` flips the order in which a warp walks its span; alternating it between consecutive
// layers makes layer l+1 start on the rows layer l touched last, which are the ones still in L2.
#include "common.cuh"

namespace clsa {
namespace {

constexpr int kThreads = kAttnWarps * 32;
constexpr int kStageBytes = kAttnStageTokens * 256 * 2;  // 16 K rows + 16 V rows of 256 bytes
constexpr int kWarpRingBytes = kAttnStages * kStageBytes;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

struct AttnArgs {
  const uint16_t* q;
  const uint16_t* kc;
  const uint16_t* vc;
  int64_t tok_stride, head_stride;
  const int64_t* seq_start;
  const int32_t* seq_len;
  const int32_t* idx;
  const int32_t* count;
  uint16_t* out;
  float* lse;
  float* partials;
  uint32_t* status;
  int64_t num_rows, span_slots;
  int q_per_seq, num_q_heads, num_kv_heads, group, top_k, num_spans, max_parts, reverse;
  float scale_log2;
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
  const int bytes = valid ? 16 : 0;  // 0 source bytes: the 16 destination bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// 2^x by the hardware approximation (2 ulp; -inf gives +0).
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ int clamp_count(int c, int top_k, uint32_t* status) {
  if (c < 0 || c > top_k) {
    flag_status(status, CLSA_DEV_BAD_COUNT);
    c = c < 0 ? 0 : top_k;
  }
  return c;
}

__global__ void __launch_bounds__(kThreads, 1) sparse_attn_kernel(const AttnArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t vwarp = (int64_t)blockIdx.x * kAttnWarps + warp;
  const int g = (int)(vwarp % a.num_kv_heads);
  const int64_t span = vwarp / a.num_kv_heads;
  if (span >= a.num_spans) return;
  const int64_t total_slots = a.num_rows * a.top_k;
  const int64_t slot_lo = span * a.span_slots;
  if (slot_lo >= total_slots) return;
  const int64_t slot_hi = min(total_slots, slot_lo + a.span_slots);

  unsigned char* ring = smem + warp * kWarpRingBytes;
  const uint32_t ring_u32 = smem_u32(ring);
  uint32_t* stage_mask = reinterpret_cast<uint32_t*>(smem + kAttnWarps * kWarpRingBytes) + warp * kAttnStages;

  const int G = a.group;
  const int qrow_a = lane >> 2;        // MMA row (query head within the group) of c0/c1; c2/c3 are row + 8
  const int qcol = (lane & 3) * 2;

  const int64_t row_first = slot_lo / a.top_k, row_last = (slot_hi - 1) / a.top_k;
  const int64_t nrows = row_last - row_first + 1;
#pragma unroll 1
  for (int64_t ri = 0; ri < nrows; ++ri) {
    const int64_t r = a.reverse ? row_last - ri : row_first + ri;
    const int64_t row_slot0 = r * a.top_k;
    const int cnt = clamp_count(a.count[r], a.top_k, lane == 0 ? a.status : nullptr);
    const int t_lo = (int)max((int64_t)0, slot_lo - row_slot0);
    const int t_hi = (int)min((int64_t)cnt, slot_hi - row_slot0);
    const bool whole = (slot_lo <= row_slot0) && (slot_hi >= row_slot0 + a.top_k);
    const int h0 = g * G;  // first query head of this KV head
    if (t_lo >= t_hi) {
      if (whole) {  // nothing selected for this row: zeros and lse = -inf
        for (int e = lane; e < G * 64; e += 32)
          reinterpret_cast<uint32_t*>(a.out + (r * a.num_q_heads + h0) * 128)[e] = 0u;
        if (a.lse != nullptr && lane < G) a.lse[r * a.num_q_heads + h0 + lane] = -INFINITY;
      }
      continue;
    }
    const int b = (int)(r / a.q_per_seq);
    const int64_t s0 = a.seq_start[b];
    const int n = a.seq_len[b];

    // Query fragments (A operand, 16 x 128): rows >= G are zero padding.
    uint32_t qa[8][4];
    {
      const uint16_t* qbase = a.q + (r * a.num_q_heads + h0) * 128;
      const bool v0 = qrow_a < G, v1 = qrow_a + 8 < G;
#pragma unroll
      for (int kk = 0; kk < 8; ++kk) {
        const int c = kk * 16 + qcol;
        qa[kk][0] = v0 ? *reinterpret_cast<const uint32_t*>(qbase + qrow_a * 128 + c) : 0u;
        qa[kk][1] = v1 ? *reinterpret_cast<const uint32_t*>(qbase + (qrow_a + 8) * 128 + c) : 0u;
        qa[kk][2] = v0 ? *reinterpret_cast<const uint32_t*>(qbase + qrow_a * 128 + c + 8) : 0u;
        qa[kk][3] = v1 ? *reinterpret_cast<const uint32_t*>(qbase + (qrow_a + 8) * 128 + c + 8) : 0u;
      }
    }

    const int nstages = (t_hi - t_lo + kAttnStageTokens - 1) / kAttnStageTokens;
    const int32_t* row_idx = a.idx + row_slot0;
    const uint16_t* kbase = a.kc + g * a.head_stride + (lane & 15) * 8;
    const uint16_t* vbase = a.vc + g * a.head_stride + (lane & 15) * 8;

    // token offset of pipeline step i
    auto stage_t0 = [&](int i) { return t_lo + (a.reverse ? nstages - 1 - i : i) * kAttnStageTokens; };
    // lanes 0..15 fetch the 16 positions of step i (-1 past the end)
    auto load_idx = [&](int i) -> int {
      if (i >= nstages || lane >= kAttnStageTokens) return -1;
      const int tt = stage_t0(i) + lane;
      return tt < t_hi ? row_idx[tt] : -1;
    };
    auto issue = [&](int i, int my_idx) {
      if (i < nstages) {
        const int buf = i % kAttnStages;
        const uint32_t kdst = ring_u32 + buf * kStageBytes, vdst = kdst + kStageBytes / 2;
        const bool in_range = my_idx >= 0 && my_idx < n;
        const uint32_t okmask = __ballot_sync(0xffffffffu, in_range) & 0xffffu;
        const bool bad = lane < kAttnStageTokens && !in_range && (stage_t0(i) + lane) < t_hi;
        if (bad) flag_status(a.status, CLSA_DEV_BAD_INDEX);
        if (lane == 0) stage_mask[buf] = okmask;
#pragma unroll
        for (int it = 0; it < 8; ++it) {
          const int j = it * 2 + (lane >> 4);  // token of the stage this lane helps fetch
          const int tok = __shfl_sync(0xffffffffu, my_idx, j);
          const bool ok = (okmask >> j) & 1u;
          const int64_t off = (s0 + (ok ? tok : 0)) * a.tok_stride;
          const uint32_t sw = (uint32_t)(j * 256 + (((lane & 15) ^ (j & 7)) << 4));
          cp_async16(kdst + sw, kbase + off, ok);
          cp_async16(vdst + sw, vbase + off, ok);
        }
      }
      cp_async_commit();
    };

    float o[16][4];
#pragma unroll
    for (int j = 0; j < 16; ++j) { o[j][0] = 0.f; o[j][1] = 0.f; o[j][2] = 0.f; o[j][3] = 0.f; }
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

    // prologue: stages 0 .. kAttnStages-2 in flight, positions of the next one in a register
    int next_idx = load_idx(0);
#pragma unroll
    for (int i = 0; i < kAttnStages - 1; ++i) {
      const int cur = next_idx;
      next_idx = load_idx(i + 1);
      issue(i, cur);
    }
#pragma unroll 1
    for (int i = 0; i < nstages; ++i) {
      {  // refill the buffer freed by step i-1
        const int cur = next_idx;
        next_idx = load_idx(i + kAttnStages);
        issue(i + kAttnStages - 1, cur);
      }
      cp_async_wait<kAttnStages - 1>();
      __syncwarp();
      const int buf = i % kAttnStages;
      const uint32_t kbuf = ring_u32 + buf * kStageBytes, vbuf = kbuf + kStageBytes / 2;
      const uint32_t okmask = stage_mask[buf];

      // S = Q K^T for 16 tokens (two 8-token tiles)
      float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
      for (int kq = 0; kq < 4; ++kq) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int tok = 8 * j + (lane & 7), chunk = 4 * kq + (lane >> 3);
          uint32_t bfrag[4];
          ldmatrix_x4(bfrag, kbuf + tok * 256 + ((chunk ^ (tok & 7)) << 4));
          mma_bf16(s[j], qa[2 * kq], bfrag[0], bfrag[1]);
          mma_bf16(s[j], qa[2 * kq + 1], bfrag[2], bfrag[3]);
        }
      }
      // online softmax, exp2 domain; masked tokens get -inf
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int j = 0; j < 2; ++j) {
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const bool ok = (okmask >> (8 * j + qcol + e)) & 1u;
          s[j][e] = ok ? s[j][e] * a.scale_log2 : -INFINITY;
          s[j][2 + e] = ok ? s[j][2 + e] * a.scale_log2 : -INFINITY;
          mx0 = fmaxf(mx0, s[j][e]);
          mx1 = fmaxf(mx1, s[j][2 + e]);
        }
      }
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
      const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
      const float mu0 = mn0 == -INFINITY ? 0.f : mn0, mu1 = mn1 == -INFINITY ? 0.f : mn1;
      const float alpha0 = fast_exp2(m0 - mu0), alpha1 = fast_exp2(m1 - mu1);
      m0 = mn0;
      m1 = mn1;
      uint32_t pa[4];
      {
        const uint32_t p00 = pack_bf16x2(fast_exp2(s[0][0] - mu0), fast_exp2(s[0][1] - mu0));
        const uint32_t p01 = pack_bf16x2(fast_exp2(s[0][2] - mu1), fast_exp2(s[0][3] - mu1));
        const uint32_t p10 = pack_bf16x2(fast_exp2(s[1][0] - mu0), fast_exp2(s[1][1] - mu0));
        const uint32_t p11 = pack_bf16x2(fast_exp2(s[1][2] - mu1), fast_exp2(s[1][3] - mu1));
        pa[0] = p00; pa[1] = p01; pa[2] = p10; pa[3] = p11;
        // the denominators use the same bf16-rounded weights as the numerators
        l0 = l0 * alpha0 + (bf16_lo(p00) + bf16_hi(p00)) + (bf16_lo(p10) + bf16_hi(p10));
        l1 = l1 * alpha1 + (bf16_lo(p01) + bf16_hi(p01)) + (bf16_lo(p11) + bf16_hi(p11));
      }
#pragma unroll
      for (int j = 0; j < 16; ++j) { o[j][0] *= alpha0; o[j][1] *= alpha0; o[j][2] *= alpha1; o[j][3] *= alpha1; }
      // O += P V
#pragma unroll
      for (int jp = 0; jp < 8; ++jp) {
        const int tok = (lane & 7) + 8 * ((lane >> 3) & 1), chunk = 2 * jp + (lane >> 4);
        uint32_t vfrag[4];
        ldmatrix_x4_trans(vfrag, vbuf + tok * 256 + ((chunk ^ (tok & 7)) << 4));
        mma_bf16(o[2 * jp], pa, vfrag[0], vfrag[1]);
        mma_bf16(o[2 * jp + 1], pa, vfrag[2], vfrag[3]);
      }
      __syncwarp();  // everyone is done with this buffer before the next step refills it
    }
    cp_async_wait<0>();

    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);

    if (whole) {
      const float inv0 = l0 > 0.f ? 1.f / l0 : 0.f, inv1 = l1 > 0.f ? 1.f / l1 : 0.f;
      uint16_t* obase = a.out + (r * a.num_q_heads + h0) * 128;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        if (qrow_a < G)
          *reinterpret_cast<uint32_t*>(obase + qrow_a * 128 + j * 8 + qcol) = pack_bf16x2(o[j][0] * inv0, o[j][1] * inv0);
        if (qrow_a + 8 < G)
          *reinterpret_cast<uint32_t*>(obase + (qrow_a + 8) * 128 + j * 8 + qcol) = pack_bf16x2(o[j][2] * inv1, o[j][3] * inv1);
      }
      if (a.lse != nullptr && (lane & 3) == 0) {
        if (qrow_a < G) a.lse[r * a.num_q_heads + h0 + qrow_a] = l0 > 0.f ? (m0 + log2f(l0)) * kLn2 : -INFINITY;
        if (qrow_a + 8 < G) a.lse[r * a.num_q_heads + h0 + qrow_a + 8] = l1 > 0.f ? (m1 + log2f(l1)) * kLn2 : -INFINITY;
      }
    } else {
      const int part = (int)(span - row_slot0 / a.span_slots);
      float* pbase = a.partials + ((r * a.max_parts + part) * a.num_q_heads + h0) * kPartialFloats;
#pragma unroll
      for (int j = 0; j < 16; ++j) {
        if (qrow_a < G)
          *reinterpret_cast<float2*>(pbase + qrow_a * kPartialFloats + j * 8 + qcol) = make_float2(o[j][0], o[j][1]);
        if (qrow_a + 8 < G)
          *reinterpret_cast<float2*>(pbase + (qrow_a + 8) * kPartialFloats + j * 8 + qcol) = make_float2(o[j][2], o[j][3]);
      }
      if ((lane & 3) == 0) {
        if (qrow_a < G) *reinterpret_cast<float2*>(pbase + qrow_a * kPartialFloats + 128) = make_float2(m0, l0);
        if (qrow_a + 8 < G) *reinterpret_cast<float2*>(pbase + (qrow_a + 8) * kPartialFloats + 128) = make_float2(m1, l1);
      }
    }
  }
}

// Log-sum-exp merge of the partials of one (query row, head): one warp each, 4 output values per lane.
__global__ void __launch_bounds__(256) attn_merge_kernel(const float* __restrict__ partials, const int32_t* __restrict__ count,
                                                         uint16_t* __restrict__ out, float* __restrict__ lse,
                                                         int64_t num_rows, int num_q_heads, int top_k, int64_t span_slots,
                                                         int max_parts) {
  const int lane = threadIdx.x & 31;
  const int64_t item = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (item >= num_rows * num_q_heads) return;
  const int64_t r = item / num_q_heads;
  const int h = (int)(item % num_q_heads);
  int cnt = count[r];
  cnt = cnt < 0 ? 0 : (cnt > top_k ? top_k : cnt);
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  float L = 0.f, M = -INFINITY;
  if (cnt > 0) {
    const int64_t slot0 = r * top_k;
    const int nparts = (int)((slot0 + cnt - 1) / span_slots - slot0 / span_slots) + 1;
    const float* base = partials + ((r * max_parts) * num_q_heads + h) * kPartialFloats;
    const int64_t pstride = (int64_t)num_q_heads * kPartialFloats;
    for (int p = 0; p < nparts; ++p) M = fmaxf(M, base[p * pstride + 128]);
    const float mu = M == -INFINITY ? 0.f : M;
    for (int p = 0; p < nparts; ++p) {
      const float* pp = base + p * pstride;
      const float w = fast_exp2(pp[128] - mu);
      const float4 ov = *reinterpret_cast<const float4*>(pp + lane * 4);
      acc[0] += w * ov.x; acc[1] += w * ov.y; acc[2] += w * ov.z; acc[3] += w * ov.w;
      L += w * pp[129];
    }
  }
  const float inv = L > 0.f ? 1.f / L : 0.f;
  uint2 packed;
  packed.x = pack_bf16x2(acc[0] * inv, acc[1] * inv);
  packed.y = pack_bf16x2(acc[2] * inv, acc[3] * inv);
  *reinterpret_cast<uint2*>(out + item * 128 + lane * 4) = packed;
  if (lse != nullptr && lane == 0) lse[item] = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
}

}  // namespace

AttnPlan make_attn_plan(const clsa_params& p, const DeviceInfo& dev) {
  AttnPlan plan;
  const int hkv = p.num_kv_heads;
  int gcd = hkv, x = kAttnWarps;
  while (x) { const int tmp = gcd % x; gcd = x; x = tmp; }
  const int step = hkv / gcd;  // blocks must come in multiples of this so that 8 * blocks % Hkv == 0
  int blocks = dev.sm_count / step * step;
  if (blocks < step) blocks = step;
  plan.num_blocks = blocks;
  plan.num_spans = (int)((int64_t)blocks * kAttnWarps / hkv);
  const int64_t rows = (int64_t)p.num_seqs * p.q_per_seq;
  const int64_t total = rows * p.top_k;
  int64_t sp = (total + plan.num_spans - 1) / plan.num_spans;
  sp = (sp + kAttnStageTokens - 1) / kAttnStageTokens * kAttnStageTokens;
  if (sp >= p.top_k) {
    sp = (sp + p.top_k - 1) / p.top_k * p.top_k;  // whole rows per span: outputs are written directly
    plan.max_parts = 1;
    plan.partial_bytes = 0;
  } else {
    plan.max_parts = (int)((p.top_k + sp - 1) / sp) + 1;
    plan.partial_bytes = (size_t)rows * plan.max_parts * p.num_q_heads * kPartialFloats * sizeof(float);
  }
  plan.span_slots = sp;
  return plan;
}

cudaError_t launch_sparse_attn(const clsa_params& p, const void* q, const int32_t* idx, const int32_t* count, void* out,
                               float* lse, float* partials, uint32_t* status, int reverse, const DeviceInfo& dev,
                               cudaStream_t stream) {
  const AttnPlan plan = make_attn_plan(p, dev);
  AttnArgs a;
  a.q = static_cast<const uint16_t*>(q);
  a.kc = static_cast<const uint16_t*>(p.k_cache);
  a.vc = static_cast<const uint16_t*>(p.v_cache);
  a.tok_stride = p.kv_token_stride;
  a.head_stride = p.kv_head_stride;
  a.seq_start = p.seq_start;
  a.seq_len = p.seq_len;
  a.idx = idx;
  a.count = count;
  a.out = static_cast<uint16_t*>(out);
  a.lse = lse;
  a.partials = partials;
  a.status = status;
  a.num_rows = (int64_t)p.num_seqs * p.q_per_seq;
  a.span_slots = plan.span_slots;
  a.q_per_seq = p.q_per_seq;
  a.num_q_heads = p.num_q_heads;
  a.num_kv_heads = p.num_kv_heads;
  a.group = p.num_q_heads / p.num_kv_heads;
  a.top_k = p.top_k;
  a.num_spans = plan.num_spans;
  a.max_parts = plan.max_parts;
  a.reverse = reverse;
  a.scale_log2 = p.sm_scale * kLog2e;
  const size_t smem = (size_t)kAttnWarps * kWarpRingBytes + kAttnWarps * kAttnStages * sizeof(uint32_t);
  cudaError_t err = cudaFuncSetAttribute(sparse_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (err != cudaSuccess) return err;
  sparse_attn_kernel<<<plan.num_blocks, kThreads, smem, stream>>>(a);
  err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  if (plan.max_parts > 1) {
    const int64_t items = a.num_rows * p.num_q_heads;
    const int64_t blocks = (items + 7) / 8;
    attn_merge_kernel<<<(unsigned)blocks, 256, 0, stream>>>(partials, count, a.out, lse, a.num_rows, p.num_q_heads,
                                                            p.top_k, plan.span_slots, plan.max_parts);
    err = cudaGetLastError();
  }
  return err;
}

}  // namespace clsa
