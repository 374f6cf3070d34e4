// GQA sparse attention over the selected rows only (Eq. 4), one launch per cross-decoder layer.
//
// The kernel is bound by the gather of K/V rows from HBM (4 flops per byte per KV head), so its
// shape is chosen for memory behaviour; the small matrix products ride on warp-level bf16 MMAs
// (m16n8k16, fp32 accumulate) with the query heads of one KV head packed into the 16 rows of one
// tile, far below tensor-pipe capacity.
//
// Decomposition. One thread-block cluster of C blocks serves one query row (sequence, query
// token); its selected tokens are cut into C * S contiguous ranges. A block has 8 autonomous
// warps: warp w serves KV head w % HC of token range w / HC (HC heads per block, S = 8 / HC
// ranges per block). A warp streams
// its range in 16-token stages through a private 3-deep cp.async ring (16-byte chunks,
// XOR-swizzled for conflict-free ldmatrix), runs S = Q K^T, an online softmax in the exp2 domain
// and O += P V per stage; there is no block-level barrier in the main loop. Split-K merge: every
// warp leaves its unnormalised partial (O, running max, running sum) in its own shared memory,
// the cluster synchronises once, and the (KV head, query head) outputs are dealt round-robin to
// the warps of the cluster, each reading the C * S partials it needs through distributed shared
// memory and combining them by log-sum-exp. Nothing goes through global memory, nothing spins.
// The launch shape is chosen per call so that all blocks are resident at once where possible:
// HC shrinks (down to one KV head per block, its 8 warps splitting the tokens) until
// rows * Hkv / HC fits the SM count, then C grows while the clusters still fit. Decoding a batch of
// 16 with 8 KV heads runs 128 single-block clusters whose merge never leaves the block; a prefill
// chunk runs one block per query row with nothing to merge.
// `reverse` flips the order in which a warp walks its range; alternating it between consecutive
// layers makes layer l+1 start on the rows layer l touched last, which are the ones still in L2.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace clsa {
namespace {

constexpr int kThreads = kAttnWarps * 32;
constexpr int kStageBytes = kAttnStageTokens * 256 * 2;  // 16 K rows + 16 V rows of 256 bytes
constexpr int kWarpRingBytes = kAttnStages * kStageBytes;
constexpr int kPartialStride = 132;                      // floats per head of a partial: 128 outputs, max, sum, pad
constexpr int kMergeBatch = 8;
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
  uint32_t* status;
  int q_per_seq, num_q_heads, num_kv_heads, group, top_k;
  int heads_per_block, subs, reverse;
  int wait_prior;  // 1: inputs may come from the kernel launched just before this one (wait for it first)
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

__global__ void __launch_bounds__(kThreads, 1) sparse_attn_kernel(const AttnArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  cg::cluster_group cluster = cg::this_cluster();
  const int C = (int)cluster.num_blocks();
  const int crank = (int)cluster.block_rank();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t r = blockIdx.x / C;                 // query row
  const int HC = a.heads_per_block, S = a.subs, G = a.group;
  const int g_local = warp % HC, sub = warp / HC;
  const int g = blockIdx.y * HC + g_local;          // KV head of this warp
  const bool active = sub < S && g < a.num_kv_heads;
  const int nsplit = C * S;                         // token ranges of the row

  unsigned char* ring = smem + warp * kWarpRingBytes;
  const uint32_t ring_u32 = smem_u32(ring);
  uint32_t* stage_mask = reinterpret_cast<uint32_t*>(smem + kAttnWarps * kWarpRingBytes) + warp * kAttnStages;

  const int qrow_a = lane >> 2;        // MMA row (query head within the group) of c0/c1; c2/c3 are row + 8
  const int qcol = (lane & 3) * 2;
  const int h0 = g * G;                // first query head of this KV head

  // Programmatic dependent launch: let the next kernel of the stream start its own prologue as soon
  // as SMs free up, and (unless the caller vouches that every input predates the previous kernel)
  // wait for the previous kernel's results before the first global read.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (a.wait_prior) asm volatile("griddepcontrol.wait;" ::: "memory");

  // The row's k slots are cut into nsplit ranges of `per` slots (a multiple of the stage size); the
  // split does not depend on the row's count, so the first positions can be fetched together with it.
  const int per = (((a.top_k + nsplit - 1) / nsplit) + kAttnStageTokens - 1) / kAttnStageTokens * kAttnStageTokens;
  const int range = crank * S + sub;
  const int slot_lo = min(a.top_k, range * per), slot_hi = min(a.top_k, slot_lo + per);
  const int32_t* row_idx = a.idx + r * a.top_k;
  int cnt = a.count[r];
  const int b = (int)(r / a.q_per_seq);
  const int64_t s0 = a.seq_start[b];
  const int n = a.seq_len[b];
  // speculative fetch of the first/last 16 positions of the range (entries past the count are unused)
  int first_idx = -1;
  if (active && lane < kAttnStageTokens) {
    const int nst = (slot_hi - slot_lo + kAttnStageTokens - 1) / kAttnStageTokens;
    const int tt = slot_lo + (a.reverse ? (nst - 1) * kAttnStageTokens : 0) + lane;
    if (tt < slot_hi) first_idx = row_idx[tt];
  }
  if (cnt < 0 || cnt > a.top_k) {
    if (threadIdx.x == 0 && crank == 0 && blockIdx.y == 0) flag_status(a.status, CLSA_DEV_BAD_COUNT);
    cnt = cnt < 0 ? 0 : a.top_k;
  }
  const int t_lo = min(cnt, slot_lo), t_hi = active ? min(cnt, slot_hi) : t_lo;

  float o[16][4];
#pragma unroll
  for (int j = 0; j < 16; ++j) { o[j][0] = 0.f; o[j][1] = 0.f; o[j][2] = 0.f; o[j][3] = 0.f; }
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

  if (t_lo < t_hi) {
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

    // prologue: stages 0 .. kAttnStages-2 in flight, positions of the next one in a register
    int next_idx;
    if (t_hi == slot_hi) {  // the range is entirely below the count: the speculative fetch was step 0
      next_idx = first_idx;
    } else {
      next_idx = load_idx(0);
    }
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
      const bool rescale = (mn0 != m0) || (mn1 != m1);
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
      if (__any_sync(0xffffffffu, rescale)) {  // the running max moved for some head: rescale the accumulators
#pragma unroll
        for (int j = 0; j < 16; ++j) { o[j][0] *= alpha0; o[j][1] *= alpha0; o[j][2] *= alpha1; o[j][3] *= alpha1; }
      }
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
  }

  if (nsplit == 1) {
    // the warp saw the whole row: normalise and write straight from the accumulators
    if (active) {
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
    }
    return;  // uniform over the cluster (a cluster of one block)
  }

  // ---- split-K merge through distributed shared memory ---------------------------------------------
  // Each warp parks its partial in its own (now idle) staging ring: [G][kPartialStride] floats.
  float* mypart = reinterpret_cast<float*>(ring);
  if (active) {
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      if (qrow_a < G)
        *reinterpret_cast<float2*>(mypart + qrow_a * kPartialStride + j * 8 + qcol) = make_float2(o[j][0], o[j][1]);
      if (qrow_a + 8 < G)
        *reinterpret_cast<float2*>(mypart + (qrow_a + 8) * kPartialStride + j * 8 + qcol) = make_float2(o[j][2], o[j][3]);
    }
    if ((lane & 3) == 0) {
      if (qrow_a < G) *reinterpret_cast<float2*>(mypart + qrow_a * kPartialStride + 128) = make_float2(m0, l0);
      if (qrow_a + 8 < G) *reinterpret_cast<float2*>(mypart + (qrow_a + 8) * kPartialStride + 128) = make_float2(m1, l1);
    }
  }
  cluster.sync();

  // Output jobs (KV head of this block's group, query head of the group) dealt over the cluster's warps.
  const int heads_here = min(HC, a.num_kv_heads - (int)blockIdx.y * HC);
  const int njobs = heads_here * G;
  for (int job = crank + C * warp; job < njobs; job += C * kAttnWarps) {
    const int jg = job / G, hh = job - jg * G;   // local KV head, query head within the group
    // partial p = (block p / S, range p % S) was left by warp (p % S) * HC + jg of block p / S
    auto part_ptr = [&](int p) -> const float* {
      const int c2 = p / S, sub2 = p - c2 * S;
      return cluster.map_shared_rank(reinterpret_cast<float*>(smem + (sub2 * HC + jg) * kWarpRingBytes), c2) +
             hh * kPartialStride;
    };
    float M = -INFINITY;
    for (int p = lane; p < nsplit; p += 32) M = fmaxf(M, part_ptr(p)[128]);
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, d));
    const float mu = M == -INFINITY ? 0.f : M;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float L = 0.f;
    for (int p0 = 0; p0 < nsplit; p0 += 32) {
      float wl = 0.f;
      if (p0 + lane < nsplit) {
        const float2 ml = *reinterpret_cast<const float2*>(part_ptr(p0 + lane) + 128);
        wl = fast_exp2(ml.x - mu);
        L += wl * ml.y;
      }
      const int chunk_n = min(32, nsplit - p0);
      for (int q0 = 0; q0 < chunk_n; q0 += kMergeBatch) {
        float4 v[kMergeBatch];
#pragma unroll
        for (int qq = 0; qq < kMergeBatch; ++qq)
          v[qq] = q0 + qq < chunk_n ? *reinterpret_cast<const float4*>(part_ptr(p0 + q0 + qq) + lane * 4)
                                    : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int qq = 0; qq < kMergeBatch; ++qq) {
          const float w = __shfl_sync(0xffffffffu, wl, (q0 + qq) & 31);
          const float wq = q0 + qq < chunk_n ? w : 0.f;
          acc.x = fmaf(wq, v[qq].x, acc.x); acc.y = fmaf(wq, v[qq].y, acc.y);
          acc.z = fmaf(wq, v[qq].z, acc.z); acc.w = fmaf(wq, v[qq].w, acc.w);
        }
      }
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) L += __shfl_xor_sync(0xffffffffu, L, d);
    const float inv = L > 0.f ? 1.f / L : 0.f;
    const int64_t item = r * a.num_q_heads + (int64_t)(blockIdx.y * HC + jg) * G + hh;
    uint2 packed;
    packed.x = pack_bf16x2(acc.x * inv, acc.y * inv);
    packed.y = pack_bf16x2(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2*>(a.out + item * 128 + lane * 4) = packed;
    if (a.lse != nullptr && lane == 0) a.lse[item] = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
  }
  cluster.sync();  // no block may exit while a neighbour can still read its shared memory
}

// Blocks of `cluster` that can be resident at once (cached per cluster size; 0 if the query fails).
static int max_resident_blocks(int cluster, size_t smem_bytes) {
  static int cache[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0};
  if (cache[cluster] != 0) return cache[cluster];
  cudaFuncSetAttribute(sparse_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes);
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
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, sparse_attn_kernel, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
  cache[cluster] = n * cluster;
  return cache[cluster];
}

}  // namespace

AttnPlan make_attn_plan(const clsa_params& p, const DeviceInfo& dev) {
  AttnPlan plan;
  plan.smem_bytes = (size_t)kAttnWarps * kWarpRingBytes + kAttnWarps * kAttnStages * sizeof(uint32_t);
  const int hkv = p.num_kv_heads;
  const int64_t rows = (int64_t)p.num_seqs * p.q_per_seq;
  // Heads per block: as few as it takes for all blocks to be resident at once (more blocks, and the
  // split over tokens then stays inside a block); all 8 warps on different heads once there are
  // more rows than SMs.
  int hc_max = 1;
  while (hc_max * 2 <= kAttnWarps && hc_max * 2 <= hkv) hc_max *= 2;
  int hc = 1;
  while (hc < hc_max && rows * ((hkv + hc - 1) / hc) > dev.sm_count) hc *= 2;
  // every token range should hold at least one 16-token stage
  while (hc < hc_max && (int64_t)(kAttnWarps / hc) * kAttnStageTokens > p.top_k) hc *= 2;
  plan.heads_per_block = hc;
  plan.subs = kAttnWarps / hc;
  plan.head_groups = (hkv + hc - 1) / hc;
  // Cluster: the largest power of two that still keeps every block resident at once.
  int c = 1;
  const int64_t blocks = rows * plan.head_groups;
  while (c < 8 && blocks * (c * 2) <= max_resident_blocks(c * 2, plan.smem_bytes) &&
         (int64_t)(c * 2) * plan.subs * kAttnStageTokens <= p.top_k)
    c *= 2;
  plan.cluster = c;
  (void)dev;
  return plan;
}

cudaError_t launch_sparse_attn(const clsa_params& p, const void* q, const int32_t* idx, const int32_t* count, void* out,
                               float* lse, uint32_t* status, int reverse, int wait_prior, const DeviceInfo& dev,
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
  a.status = status;
  a.q_per_seq = p.q_per_seq;
  a.num_q_heads = p.num_q_heads;
  a.num_kv_heads = p.num_kv_heads;
  a.group = p.num_q_heads / p.num_kv_heads;
  a.top_k = p.top_k;
  a.heads_per_block = plan.heads_per_block;
  a.subs = plan.subs;
  a.reverse = reverse;
  a.wait_prior = wait_prior;
  a.scale_log2 = p.sm_scale * kLog2e;
  cudaError_t err = cudaFuncSetAttribute(sparse_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)plan.smem_bytes);
  if (err != cudaSuccess) return err;
  const int64_t rows = (int64_t)p.num_seqs * p.q_per_seq;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(rows * plan.cluster), (unsigned)plan.head_groups, 1);
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
  return cudaLaunchKernelEx(&cfg, sparse_attn_kernel, a);
}

}  // namespace clsa
