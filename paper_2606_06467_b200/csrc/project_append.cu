// Eq. 2 for the newest tokens of every sequence and the cache append that precedes Eq. 3:
//   q_idx = h W^Q_idx,  K_idx row = h W^K_idx,  K row = h W^K,  V row = h W^V     (bf16 in, fp32 sums, bf16 out)
//
// At decode the state matrix has B*T <= a few dozen rows, so the op is a stream of the weight matrices
// (11.8 MB for d_model 2560, d_idx 128, 8 KV heads of 128) against a handful of rows: bound by HBM
// latency and bandwidth, not by arithmetic. The four weight matrices are treated as one list of output
// features; a block owns 16 of them (two n8 tiles) and splits the d_model contraction over its warps.
// Each lane fetches 16 bytes (8 consecutive features of d_model) of its weight row and of its two state
// rows per step, and feeds them to two warp-level m16n8k16 MMAs. The k index inside an MMA is a dummy
// summation index, so the lanes' 8-element runs are used as they come (no shuffle, no shared-memory
// staging): A and B apply the same permutation of k. Partial sums of the warps meet in shared memory
// in a fixed order, so results do not depend on scheduling.
#include "common.cuh"

namespace clsa {
namespace {

constexpr int kColsPerBlock = 16;  // two n8 tiles

struct ProjArgs {
  const uint16_t* h;       // [rows][d_model]
  const uint16_t* w[4];    // q_idx, k_idx, k, v: [n_out][d_model]
  int seg_end[4];          // running ends of the four feature ranges in the combined list
  uint16_t* q_idx_out;     // [rows][d_idx]
  uint16_t* idx_k_cache;
  uint16_t* k_cache;
  uint16_t* v_cache;
  int64_t idx_token_stride, kv_token_stride, kv_head_stride;
  const int64_t* seq_start;
  const int32_t* seq_len;
  const int32_t* block_table;
  int block_shift, block_mask, max_blocks_per_seq;
  int rows, q_per_seq, d_model, d_idx, head_dim, max_seq_len;
  uint32_t* status;
};

__device__ __forceinline__ uint4 ld_stream16(const void* p) {
  uint4 v;
  asm volatile("ld.global.cs.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ uint4 ld_cached16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// MT = m16 tiles of state rows a block keeps accumulators for (the weights are fetched once for all of them).
// With one row tile, 16 warps take 5 k-steps each at d_model 2560 and issue all their loads (20 x 16 B per
// thread) before the first MMA: the whole 80 KB weight slab of the block is in flight at once, one memory
// round trip. More row tiles need more registers per step, so fewer steps are fetched together.
template <int MT, int kWarps>
__global__ void __launch_bounds__(kWarps * 32) project_append_kernel(const ProjArgs a) {
  constexpr int kThreads = kWarps * 32;
  constexpr int kUnroll = MT == 1 ? 5 : (MT == 2 ? 3 : 2);
  __shared__ float part[kWarps][MT][2][128];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, j = lane & 3;
  const int col0 = blockIdx.x * kColsPerBlock;  // first feature of this block in the combined list
  const int row0 = blockIdx.y * (MT * 16);

  // the block's 16 features lie in one of the four matrices (every range is a multiple of 16 long)
  int seg = 0;
  while (seg < 3 && col0 >= a.seg_end[seg]) ++seg;
  const int seg_begin = seg == 0 ? 0 : a.seg_end[seg - 1];
  const int local0 = col0 - seg_begin;
  const uint16_t* wrow[2];
  wrow[0] = a.w[seg] + (int64_t)(local0 + g) * a.d_model + j * 8;
  wrow[1] = wrow[0] + (int64_t)8 * a.d_model;
  const uint16_t* hrow[MT][2];
#pragma unroll
  for (int m = 0; m < MT; ++m) {
    const int r0 = min(row0 + m * 16 + g, a.rows - 1), r1 = min(row0 + m * 16 + g + 8, a.rows - 1);
    hrow[m][0] = a.h + (int64_t)r0 * a.d_model + j * 8;
    hrow[m][1] = a.h + (int64_t)r1 * a.d_model + j * 8;
  }

  float acc[MT][2][4];
#pragma unroll
  for (int m = 0; m < MT; ++m)
#pragma unroll
    for (int n = 0; n < 2; ++n)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[m][n][i] = 0.f;

  const int steps = a.d_model / 32;
  for (int s0 = warp; s0 < steps; s0 += kWarps * kUnroll) {
    uint4 wv[kUnroll][2], hv[kUnroll][MT][2];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const int s = s0 + u * kWarps;
      if (s < steps) {
#pragma unroll
        for (int n = 0; n < 2; ++n) wv[u][n] = ld_stream16(wrow[n] + s * 32);
#pragma unroll
        for (int m = 0; m < MT; ++m) {
          hv[u][m][0] = ld_cached16(hrow[m][0] + s * 32);
          hv[u][m][1] = ld_cached16(hrow[m][1] + s * 32);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      if (s0 + u * kWarps < steps) {
#pragma unroll
        for (int m = 0; m < MT; ++m)
#pragma unroll
          for (int n = 0; n < 2; ++n) {
            mma_bf16(acc[m][n], hv[u][m][0].x, hv[u][m][1].x, hv[u][m][0].y, hv[u][m][1].y, wv[u][n].x, wv[u][n].y);
            mma_bf16(acc[m][n], hv[u][m][0].z, hv[u][m][1].z, hv[u][m][0].w, hv[u][m][1].w, wv[u][n].z, wv[u][n].w);
          }
      }
    }
  }

  // accumulator (row g / g+8, features 2j, 2j+1 of tile n) -> part[warp][m][n][row * 8 + feature]
#pragma unroll
  for (int m = 0; m < MT; ++m)
#pragma unroll
    for (int n = 0; n < 2; ++n) {
      *reinterpret_cast<float2*>(&part[warp][m][n][g * 8 + 2 * j]) = make_float2(acc[m][n][0], acc[m][n][1]);
      *reinterpret_cast<float2*>(&part[warp][m][n][(g + 8) * 8 + 2 * j]) = make_float2(acc[m][n][2], acc[m][n][3]);
    }
  __syncthreads();

  // one thread per (row, feature pair): sum the warps' partials in warp order, round once, store
  for (int e = threadIdx.x; e < MT * 16 * 8; e += kThreads) {
    const int m = e / 128, r = (e % 128) / 8, pair = e % 8;  // features 2*pair, 2*pair + 1 of the block's 16
    const int n = pair / 4, f = (pair % 4) * 2;
    const int row = row0 + m * 16 + r;
    if (row >= a.rows) continue;
    float s0 = 0.f, s1 = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      const float2 v = *reinterpret_cast<const float2*>(&part[w][m][n][r * 8 + f]);
      s0 += v.x;
      s1 += v.y;
    }
    const uint32_t packed = pack_bf16x2(s0, s1);
    const int feat = local0 + n * 8 + f;  // feature inside its own matrix
    uint16_t* dst;
    if (seg == 0) {
      dst = a.q_idx_out + (int64_t)row * a.d_idx + feat;
    } else {
      const int b = row / a.q_per_seq, t = row % a.q_per_seq;
      const int len = a.seq_len[b];
      if (len < a.q_per_seq || len > a.max_seq_len) {
        flag_status(a.status, CLSA_DEV_BAD_SEQLEN);
        continue;
      }
      const int pos = len - a.q_per_seq + t;
      int64_t crow;
      if (a.block_table != nullptr)
        crow = ((int64_t)a.block_table[(int64_t)b * a.max_blocks_per_seq + (pos >> a.block_shift)] << a.block_shift) +
               (pos & a.block_mask);
      else
        crow = a.seq_start[b] + pos;
      if (seg == 1) {
        dst = a.idx_k_cache + crow * a.idx_token_stride + feat;
      } else {
        uint16_t* base = seg == 2 ? a.k_cache : a.v_cache;
        dst = base + crow * a.kv_token_stride + (int64_t)(feat / a.head_dim) * a.kv_head_stride + feat % a.head_dim;
      }
    }
    *reinterpret_cast<uint32_t*>(dst) = packed;
  }
}

}  // namespace

cudaError_t launch_project_append(const clsa_params& p, int d_model, const void* h, const void* w_q_idx,
                                  const void* w_k_idx, const void* w_k, const void* w_v, void* q_idx_out,
                                  void* idx_k_out, void* k_out, void* v_out,
                                  uint32_t* status, const DeviceInfo& dev, cudaStream_t stream) {
  (void)dev;
  ProjArgs a;
  a.h = static_cast<const uint16_t*>(h);
  a.w[0] = static_cast<const uint16_t*>(w_q_idx);
  a.w[1] = static_cast<const uint16_t*>(w_k_idx);
  a.w[2] = static_cast<const uint16_t*>(w_k);
  a.w[3] = static_cast<const uint16_t*>(w_v);
  const int kv = w_k != nullptr ? p.num_kv_heads * p.head_dim : 0;
  a.seg_end[0] = p.idx_dim;
  a.seg_end[1] = 2 * p.idx_dim;
  a.seg_end[2] = 2 * p.idx_dim + kv;
  a.seg_end[3] = 2 * p.idx_dim + 2 * kv;
  a.q_idx_out = static_cast<uint16_t*>(q_idx_out);
  a.idx_k_cache = static_cast<uint16_t*>(idx_k_out);
  a.k_cache = static_cast<uint16_t*>(k_out);
  a.v_cache = static_cast<uint16_t*>(v_out);
  a.idx_token_stride = p.idx_token_stride;
  a.kv_token_stride = p.kv_token_stride;
  a.kv_head_stride = p.kv_head_stride;
  a.seq_start = p.seq_start;
  a.seq_len = p.seq_len;
  a.block_table = p.block_table;
  a.block_shift = 0;
  if (p.block_table != nullptr)
    while ((1 << a.block_shift) < p.block_size) ++a.block_shift;
  a.block_mask = p.block_table != nullptr ? p.block_size - 1 : 0;
  a.max_blocks_per_seq = p.max_blocks_per_seq;
  a.rows = p.num_seqs * p.q_per_seq;
  a.q_per_seq = p.q_per_seq;
  a.d_model = d_model;
  a.d_idx = p.idx_dim;
  a.head_dim = p.head_dim;
  a.max_seq_len = p.max_seq_len;
  a.status = status;
  const int col_blocks = a.seg_end[3] / kColsPerBlock;
  const int mt = a.rows <= 16 ? 1 : (a.rows <= 32 ? 2 : 4);
  dim3 grid(col_blocks, (a.rows + mt * 16 - 1) / (mt * 16));
  if (mt == 1) project_append_kernel<1, 16><<<grid, 16 * 32, 0, stream>>>(a);
  else if (mt == 2) project_append_kernel<2, 16><<<grid, 16 * 32, 0, stream>>>(a);
  else project_append_kernel<4, 8><<<grid, 8 * 32, 0, stream>>>(a);
  return cudaGetLastError();
}

}  // namespace clsa
