// Shared declarations of the CLSA CUDA library: workspace layout, launch plans, small device helpers.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "clsa.h"

namespace clsa {

// ---------------------------------------------------------------------------------------------
// Host-side plans
// ---------------------------------------------------------------------------------------------
struct DeviceInfo {
  int sm_count;
  int max_smem_optin;  // bytes of dynamic shared memory a block may opt in to
  int l2_bytes;
  int clock_khz;       // peak SM clock
};
// Cached per device (queried once). Returns false if the CUDA runtime reports an error.
bool device_info(DeviceInfo* out);

constexpr size_t kStatusBytes = 256;   // status word, scheduling counters and padding at the start of the workspace
constexpr int kSchedWord = 16;         // 32-bit word of that header where the score kernel's two ticket counters sit (zero between launches)
constexpr int kAttnWarpsNarrow = 12;    // warps per attention block (groups of up to 8 query heads per KV head), each an autonomous worker
constexpr int kAttnWarpsWide = 8;      // the same for groups of 9..16 query heads (more registers per thread)
constexpr int kAttnStageTokens = 16;   // tokens per pipeline stage (one PV MMA k-step)
constexpr int kAttnStages = 2;         // cp.async ring depth per warp: one stage computed, one in flight

// Launch shape of the sparse-attention kernel.
struct AttnPlan {
  int warps;            // warps per block: 12 (query-head groups up to 8) or 8
  int cluster;          // C: blocks per query row (a thread-block cluster), 1/2/4/8
  int heads_per_block;  // HC: KV heads served by one block (a power of two that divides the warps)
  int rows_per_block;   // RB: query rows served by one block (1 unless a chunk launch has short per-warp ranges)
  int subs;             // S = warps / HC / RB: token ranges of one row per block
  int head_groups;      // ceil(Hkv / HC): grid.y
  size_t smem_bytes;
};
// throughput: 0 = a launch on its own (whole-GPU shape); 1 = a few large blocks (the launch shares the GPU with its
// neighbours on the stream); 2 = the same with half the KV heads per block, where that is possible (twice the
// blocks: used for the last layers of a chain, see chain_fine_tail); 3 = the shape of a launch that computes two layers
// at once (8 warps with two head tiles each), also available to a single layer so that a pair's results can be
// reproduced; 4 = as 3 with half the KV heads per block where the plan cuts the step's blocks finely
AttnPlan make_attn_plan(const clsa_params& p, const DeviceInfo& dev, int throughput);
// The launch shapes of an L-layer chain: how many leading layers go two per launch, and how many trailing layers (of
// those, or of all when none are paired) use the finer shape (throughput = 4 or 2) so that the chain's blocks fill the
// SMs evenly to the end.
struct ChainTail {
  int layers;  // trailing layers that use the finer shape
  int paired;  // leading layers of the chain that are computed two per launch (even; 0 = none)
};
ChainTail chain_fine_tail(const clsa_params& p, const DeviceInfo& dev);

// Launch shape of the token-granular decode attention kernel (sparse_attn_sk.cu).
struct SkPlan {
  int warps;             // warps per block, each an autonomous worker
  int blocks;            // grid size: one block per SM (fewer for small launches)
  int workers;           // W: warps that get a span of the stage list (<= blocks * wpb, <= total_stages)
  int wpb;               // workers per block (<= warps)
  int aligned;           // 1: every unit has workers of its own (no span crosses a unit boundary); 0: flat split
  int unit_stages;       // NS = ceil(k / 16): 16-token stages per (query row, KV head) unit
  int64_t units;         // rows * Hkv
  int64_t total_stages;  // units * NS
  size_t smem_bytes;
};
SkPlan make_sk_plan(const clsa_params& p, const DeviceInfo& dev);
size_t sk_counter_bytes(const clsa_params& p, const SkPlan& plan);  // arrival counters of one launch
size_t sk_partial_bytes(const clsa_params& p, const SkPlan& plan);  // partial slots of one launch

struct TopkPlan {
  int cluster;      // blocks per (sequence, query) row, a thread-block cluster
  int slice_cap;    // score slots each block keeps in shared memory (0 = re-read global memory each pass)
  int one_sweep;    // the one-sweep kernel goes first; the general kernel then only finishes the rows it marks
  size_t smem_bytes;
};
// one_sweep_fits: whether the one-sweep kernel can take this launch (topk_prefilter_fits)
TopkPlan make_topk_plan(const clsa_params& p, const DeviceInfo& dev, bool one_sweep_fits);

struct WorkspaceLayout {
  // Scratch of a decode attention launch that has the GPU to itself (q_per_seq == 1; empty otherwise): arrival
  // counters, then partial slots.
  size_t attn_off, attn_bytes;
  size_t attn_counter_bytes;
  size_t attn_part_off;             // start of the partial slots
  size_t scores_off, scores_bytes;  // fp32 score matrix of clsa_decode_step
  int64_t score_stride;
  size_t total;
};
WorkspaceLayout make_workspace_layout(const clsa_params& p, const DeviceInfo& dev);

// ---------------------------------------------------------------------------------------------
// Kernel launchers (each returns the cudaError_t of its launches)
// ---------------------------------------------------------------------------------------------
// sched: two 32-bit counters, zero between launches, for the kernel's on-demand tile schedule (in a workspace they
// sit kSchedWord words behind the status word)
cudaError_t launch_index_scores_decode(const clsa_params& p, const void* q_idx, float* scores, int64_t score_stride,
                                       uint32_t* status, uint32_t* sched, const DeviceInfo& dev, cudaStream_t stream);
cudaError_t launch_index_scores_gemm(const clsa_params& p, const void* q_idx, float* scores, int64_t score_stride,
                                     uint32_t* status, const DeviceInfo& dev, cudaStream_t stream);
// Buffers of the fused chunk routing (clsa_index_topk, T > 1) that the GEMM's filtering and hand-back modes use.
struct GemmFused {
  const float* pivot;          // [rows] per query row: keys scoring below it cannot be among the row's k largest
  uint2* cand;                 // [rows][cand_cap] (score bits, position) candidates
  uint32_t* cand_count;        // [rows] candidates appended (may exceed cand_cap: the row overflowed)
  int cand_cap;
  const int32_t* slot_of_row;  // [rows] scratch row of a query row that was handed back, or -1
  const uint32_t* qblock_flag; // [num_seqs * ceil(T / 128)] query blocks that hold a handed-back row
  const uint32_t* nslots;      // rows handed back so far
};
cudaError_t launch_index_gemm_sample(const clsa_params& p, const void* q_idx, float* sample, int64_t sample_stride,
                                     int sample_gs, uint32_t* status, const DeviceInfo& dev, cudaStream_t stream);
int index_gemm_filter_hole_slack(const clsa_params& p, const DeviceInfo& dev);
cudaError_t launch_index_gemm_filter(const clsa_params& p, const void* q_idx, const GemmFused& fx, uint32_t* status,
                                     const DeviceInfo& dev, cudaStream_t stream);
cudaError_t launch_index_gemm_handed_back(const clsa_params& p, const void* q_idx, float* scratch, int64_t score_stride,
                                          const GemmFused& fx, uint32_t* status, const DeviceInfo& dev, cudaStream_t stream);
// Scores and TopK of a prefill chunk in one go, the score matrix never materialised (index_topk.cu). `scratch` is
// index_topk_scratch_bytes(p) bytes, 256-byte aligned; fits = false: the shape is outside what the fused route
// handles (the caller materialises the scores instead).
bool index_topk_fits(const clsa_params& p, const DeviceInfo& dev);
size_t index_topk_scratch_bytes(const clsa_params& p);
cudaError_t launch_index_topk(const clsa_params& p, const void* q_idx, int32_t* idx, int32_t* count, unsigned char* scratch,
                              uint32_t* status, const DeviceInfo& dev, cudaStream_t stream);
// Exact TopK of every row from its candidate list (topk_filter.cu); rows that cannot be finished get count = -1.
int topk_candidates_capacity();  // entries per row's list
size_t topk_candidates_smem(int max_seq_len, const DeviceInfo& dev);
cudaError_t launch_topk_candidates(const clsa_params& p, const uint2* cand, const uint32_t* cand_count, const float* pivot,
                                   int32_t* idx, int32_t* count, uint32_t* status, const DeviceInfo& dev, cudaStream_t stream);
// The general top-k kernel for the rows listed in row_of_slot[0 .. *nslots), row j reading row j of `scores`.
cudaError_t launch_topk_slots(const clsa_params& p, const float* scores, int64_t score_stride, const int32_t* row_of_slot,
                              const uint32_t* nslots, int max_slots, int32_t* idx, int32_t* count, uint32_t* status,
                              const DeviceInfo& dev, cudaStream_t stream);

cudaError_t launch_topk(const clsa_params& p, const float* scores, int64_t score_stride, int32_t* idx, int32_t* count,
                        uint32_t* status, const DeviceInfo& dev, cudaStream_t stream);
bool topk_prefilter_fits(const clsa_params& p, const float* scores, int64_t score_stride, const DeviceInfo& dev);
cudaError_t launch_topk_prefilter(const clsa_params& p, const float* scores, int64_t score_stride, int32_t* idx,
                                  int32_t* count, uint32_t* status, const DeviceInfo& dev, cudaStream_t stream);
// q2 / out2: nullptr, or the queries and outputs of a second layer that the same launch computes over the same staged
// rows (throughput_plan 3 or 4, groups of up to 8 query heads).
cudaError_t launch_sparse_attn(const clsa_params& p, const void* q, const int32_t* idx, const int32_t* count, void* out,
                               float* lse, uint32_t* status, int reverse, int wait_prior, int only_q_pending,
                               int keep_for_next, int throughput_plan, const void* q2, void* out2,
                               const DeviceInfo& dev, cudaStream_t stream);
// Share of its rounds of one-block-per-SM that the whole-unit kernel's launch-on-its-own shape fills (0..1).
double attn_alone_occupancy(const clsa_params& p, const DeviceInfo& dev);

// Decode attention with token-granular work items (q_per_seq == 1). arrive: sk_counter_bytes(plan) of counters that
// are zero (every launch leaves them so); part: sk_partial_bytes(p, plan) of partial slots. Launches in flight
// together need counters and slots of their own.
cudaError_t launch_sparse_attn_sk(const clsa_params& p, const SkPlan& plan, const void* q, const int32_t* idx,
                                  const int32_t* count, void* out, float* lse, uint32_t* status, uint32_t* arrive,
                                  float* part, int reverse, int wait_prior, int only_q_pending, int keep_rows,
                                  const DeviceInfo& dev, cudaStream_t stream);
// The same gather without the arithmetic (measurement aid); part as above (used as a sink).
cudaError_t launch_gather_probe(const clsa_params& p, const SkPlan& plan, const int32_t* idx, const int32_t* count,
                                uint32_t* status, float* part, int reverse, int keep_rows, const DeviceInfo& dev,
                                cudaStream_t stream);
// Of every 8 consecutive 16-token stages of a row's selected set, how many a decode launch with the GPU to itself
// fetches evict_last (the others evict_first) when the next launch reads the same rows again; -1: all of them.
int pinned_stages_of_eight(const clsa_params& p, const DeviceInfo& dev);

// idx_k_out / k_out / v_out: the caches of p, writable (k_out and v_out may be null together with w_k and w_v)
cudaError_t launch_project_append(const clsa_params& p, int d_model, const void* h, const void* w_q_idx,
                                  const void* w_k_idx, const void* w_k, const void* w_v, void* q_idx_out,
                                  void* idx_k_out, void* k_out, void* v_out,
                                  uint32_t* status, const DeviceInfo& dev, cudaStream_t stream);

// ---------------------------------------------------------------------------------------------
// Device helpers
// ---------------------------------------------------------------------------------------------
#ifdef __CUDACC__
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Round-to-nearest-even fp32 -> bf16 pair packed as (hi << 16) | lo.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

__device__ __forceinline__ void flag_status(uint32_t* status, uint32_t bit) {
  if (status != nullptr) atomicOr(status, bit);
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
#endif

}  // namespace clsa
