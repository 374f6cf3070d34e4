// C-ABI entry points: argument validation, workspace carving and the launch sequence.
// Every check that can refuse a call runs here on the host before anything is enqueued.
#include <math.h>
#include <mutex>

#include "common.cuh"

namespace clsa {

bool device_info(DeviceInfo* out) {
  static std::mutex mu;
  static DeviceInfo cache[64];
  static bool have[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return false; }
  if (dev < 0 || dev >= 64) return false;
  std::lock_guard<std::mutex> lock(mu);
  if (!have[dev]) {
    DeviceInfo d;
    if (cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&d.max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&d.l2_bytes, cudaDevAttrL2CacheSize, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&d.clock_khz, cudaDevAttrClockRate, dev) != cudaSuccess) {
      cudaGetLastError();
      return false;
    }
    cache[dev] = d;
    have[dev] = true;
  }
  *out = cache[dev];
  return true;
}

// header | scratch of the decode attention launches | fp32 score matrix of clsa_decode_step
WorkspaceLayout make_workspace_layout(const clsa_params& p, const DeviceInfo& dev) {
  WorkspaceLayout w;
  auto align = [](size_t x) { return (x + 255) / 256 * 256; };
  w.attn_off = kStatusBytes;
  w.attn_bytes = w.attn_counter_bytes = 0;
  w.attn_part_off = w.attn_off;
  if (p.q_per_seq == 1) {
    const SkPlan alone = make_sk_plan(p, dev);
    w.attn_counter_bytes = sk_counter_bytes(p, alone);
    w.attn_part_off = w.attn_off + w.attn_counter_bytes;
    w.attn_bytes = w.attn_counter_bytes + sk_partial_bytes(p, alone);
  }
  w.scores_off = w.attn_off + w.attn_bytes;
  w.score_stride = ((int64_t)p.max_seq_len + 63) / 64 * 64;
  w.scores_bytes = align((size_t)p.num_seqs * p.q_per_seq * w.score_stride * sizeof(float));
  // a prefill chunk's fused routing (clsa_index_topk) uses the same bytes for its own scratch instead
  const size_t fused = p.q_per_seq > 1 ? index_topk_scratch_bytes(p) : 0;
  w.total = w.scores_off + (w.scores_bytes > fused ? w.scores_bytes : fused);
  return w;
}

// L2 policy of a decode launch that has the GPU to itself and whose rows the next launch reads again (a decoder's
// layers issued one by one). If the selected set of the batch fits in the part of L2 that such a gather can keep
// (about half of it: rows are held on both sides of the chip), everything is fetched evict_last. If it does not, some
// of it is evicted before the next layer arrives whatever the order; then of every 8 consecutive 16-token stages the
// first few -- the share that fits -- are fetched evict_last and the others evict_first: every layer finds the same
// rows in L2; hits and misses alternate inside every warp's pipeline, so that the L2 port and HBM are busy together
// instead of one after the other (as they are when a launch first walks what its predecessor left behind and then
// the rest); and the rows that will not be kept anyway do not push the kept ones out.
int pinned_stages_of_eight(const clsa_params& p, const DeviceInfo& dev) {
  const double k_eff = (double)(p.top_k < p.max_seq_len ? p.top_k : p.max_seq_len);
  const double gathered = (double)p.num_seqs * p.q_per_seq * k_eff * p.num_kv_heads * p.head_dim * 4.0;
  const double keepable = 0.5 * (double)dev.l2_bytes;
  const int pin = (int)(8.0 * keepable / gathered + 0.5);
  return pin >= 8 ? -1 : (pin < 1 ? 1 : pin);
}

namespace {

bool aligned(const void* ptr, size_t a) { return (reinterpret_cast<uintptr_t>(ptr) % a) == 0; }

// Checks of the scalar fields only (shared by every entry point).
clsa_status check_shape(const clsa_params* p) {
  if (p == nullptr) return CLSA_ERR_INVALID_ARG;
  if (p->num_seqs < 1 || p->q_per_seq < 1 || p->num_q_heads < 1 || p->num_kv_heads < 1 || p->head_dim < 1 ||
      p->idx_dim < 1 || p->top_k < 1 || p->num_layers < 1)
    return CLSA_ERR_INVALID_ARG;
  if (p->num_q_heads % p->num_kv_heads != 0) return CLSA_ERR_INVALID_ARG;
  if (p->causal != 0 && p->causal != 1) return CLSA_ERR_INVALID_ARG;
  if (p->max_seq_len < p->q_per_seq) return CLSA_ERR_INVALID_ARG;
  if (!isfinite(p->sm_scale) || !(p->sm_scale > 0.f)) return CLSA_ERR_INVALID_ARG;  // the kernels take maxima before scaling
  if (p->num_layers > 4096) return CLSA_ERR_INVALID_ARG;
  // the decode attention kernel numbers its 16-token stages with 32 bits
  if ((double)p->num_seqs * p->q_per_seq * p->num_kv_heads * ((p->top_k + 15) / 16) >= 2147483648.0) return CLSA_ERR_UNSUPPORTED;
  if ((int64_t)p->num_seqs * p->q_per_seq > (int64_t)1 << 30) return CLSA_ERR_INVALID_ARG;
  if (p->head_dim != 128) return CLSA_ERR_UNSUPPORTED;
  if (p->idx_dim != 64 && p->idx_dim != 128) return CLSA_ERR_UNSUPPORTED;
  if (p->num_q_heads / p->num_kv_heads > 16) return CLSA_ERR_UNSUPPORTED;
  return CLSA_OK;
}

clsa_status check_seq(const clsa_params* p) {
  if (p->seq_len == nullptr || !aligned(p->seq_len, 4)) return CLSA_ERR_INVALID_ARG;
  if (p->block_table == nullptr) {
    if (p->seq_start == nullptr || !aligned(p->seq_start, 8)) return CLSA_ERR_INVALID_ARG;
  } else {
    if (!aligned(p->block_table, 4)) return CLSA_ERR_INVALID_ARG;
    const int bs = p->block_size;
    if (bs < 16 || bs > 4096 || (bs & (bs - 1)) != 0) return CLSA_ERR_INVALID_ARG;
    if ((int64_t)p->max_blocks_per_seq * bs < p->max_seq_len) return CLSA_ERR_INVALID_ARG;
  }
  return CLSA_OK;
}

clsa_status check_idx_cache(const clsa_params* p) {
  if (p->idx_k_cache == nullptr || !aligned(p->idx_k_cache, 16)) return CLSA_ERR_INVALID_ARG;
  if (p->idx_token_stride < p->idx_dim || p->idx_token_stride % 8 != 0) return CLSA_ERR_INVALID_ARG;
  return CLSA_OK;
}

clsa_status check_kv_cache(const clsa_params* p) {
  if (p->k_cache == nullptr || p->v_cache == nullptr) return CLSA_ERR_INVALID_ARG;
  if (!aligned(p->k_cache, 16) || !aligned(p->v_cache, 16)) return CLSA_ERR_INVALID_ARG;
  if (p->kv_head_stride < p->head_dim || p->kv_head_stride % 8 != 0) return CLSA_ERR_INVALID_ARG;
  if (p->kv_token_stride < p->head_dim || p->kv_token_stride % 8 != 0) return CLSA_ERR_INVALID_ARG;
  return CLSA_OK;
}

clsa_status check_workspace(const void* ws, size_t ws_bytes, size_t need) {
  if (ws == nullptr || !aligned(ws, 256) || ws_bytes < need) return CLSA_ERR_WORKSPACE;
  return CLSA_OK;
}

// Below this occupancy of the whole-unit shape a launch with the GPU to itself takes the token-granular kernel. Where
// the whole-unit shape fills about two thirds or more of its rounds it is as fast or faster (its merge stays inside a
// block, and while the rows come from DRAM idle SMs cost nothing); well below that the idle SMs dominate.
constexpr double kTokenGranularBelow = 0.6;

#define CLSA_TRY(expr)                     \
  do {                                     \
    const clsa_status st__ = (expr);       \
    if (st__ != CLSA_OK) return st__;      \
  } while (0)

clsa_status from_cuda(cudaError_t e) { return e == cudaSuccess ? CLSA_OK : CLSA_ERR_CUDA; }

clsa_status check_hints(const clsa_attn_hints* h) {
  if (h == nullptr) return CLSA_OK;
  for (int32_t v : {h->reverse, h->keep_rows, h->only_q_pending})
    if (v != 0 && v != 1) return CLSA_ERR_INVALID_ARG;
  if (h->shared_gpu < 0 || h->shared_gpu > 4) return CLSA_ERR_INVALID_ARG;
  return CLSA_OK;
}

// One attention launch. A decode launch (one query per sequence) that has the GPU to itself goes to the
// token-granular kernel and merges its split partials through the workspace; launches that share the GPU with their
// neighbours (chained layers) and chunk launches (T > 1, far more query rows than SMs) go to the kernel that gives
// whole (row, KV head) units to blocks.
cudaError_t launch_attention(const clsa_params& p, const void* q, const int32_t* idx, const int32_t* count, void* out,
                             float* lse, uint32_t* status, unsigned char* ws_base, const WorkspaceLayout& w,
                             const clsa_attn_hints& h, int wait_prior, const void* q2, void* out2,
                             const DeviceInfo& dev, cudaStream_t s) {
  // With the GPU to itself, a decode launch whose (row, KV head) units would leave many SMs idle in the last round of
  // whole-unit blocks (20 rows x 8 heads: 160 units on 148 SMs) cuts its work at token granularity instead.
  if (p.q_per_seq == 1 && h.shared_gpu == 0 && attn_alone_occupancy(p, dev) < kTokenGranularBelow) {
    const SkPlan plan = make_sk_plan(p, dev);
    auto arrive = reinterpret_cast<uint32_t*>(ws_base + w.attn_off);
    auto part = reinterpret_cast<float*>(ws_base + w.attn_part_off);
    return launch_sparse_attn_sk(p, plan, q, idx, count, out, lse, status, arrive, part, h.reverse, wait_prior,
                                 h.only_q_pending, h.keep_rows, dev, s);
  }
  return launch_sparse_attn(p, q, idx, count, out, lse, status, h.reverse, wait_prior, h.only_q_pending, h.keep_rows,
                            h.shared_gpu, q2, out2, dev, s);
}

// The L attention launches that share one index. Layer 0 follows whatever produced the index and must wait for it;
// every later layer reads only what was complete before its predecessor started (the index, the caches, the caller's
// queries), so it does not wait, and several layers are in flight at once. All of them walk the selected set in the
// same direction: a layer then trails its predecessor by a few microseconds over the same rows and finds them in L2.
// The end of the chain uses smaller blocks so that it ends flush (chain_fine_tail).
cudaError_t launch_layers(const clsa_params& p, const void* const* q_layers, void* const* out_layers, const int32_t* idx,
                          const int32_t* count, uint32_t* status, unsigned char* ws_base, const DeviceInfo& dev,
                          cudaStream_t s) {
  const WorkspaceLayout w = make_workspace_layout(p, dev);
  const ChainTail tail = chain_fine_tail(p, dev);
  // The leading layers two per launch: both read the same rows, which are then copied from L2 once for the two.
  for (int l = 0; l + 1 < tail.paired; l += 2) {
    const bool fine = l >= tail.paired - tail.layers;  // the last pairs of the chain in the finer shape
    const clsa_attn_hints h = {0, fine ? 4 : 3, l + 2 < p.num_layers ? 1 : 0, 0};
    const cudaError_t err = launch_attention(p, q_layers[l], idx, count, out_layers[l], nullptr, status, ws_base, w, h,
                                             l == 0 ? 1 : 0, q_layers[l + 1], out_layers[l + 1], dev, s);
    if (err != cudaSuccess) return err;
  }
  for (int l = tail.paired; l < p.num_layers; ++l) {
    const bool fine = tail.paired == 0 && l >= p.num_layers - tail.layers;
    const clsa_attn_hints h = {0, fine ? 2 : 1, l + 1 < p.num_layers ? 1 : 0, 0};
    const cudaError_t err = launch_attention(p, q_layers[l], idx, count, out_layers[l], nullptr, status, ws_base, w, h,
                                             l == 0 ? 1 : 0, nullptr, nullptr, dev, s);
    if (err != cudaSuccess) return err;
  }
  return cudaSuccess;
}

}  // namespace
}  // namespace clsa

using namespace clsa;

extern "C" {

clsa_status clsa_workspace_bytes(const clsa_params* p, size_t* bytes) {
  if (bytes == nullptr) return CLSA_ERR_INVALID_ARG;
  CLSA_TRY(check_shape(p));
  DeviceInfo dev;
  if (!device_info(&dev)) return CLSA_ERR_CUDA;
  *bytes = make_workspace_layout(*p, dev).total;
  return CLSA_OK;
}

clsa_status clsa_index_scores(const clsa_params* p, const void* q_idx, float* scores, int64_t score_stride,
                              void* workspace, size_t workspace_bytes, clsa_stream stream) {
  CLSA_TRY(check_shape(p));
  CLSA_TRY(check_seq(p));
  CLSA_TRY(check_idx_cache(p));
  if (q_idx == nullptr || scores == nullptr || !aligned(q_idx, 16) || !aligned(scores, 4)) return CLSA_ERR_INVALID_ARG;
  if (score_stride < p->max_seq_len) return CLSA_ERR_INVALID_ARG;
  if (p->q_per_seq > 1) {
    // the GEMM path addresses rows through 32-bit TMA coordinates and needs the extent of the cache
    if (p->num_cache_rows < 1 || p->num_cache_rows > 0x7fffffffLL) return CLSA_ERR_INVALID_ARG;
    if ((int64_t)p->num_seqs * p->q_per_seq > 0x7fffffffLL) return CLSA_ERR_INVALID_ARG;
  }
  CLSA_TRY(check_workspace(workspace, workspace_bytes, kStatusBytes));
  DeviceInfo dev;
  if (!device_info(&dev)) return CLSA_ERR_CUDA;
  if (p->q_per_seq > 1)
    return from_cuda(launch_index_scores_gemm(*p, q_idx, scores, score_stride, static_cast<uint32_t*>(workspace), dev,
                                              static_cast<cudaStream_t>(stream)));
  return from_cuda(launch_index_scores_decode(*p, q_idx, scores, score_stride, static_cast<uint32_t*>(workspace),
                                              static_cast<uint32_t*>(workspace) + kSchedWord, dev,
                                              static_cast<cudaStream_t>(stream)));
}

clsa_status clsa_topk(const clsa_params* p, const float* scores, int64_t score_stride, int32_t* idx, int32_t* count,
                      void* workspace, size_t workspace_bytes, clsa_stream stream) {
  CLSA_TRY(check_shape(p));
  CLSA_TRY(check_seq(p));
  if (scores == nullptr || idx == nullptr || count == nullptr) return CLSA_ERR_INVALID_ARG;
  if (!aligned(scores, 4) || !aligned(idx, 4) || !aligned(count, 4)) return CLSA_ERR_INVALID_ARG;
  if (score_stride < p->max_seq_len) return CLSA_ERR_INVALID_ARG;
  CLSA_TRY(check_workspace(workspace, workspace_bytes, kStatusBytes));
  DeviceInfo dev;
  if (!device_info(&dev)) return CLSA_ERR_CUDA;
  return from_cuda(launch_topk(*p, scores, score_stride, idx, count, static_cast<uint32_t*>(workspace), dev,
                               static_cast<cudaStream_t>(stream)));
}

clsa_status clsa_index_topk(const clsa_params* p, const void* q_idx, int32_t* idx, int32_t* count, void* workspace,
                            size_t workspace_bytes, clsa_stream stream) {
  CLSA_TRY(check_shape(p));
  CLSA_TRY(check_seq(p));
  CLSA_TRY(check_idx_cache(p));
  if (q_idx == nullptr || idx == nullptr || count == nullptr) return CLSA_ERR_INVALID_ARG;
  if (!aligned(q_idx, 16) || !aligned(idx, 4) || !aligned(count, 4)) return CLSA_ERR_INVALID_ARG;
  if (p->q_per_seq > 1) {
    if (p->num_cache_rows < 1 || p->num_cache_rows > 0x7fffffffLL) return CLSA_ERR_INVALID_ARG;
    if ((int64_t)p->num_seqs * p->q_per_seq > 0x7fffffffLL) return CLSA_ERR_INVALID_ARG;
  }
  if (workspace == nullptr || !aligned(workspace, 256)) return CLSA_ERR_WORKSPACE;
  DeviceInfo dev;
  if (!device_info(&dev)) return CLSA_ERR_CUDA;
  const WorkspaceLayout w = make_workspace_layout(*p, dev);
  CLSA_TRY(check_workspace(workspace, workspace_bytes, w.total));
  auto base = static_cast<unsigned char*>(workspace);
  auto status = reinterpret_cast<uint32_t*>(base);
  auto s = static_cast<cudaStream_t>(stream);
  if (p->q_per_seq > 1 && index_topk_fits(*p, dev))
    return from_cuda(launch_index_topk(*p, q_idx, idx, count, base + w.scores_off, status, dev, s));
  auto scores = reinterpret_cast<float*>(base + w.scores_off);
  cudaError_t err = p->q_per_seq > 1 ? launch_index_scores_gemm(*p, q_idx, scores, w.score_stride, status, dev, s)
                                     : launch_index_scores_decode(*p, q_idx, scores, w.score_stride, status, status + kSchedWord, dev, s);
  if (err != cudaSuccess) return CLSA_ERR_CUDA;
  return from_cuda(launch_topk(*p, scores, w.score_stride, idx, count, status, dev, s));
}

clsa_status clsa_sparse_attn_hinted(const clsa_params* p, const void* q, const int32_t* idx, const int32_t* count,
                                    void* out, float* lse, const clsa_attn_hints* hints, void* workspace,
                                    size_t workspace_bytes, clsa_stream stream) {
  CLSA_TRY(check_shape(p));
  CLSA_TRY(check_seq(p));
  CLSA_TRY(check_kv_cache(p));
  CLSA_TRY(check_hints(hints));
  if (q == nullptr || idx == nullptr || count == nullptr || out == nullptr) return CLSA_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(out, 16) || !aligned(idx, 4) || !aligned(count, 4) || !aligned(lse, 4))
    return CLSA_ERR_INVALID_ARG;
  if (workspace == nullptr || !aligned(workspace, 256)) return CLSA_ERR_WORKSPACE;
  DeviceInfo dev;
  if (!device_info(&dev)) return CLSA_ERR_CUDA;
  const WorkspaceLayout w = make_workspace_layout(*p, dev);
  const clsa_attn_hints h = hints != nullptr ? *hints : clsa_attn_hints{0, 0, 0, 0};
  // a decode launch with the GPU to itself merges its split partials through the scratch behind the header
  CLSA_TRY(check_workspace(workspace, workspace_bytes, p->q_per_seq == 1 && h.shared_gpu == 0 ? w.scores_off : kStatusBytes));
  auto base = static_cast<unsigned char*>(workspace);
  return from_cuda(launch_attention(*p, q, idx, count, out, lse, reinterpret_cast<uint32_t*>(base), base, w, h, 1, nullptr, nullptr, dev,
                                    static_cast<cudaStream_t>(stream)));
}

clsa_status clsa_sparse_attn(const clsa_params* p, const void* q, const int32_t* idx, const int32_t* count, void* out,
                             float* lse, void* workspace, size_t workspace_bytes, clsa_stream stream) {
  return clsa_sparse_attn_hinted(p, q, idx, count, out, lse, nullptr, workspace, workspace_bytes, stream);
}

clsa_status clsa_gather_probe(const clsa_params* p, const int32_t* idx, const int32_t* count, const clsa_attn_hints* hints,
                              void* workspace, size_t workspace_bytes, clsa_stream stream) {
  CLSA_TRY(check_shape(p));
  CLSA_TRY(check_seq(p));
  CLSA_TRY(check_kv_cache(p));
  CLSA_TRY(check_hints(hints));
  if (idx == nullptr || count == nullptr || !aligned(idx, 4) || !aligned(count, 4)) return CLSA_ERR_INVALID_ARG;
  if (p->q_per_seq != 1) return CLSA_ERR_UNSUPPORTED;
  if (workspace == nullptr || !aligned(workspace, 256)) return CLSA_ERR_WORKSPACE;
  DeviceInfo dev;
  if (!device_info(&dev)) return CLSA_ERR_CUDA;
  const WorkspaceLayout w = make_workspace_layout(*p, dev);
  CLSA_TRY(check_workspace(workspace, workspace_bytes, w.scores_off));
  const clsa_attn_hints h = hints != nullptr ? *hints : clsa_attn_hints{0, 0, 0, 0};
  auto base = static_cast<unsigned char*>(workspace);
  const SkPlan plan = make_sk_plan(*p, dev);
  return from_cuda(launch_gather_probe(*p, plan, idx, count, reinterpret_cast<uint32_t*>(base),
                                       reinterpret_cast<float*>(base + w.attn_part_off), h.reverse, h.keep_rows, dev,
                                       static_cast<cudaStream_t>(stream)));
}

// Argument checks shared by the two whole-step entry points.
static clsa_status check_step_args(const clsa_params* p, const void* q_idx, const void* const* q_layers,
                                   void* const* out_layers, const int32_t* idx, const int32_t* count) {
  CLSA_TRY(check_shape(p));
  CLSA_TRY(check_seq(p));
  CLSA_TRY(check_idx_cache(p));
  CLSA_TRY(check_kv_cache(p));
  if (q_idx == nullptr || q_layers == nullptr || out_layers == nullptr || idx == nullptr || count == nullptr)
    return CLSA_ERR_INVALID_ARG;
  if (!aligned(q_idx, 16) || !aligned(idx, 4) || !aligned(count, 4)) return CLSA_ERR_INVALID_ARG;
  for (int l = 0; l < p->num_layers; ++l)
    if (q_layers[l] == nullptr || out_layers[l] == nullptr || !aligned(q_layers[l], 16) || !aligned(out_layers[l], 16))
      return CLSA_ERR_INVALID_ARG;
  if (p->q_per_seq != 1) return CLSA_ERR_UNSUPPORTED;
  return CLSA_OK;
}

// index scores -> top-k -> L attention launches, all on `s`, scratch carved from `base` by `w`
static clsa_status run_step(const clsa_params* p, const void* q_idx, const void* const* q_layers, void* const* out_layers,
                            int32_t* idx, int32_t* count, unsigned char* base, uint32_t* status, const WorkspaceLayout& w,
                            const DeviceInfo& dev, cudaStream_t s) {
  auto scores = reinterpret_cast<float*>(base + w.scores_off);
  auto sched = reinterpret_cast<uint32_t*>(base) + kSchedWord;
  if (launch_index_scores_decode(*p, q_idx, scores, w.score_stride, status, sched, dev, s) != cudaSuccess) return CLSA_ERR_CUDA;
  if (launch_topk(*p, scores, w.score_stride, idx, count, status, dev, s) != cudaSuccess) return CLSA_ERR_CUDA;
  if (launch_layers(*p, q_layers, out_layers, idx, count, status, base, dev, s) != cudaSuccess) return CLSA_ERR_CUDA;
  return CLSA_OK;
}

clsa_status clsa_decode_step(const clsa_params* p, const void* q_idx, const void* const* q_layers,
                             void* const* out_layers, int32_t* idx, int32_t* count, void* workspace,
                             size_t workspace_bytes, clsa_stream stream) {
  CLSA_TRY(check_step_args(p, q_idx, q_layers, out_layers, idx, count));
  if (workspace == nullptr || !aligned(workspace, 256)) return CLSA_ERR_WORKSPACE;
  DeviceInfo dev;
  if (!device_info(&dev)) return CLSA_ERR_CUDA;
  const WorkspaceLayout w = make_workspace_layout(*p, dev);
  CLSA_TRY(check_workspace(workspace, workspace_bytes, w.total));
  auto base = static_cast<unsigned char*>(workspace);
  return run_step(p, q_idx, q_layers, out_layers, idx, count, base, reinterpret_cast<uint32_t*>(base), w, dev,
                  static_cast<cudaStream_t>(stream));
}

clsa_status clsa_sparse_attn_layers(const clsa_params* p, const void* const* q_layers, const int32_t* idx,
                                    const int32_t* count, void* const* out_layers, void* workspace,
                                    size_t workspace_bytes, clsa_stream stream) {
  CLSA_TRY(check_shape(p));
  CLSA_TRY(check_seq(p));
  CLSA_TRY(check_kv_cache(p));
  if (q_layers == nullptr || out_layers == nullptr || idx == nullptr || count == nullptr) return CLSA_ERR_INVALID_ARG;
  if (!aligned(idx, 4) || !aligned(count, 4)) return CLSA_ERR_INVALID_ARG;
  for (int l = 0; l < p->num_layers; ++l)
    if (q_layers[l] == nullptr || out_layers[l] == nullptr || !aligned(q_layers[l], 16) || !aligned(out_layers[l], 16))
      return CLSA_ERR_INVALID_ARG;
  if (workspace == nullptr || !aligned(workspace, 256)) return CLSA_ERR_WORKSPACE;
  DeviceInfo dev;
  if (!device_info(&dev)) return CLSA_ERR_CUDA;
  CLSA_TRY(check_workspace(workspace, workspace_bytes, kStatusBytes));
  auto base = static_cast<unsigned char*>(workspace);
  return from_cuda(launch_layers(*p, q_layers, out_layers, idx, count, reinterpret_cast<uint32_t*>(base), base, dev,
                                 static_cast<cudaStream_t>(stream)));
}

clsa_status clsa_project_append(const clsa_params* p, int32_t d_model, const void* h, const void* w_q_idx,
                                const void* w_k_idx, const void* w_k, const void* w_v, void* q_idx_out,
                                void* idx_k_cache_out, void* k_cache_out, void* v_cache_out, void* workspace,
                                size_t workspace_bytes, clsa_stream stream) {
  CLSA_TRY(check_shape(p));
  CLSA_TRY(check_seq(p));
  if (p->idx_token_stride < p->idx_dim || p->idx_token_stride % 8 != 0) return CLSA_ERR_INVALID_ARG;
  if (h == nullptr || w_q_idx == nullptr || w_k_idx == nullptr || q_idx_out == nullptr || idx_k_cache_out == nullptr)
    return CLSA_ERR_INVALID_ARG;
  if ((w_k == nullptr) != (w_v == nullptr)) return CLSA_ERR_INVALID_ARG;
  if ((w_k != nullptr) != (k_cache_out != nullptr) || (w_v != nullptr) != (v_cache_out != nullptr)) return CLSA_ERR_INVALID_ARG;
  if (!aligned(h, 16) || !aligned(w_q_idx, 16) || !aligned(w_k_idx, 16) || !aligned(w_k, 16) || !aligned(w_v, 16) ||
      !aligned(q_idx_out, 16) || !aligned(idx_k_cache_out, 16) || !aligned(k_cache_out, 16) || !aligned(v_cache_out, 16))
    return CLSA_ERR_INVALID_ARG;
  if (d_model < 32) return CLSA_ERR_INVALID_ARG;
  if (d_model % 32 != 0) return CLSA_ERR_UNSUPPORTED;
  if (w_k != nullptr) {
    if (p->kv_head_stride < p->head_dim || p->kv_head_stride % 8 != 0) return CLSA_ERR_INVALID_ARG;
    if (p->kv_token_stride < p->head_dim || p->kv_token_stride % 8 != 0) return CLSA_ERR_INVALID_ARG;
  }
  CLSA_TRY(check_workspace(workspace, workspace_bytes, kStatusBytes));
  DeviceInfo dev;
  if (!device_info(&dev)) return CLSA_ERR_CUDA;
  return from_cuda(launch_project_append(*p, d_model, h, w_q_idx, w_k_idx, w_k, w_v, q_idx_out, idx_k_cache_out, k_cache_out,
                                         v_cache_out, static_cast<uint32_t*>(workspace), dev, static_cast<cudaStream_t>(stream)));
}

// ---- entry point that allocates nothing -----------------------------------------------------------
// Scratch of clsa_decode_step_static: a whole workspace (status header, attention merge scratch, fp32 score
// matrix) in a file-scope device array that every GPU loading this library keeps until the process exits.
namespace {
constexpr size_t kStaticScratchBytes = kStatusBytes + ((size_t)16 << 20);
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code `g_static_scratch` is only a handle for the runtime, not a device address: the real
// address is asked for once per device, with that device current, and cached.
cudaError_t static_scratch_address(unsigned char** out) {
  static std::mutex mu;
  static unsigned char* addr[64] = {};
  int dev = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(mu);
  if (addr[dev] == nullptr) {
    void* ptr = nullptr;
    err = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (err != cudaSuccess) return err;
    addr[dev] = static_cast<unsigned char*>(ptr);
  }
  *out = addr[dev];
  return cudaSuccess;
}
}  // namespace

clsa_status clsa_decode_step_static(const clsa_params* p, const void* q_idx, const void* const* q_layers,
                                    void* const* out_layers, int32_t* idx, int32_t* count, uint32_t* dev_status,
                                    clsa_stream stream) {
  CLSA_TRY(check_step_args(p, q_idx, q_layers, out_layers, idx, count));
  if (!aligned(dev_status, 4)) return CLSA_ERR_INVALID_ARG;
  DeviceInfo dev;
  if (!device_info(&dev)) return CLSA_ERR_CUDA;
  const WorkspaceLayout w = make_workspace_layout(*p, dev);
  if (w.total > kStaticScratchBytes) return CLSA_ERR_WORKSPACE;  // beyond the fixed scratch
  unsigned char* base = nullptr;
  if (static_scratch_address(&base) != cudaSuccess) return CLSA_ERR_CUDA;
  auto s = static_cast<cudaStream_t>(stream);
  // The array keeps whatever the previous call left. What must start at zero is cleared on every call, whoever owns
  // the status word: the header (status word, the score kernel's ticket counters) -- a call that was cut short, or
  // two calls that raced, cannot poison later ones. The scores need no clearing (every entry that is read is written
  // first).
  if (cudaMemsetAsync(base, 0, kStatusBytes, s) != cudaSuccess) return CLSA_ERR_CUDA;
  uint32_t* status = dev_status != nullptr ? dev_status : reinterpret_cast<uint32_t*>(base);
  return run_step(p, q_idx, q_layers, out_layers, idx, count, base, status, w, dev, s);
}

clsa_status clsa_chain_plan(const clsa_params* p, int32_t sm_count, int32_t clock_khz, int32_t* fine_layers,
                            int32_t* paired_layers) {
  if (fine_layers == nullptr || paired_layers == nullptr || sm_count < 1 || clock_khz < 1) return CLSA_ERR_INVALID_ARG;
  CLSA_TRY(check_shape(p));
  DeviceInfo dev = {sm_count, 227 * 1024, 0, clock_khz};
  const ChainTail t = chain_fine_tail(*p, dev);
  *fine_layers = t.layers;
  *paired_layers = t.paired;
  return CLSA_OK;
}

clsa_status clsa_clear_status(void* workspace, size_t workspace_bytes, clsa_stream stream) {
  CLSA_TRY(check_workspace(workspace, workspace_bytes, kStatusBytes));
  return from_cuda(cudaMemsetAsync(workspace, 0, kStatusBytes, static_cast<cudaStream_t>(stream)));
}

clsa_status clsa_device_status(const void* workspace, uint32_t* bits, clsa_stream stream) {
  if (workspace == nullptr || bits == nullptr) return CLSA_ERR_INVALID_ARG;
  auto s = static_cast<cudaStream_t>(stream);
  cudaError_t err = cudaMemcpyAsync(bits, workspace, sizeof(uint32_t), cudaMemcpyDeviceToHost, s);
  if (err == cudaSuccess) err = cudaStreamSynchronize(s);
  return from_cuda(err);
}

const char* clsa_status_string(clsa_status s) {
  switch (s) {
    case CLSA_OK: return "ok";
    case CLSA_ERR_INVALID_ARG: return "invalid argument";
    case CLSA_ERR_UNSUPPORTED: return "unsupported shape";
    case CLSA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case CLSA_ERR_CUDA: return "CUDA runtime error";
  }
  return "unknown status";
}

int clsa_version(void) { return 200; }

}  // extern "C"
